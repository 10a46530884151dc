"""Parity of the CUDA path against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle as o
import zl_inputs as zi
from conftest import load_hand_examples

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2001_01347_b200 as zl

OBJ = [0, 1]


def gpu_select(ts_np, objective, flags=0, options=None):
    ts_np = np.ascontiguousarray(ts_np, dtype=np.int64)
    B, n, R = ts_np.shape
    h = zl.ZipLine(n, R, B, objective, 0, flags)
    for k, v in (options or {}).items():
        h.set_option(k, v)
    d_ts = torch.from_numpy(ts_np).cuda()
    sel = h.select_batched(d_ts)
    torch.cuda.synchronize()
    got = (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy())
    if "no_filter" not in (options or {}):
        # each objective has two routes (RANGE: filter pass + one sort, SUM: time buckets; or the segment
        # sweep for both): they must agree exactly
        h.set_option("no_filter", 1)
        sel2 = h.select_batched(d_ts)
        torch.cuda.synchronize()
        for a, b in zip(got, (sel2.idx.cpu().numpy(), sel2.barrier.cpu().numpy(), sel2.wait.cpu().numpy(),
                              sel2.status.cpu().numpy())):
            assert (a == b).all(), "fast route and segment-sweep route disagree"
    h.destroy()
    return got


def assert_same(ts_np, objective, got, fn=None, which=None):
    idx, barrier, wait, status = got
    fn = fn or o.sweep_window
    which = range(ts_np.shape[0]) if which is None else which
    for b in which:
        w, t, ix = fn(ts_np[b], objective)
        assert status[b] == 0, (b, status[b])
        assert (int(wait[b]), int(barrier[b])) == (w, t), (b, objective, int(wait[b]), int(barrier[b]), w, t)
        assert (idx[b] == ix).all(), (b, idx[b][:8], ix[:8])


# ---------------------------------------------------------------- small cases
@pytest.mark.parametrize("objective", OBJ)
def test_hand_examples(objective):
    for name, M, rng_exp, sum_exp in load_hand_examples():
        exp = rng_exp if objective == 0 else sum_exp
        idx, barrier, wait, status = gpu_select(np.array([M]), objective)
        assert status[0] == 0
        assert (int(wait[0]), int(barrier[0]), idx[0].tolist()) == (exp[0], exp[1], exp[2]), name


@pytest.mark.parametrize("objective", OBJ)
@pytest.mark.parametrize("regime", ["dense", "sparse", "strict"])
def test_random_tiny_vs_enumerator(objective, regime):
    rng = np.random.default_rng(100 + objective)
    for n, R in ((1, 1), (1, 5), (2, 2), (3, 4), (4, 5), (5, 3), (2, 9), (6, 3)):
        B = 64
        if regime == "dense":
            inc, off = rng.integers(0, 4, size=(B, n, R)), rng.integers(0, 5, size=(B, n, 1))
        elif regime == "sparse":
            inc, off = rng.integers(0, 10 ** 9, size=(B, n, R)), rng.integers(0, 10 ** 9, size=(B, n, 1))
        else:
            inc, off = rng.integers(1, 50, size=(B, n, R)), rng.integers(0, 60, size=(B, n, 1))
        ts = (off + np.cumsum(inc, axis=2)).astype(np.int64)
        assert_same(ts, objective, gpu_select(ts, objective), fn=o.enumerate_all)


@pytest.mark.parametrize("checked", [0, 1])
@pytest.mark.parametrize("regime", ["dense", "sparse", "strict"])
def test_filter_route_on_tiny_shapes_vs_enumerator(regime, checked):
    # ZL_FLAG_FORCE_FILTER: the head, filter and tail kernels and the route's last kernel (cell scan, refinement, bucket
    # sweep, segment sweep, outputs) on shapes that the exhaustive search can check; with `checked`, the self-checking
    # variants of the kernels, which must find nothing to report
    rng = np.random.default_rng(300)
    flags = zl.ZL_FLAG_FORCE_FILTER | (zl.ZL_FLAG_DEBUG_CHECKS if checked else 0)
    for n, R in ((1, 1), (1, 5), (2, 2), (3, 4), (4, 5), (5, 3), (2, 9), (6, 3)):
        B = 64
        if regime == "dense":
            inc, off = rng.integers(0, 4, size=(B, n, R)), rng.integers(0, 5, size=(B, n, 1))
        elif regime == "sparse":
            inc, off = rng.integers(0, 10 ** 9, size=(B, n, R)), rng.integers(0, 10 ** 9, size=(B, n, 1))
        else:
            inc, off = rng.integers(1, 50, size=(B, n, R)), rng.integers(0, 60, size=(B, n, 1))
        ts = (off + np.cumsum(inc, axis=2)).astype(np.int64)
        h = zl.ZipLine(n, R, B, 0, 0, flags)
        assert h.route == 1
        sel = h.select_batched(torch.from_numpy(ts).cuda())
        torch.cuda.synchronize()
        assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()),
                    fn=o.enumerate_all)
        if checked:
            assert h.debug_report() == (0, 0, 0)
            nb, bad = h.check_canaries()
            assert nb > 0 and bad == 0
        h.destroy()


@pytest.mark.parametrize("variant", [1, 2])
def test_filter_ring_variants_are_exact(variant):
    # the filter pass whose rows arrive through a shared-memory ring filled by the copy engine (bulk copies counted on
    # mbarriers, 1) or by 16-byte copies of every lane (2): slower than the default kernels on these workloads, kept as
    # options, and exact
    for w in (zi.CONFIGS["c4"].with_(B=6, n=200, R=700), zi.CONFIGS["c3"].with_(B=40), zi.CONFIGS["c2"].with_(B=30, n=100, R=150)):
        ts = zi.generate(w)
        for flags in (0, zl.ZL_FLAG_DEBUG_CHECKS, zl.ZL_FLAG_FULL_SWEEP):
            h = zl.ZipLine(w.n, w.R, w.B, 0, 0, flags)
            h.set_option("filter_bulk", variant)
            sel = h.select_batched(torch.from_numpy(ts).cuda())
            torch.cuda.synchronize()
            assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))
            if flags & zl.ZL_FLAG_DEBUG_CHECKS:
                assert h.debug_report() == (0, 0, 0) and h.check_canaries()[1] == 0
            h.destroy()


@pytest.mark.parametrize("variant", [0, 1, 2])
def test_filter_route_rows_far_from_arithmetic(variant):
    # rows with rare long iterations among short ones: the number of a row's elements before the first exhausted row's
    # end is then badly estimated from the row's end points, and the filter pass has to go on past what it asked for
    rng = np.random.default_rng(302)
    for n, R, B in ((64, 100, 40), (17, 257, 300), (513, 256, 9), (129, 257, 17), (300, 1025, 3)):
        inc = np.where(rng.random((B, n, R)) < 0.02, 5000, rng.integers(1, 30, size=(B, n, R)))
        ts = (rng.integers(0, 1000, size=(B, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        for flags in (0, zl.ZL_FLAG_DEBUG_CHECKS):
            h = zl.ZipLine(n, R, B, 0, 0, flags)
            assert h.route == 1
            if variant:
                h.set_option("filter_bulk", variant)
            sel = h.select_batched(torch.from_numpy(ts).cuda())
            torch.cuda.synchronize()
            assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))
            if flags:
                assert h.debug_report() == (0, 0, 0) and h.check_canaries()[1] == 0
            h.destroy()


def test_many_survivor_phases_in_one_kernel_and_in_kernels_of_their_own():
    # instances with more survivors than one CTA finishes: the phases behind the tail kernel run inside the route's single
    # last kernel (grid-wide barriers between them) or as a kernel each; both must give the oracle's result
    rng = np.random.default_rng(303)
    shapes = [(100, 150, 40, 0), (128, 256, 64, 1), (257, 65, 9, 2)]
    for n, R, B, kind in shapes:
        if kind == 0:
            ts = zi.generate(zi.CONFIGS["c2"].with_(B=B, n=n, R=R))
        elif kind == 1:      # a homogeneous cluster: every row is slow, most elements raise the running maximum
            v = rng.integers(99_000, 101_000, size=(B, n, 1))
            ts = (rng.integers(0, 100_000, size=(B, n, 1)) + np.cumsum(v + rng.integers(0, 50, size=(B, n, R)), axis=2)).astype(np.int64)
        else:
            ts = (rng.integers(0, 5, size=(B, n, 1)) + np.cumsum(rng.integers(0, 3, size=(B, n, R)), axis=2)).astype(np.int64)
        for mode in (1, 2):
            got = gpu_select(ts, 0, options={"rest_split": mode})
            assert_same(ts, 0, got)
    # left to itself a handle takes the form from what its previous call met: a kernel per phase after a call with such
    # instances, the single kernel again after a call without
    heavy = ts_heavy = (rng.integers(0, 100_000, size=(8, 128, 1)) + np.cumsum(100_000 + rng.integers(0, 50, size=(8, 128, 256)), axis=2)).astype(np.int64)
    light = zi.generate(zi.CONFIGS["c3"].with_(B=8))
    h = zl.ZipLine(128, 256, 8, 0)
    assert h.launches_per_call == 4
    for ts, after in ((heavy, 9), (heavy, 9), (light, 4), (light, 4), (heavy, 9)):
        sel = h.select_batched(torch.from_numpy(ts).cuda())
        torch.cuda.synchronize()
        assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))
        assert h.launches_per_call == after
    h.destroy()


def test_filter_route_dense_ties_just_above_the_single_batch_size():
    # 256 instances of slightly more than 4096 timestamps with many equal values: the filter route's natural smallest shapes
    rng = np.random.default_rng(301)
    for n, R, hi in ((65, 64, 3), (33, 125, 2), (130, 32, 4)):
        B = 256
        ts = (rng.integers(0, 5, size=(B, n, 1)) + np.cumsum(rng.integers(0, hi, size=(B, n, R)), axis=2)).astype(np.int64)
        assert_same(ts, 0, gpu_select(ts, 0))


@pytest.mark.parametrize("objective", OBJ)
def test_ragged_medium_shapes_vs_sweep(objective):
    # sizes that span several batches / rounds and leave ragged tails (n, R not powers of two)
    rng = np.random.default_rng(7 + objective)
    for n, R, B, hi in ((7, 40, 9, 1000), (33, 17, 5, 30), (100, 150, 3, 10 ** 5), (10, 150, 4, 5000),
                        (257, 65, 2, 3), (1000, 15, 2, 200_000), (50, 1, 3, 100), (1, 300, 2, 10)):
        inc = rng.integers(0, hi, size=(B, n, R))
        ts = (rng.integers(0, 3 * hi, size=(B, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        assert_same(ts, objective, gpu_select(ts, objective))


@pytest.mark.parametrize("objective", OBJ)
def test_all_equal_and_identical_rows(objective):
    ts = np.full((2, 37, 50), 12345, dtype=np.int64)
    idx, barrier, wait, status = gpu_select(ts, objective)
    assert (status == 0).all() and (wait == 0).all() and (barrier == 12345).all() and (idx == 49).all()
    row = np.cumsum(np.arange(1, 201))
    ts = np.broadcast_to(row, (3, 300, 200)).astype(np.int64).copy()
    assert_same(ts, objective, gpu_select(ts, objective))


@pytest.mark.parametrize("objective", OBJ)
def test_uniform_shift_and_wide_spans(objective):
    w = zi.CONFIGS["c3"].with_(B=3, n=40, R=70)
    ts = zi.generate(w)
    base = gpu_select(ts, objective)
    assert_same(ts, objective, base)
    shift = 1_700_000_000_000_000
    idx, barrier, wait, status = gpu_select(ts + shift, objective)
    assert (idx == base[0]).all() and (wait == base[2]).all() and (barrier == base[1] + shift).all()
    # spans beyond 32 bits take the wide-key path
    wide = ts * 3000
    assert int(wide.max() - wide.min()) > 2 ** 33
    assert_same(wide, objective, gpu_select(wide, objective))


@pytest.mark.parametrize("objective", OBJ)
def test_launch_shapes_do_not_change_results(objective):
    w = zi.CONFIGS["c4"].with_(B=2, n=96, R=300)
    ts = zi.generate(w)
    ref = gpu_select(ts, objective)
    assert_same(ts, objective, ref)
    for opts in ({"segments": 7}, {"segments": 16, "threads": 128}, {"lanes_per_row": 1, "threads": 256},
                 {"lanes_per_row": 32, "segments": 3}, {"round_factor": 5}, {"round_factor": 2000, "segments": 2},
                 {"filter_round": 2}, {"filter_round": 8, "filter_threads": 64}, {"filter_round": 256}):
        got = gpu_select(ts, objective, options=opts)
        for a, b in zip(ref, got):
            assert (a == b).all(), opts
    full = gpu_select(ts, objective, flags=zl.ZL_FLAG_FULL_SWEEP, options={"segments": 5})
    for a, b in zip(ref, full):
        assert (a == b).all()


# ---------------------------------------------------------------- the five workloads
@pytest.mark.parametrize("objective", OBJ)
def test_config_c1_vs_enumerator(objective):
    ts = zi.generate(zi.CONFIGS["c1"])
    assert_same(ts, objective, gpu_select(ts, objective), fn=o.enumerate_all)


@pytest.mark.parametrize("objective", OBJ)
def test_config_c2_full_batch(objective):
    ts = zi.generate(zi.CONFIGS["c2"])
    got = gpu_select(ts, objective)
    assert_same(ts, objective, got)                               # every instance


@pytest.mark.parametrize("objective", OBJ)
def test_config_c3_full_batch(objective):
    ts = zi.generate(zi.CONFIGS["c3"])
    got = gpu_select(ts, objective)
    assert_same(ts, objective, got)                               # every instance


@pytest.mark.parametrize("objective", OBJ)
def test_config_c4_full_batch(objective):
    ts = zi.generate(zi.CONFIGS["c4"])
    got = gpu_select(ts, objective)
    assert (got[3] == 0).all()
    assert_same(ts, objective, got)                               # every instance


def test_config_c5_full_batch():
    # every instance, both objectives; the oracle runs in worker processes while this one holds the GPU
    from oracle_pool import solve_all
    w = zi.CONFIGS["c5"]
    expected = solve_all(w, range(w.B), OBJ)
    ts = zi.generate(w)
    for objective in OBJ:
        _check_c5(ts, objective, gpu_select(ts, objective), expected)


def _check_c5(ts, objective, got, expected):
    assert (got[3] == 0).all()
    for b in range(ts.shape[0]):
        wt, bar, ix = expected[(b, objective)]
        assert (int(got[2][b]), int(got[1][b])) == (wt, bar), (b, objective)
        assert (got[0][b] == ix).all(), (b, objective)
    # properties that hold for every instance at any size
    idx, barrier, wait, _ = got
    for b in range(ts.shape[0]):
        chosen = ts[b][np.arange(ts.shape[1]), idx[b]]
        assert chosen.max() == barrier[b] and (chosen <= barrier[b]).all()
        assert wait[b] == (barrier[b] - chosen.min() if objective == 0 else (barrier[b] - chosen).sum())


# ---------------------------------------------------------------- errors and flags
def test_per_instance_errors():
    ts = np.cumsum(np.ones((3, 4, 6), dtype=np.int64), axis=2) * 10
    ts[1, 2, 3] = 5                      # row 2 of instance 1 goes backwards
    idx, barrier, wait, status = gpu_select(ts, 0, flags=zl.ZL_FLAG_CHECK_SORTED)
    assert status.tolist() == [0, zl.binding.ZL_ERR_UNSORTED, 0]
    assert (idx[1] == -1).all() and barrier[1] == np.iinfo(np.int64).min and wait[1] == np.iinfo(np.int64).min
    assert_same(ts, 0, (idx, barrier, wait, status), which=[0, 2])
    ts2 = ts.copy()
    ts2[1] = ts[0]
    ts2[2, 0, 0] = -4                    # negative timestamp
    idx, barrier, wait, status = gpu_select(ts2, 0)
    assert status.tolist() == [0, 0, zl.binding.ZL_ERR_INVALID_ARG]


def test_round_limit_gives_timeout_and_the_handle_stays_usable():
    # the segment sweep with a round limit of 1: instances that need more rounds give up with ZL_ERR_TIMEOUT and the
    # sentinel outputs (nothing faults or hangs: the loop returns); the next call on the same handle is clean
    w = zi.CONFIGS["c2"].with_(B=6)
    ts = zi.generate(w)
    ts[2] = 1000                          # instance 2: one timestamp everywhere, a single round does it
    d = torch.from_numpy(ts).cuda()
    for objective in OBJ:
        h = zl.ZipLine(w.n, w.R, w.B, objective)
        h.set_option("no_filter", 1)
        h.set_option("max_rounds", 1)
        sel = h.select_batched(d)
        torch.cuda.synchronize()
        status = sel.status.cpu().numpy()
        assert (status[[0, 1, 3, 4, 5]] == zl.binding.ZL_ERR_TIMEOUT).all() and status[2] == 0
        bad = status != 0
        assert (sel.idx.cpu().numpy()[bad] == -1).all()
        assert (sel.barrier.cpu().numpy()[bad] == np.iinfo(np.int64).min).all() and (sel.wait.cpu().numpy()[bad] == np.iinfo(np.int64).min).all()
        assert_same(ts, objective, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), status), which=[2])
        h.set_option("max_rounds", 0)
        sel = h.select_batched(d)
        torch.cuda.synchronize()
        assert_same(ts, objective, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))
        h.destroy()


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_checked_kernels_find_nothing_and_canaries_survive(name):
    # ZL_FLAG_DEBUG_CHECKS: the index checks record no violation and no store ran past the end of a scratch buffer, on
    # every workload, both objectives; the results are the unchecked kernels'
    w = zi.CONFIGS[name]
    if name == "c2":
        w = w.with_(B=512)
    ts = zi.generate(w)
    d = torch.from_numpy(ts).cuda()
    for objective in OBJ:
        h = zl.ZipLine(w.n, w.R, w.B, objective, 0, zl.ZL_FLAG_DEBUG_CHECKS)
        sel = h.select_batched(d)
        torch.cuda.synchronize()
        assert h.debug_report() == (0, 0, 0)
        nb, bad = h.check_canaries()
        assert nb > 0 and bad == 0
        h2 = zl.ZipLine(w.n, w.R, w.B, objective)
        ref = h2.select_batched(d)
        torch.cuda.synchronize()
        assert (ref.status == 0).all()
        for a, b in ((sel.idx, ref.idx), (sel.barrier, ref.barrier), (sel.wait, ref.wait), (sel.status, ref.status)):
            assert torch.equal(a, b)
        assert h2.check_canaries() == (0, 0)
        h.destroy()
        h2.destroy()


def test_calls_from_another_device_are_refused():
    # the stream-ordered entry points only enqueue: with another device current they would launch on the wrong GPU
    if torch.cuda.device_count() < 2:
        pytest.skip("needs a second device to be current")
    h = zl.ZipLine(4, 4, 2)
    ts = torch.zeros((2, 4, 4), dtype=torch.int64, device="cuda:0")
    with torch.cuda.device(1):
        with pytest.raises(zl.ZipLineError) as e:
            h.select_batched(ts)
        assert e.value.code == zl.binding.ZL_ERR_INVALID_ARG
    h.destroy()


def test_host_detected_errors():
    with pytest.raises(zl.ZipLineError):
        zl.ZipLine(zl.zl_max_workers() + 1, 4, 1)
    with pytest.raises(zl.ZipLineError):
        zl.ZipLine(0, 4, 1)
    h = zl.ZipLine(4, 4, 2)
    ts = torch.zeros((3, 4, 4), dtype=torch.int64, device="cuda")
    with pytest.raises(zl.ZipLineError):
        h.select_batched(ts)             # B > max_batch
    with pytest.raises(zl.ZipLineError):
        h.set_option("no_such_option", 1)
    assert h.launches_per_call == 1 and h.workspace_bytes > 0      # tiny shape: one kernel does everything
    h.set_option("no_small", 1)
    assert h.launches_per_call == 5                                  # ... or the bucket route: prologue, plan, buckets, sweep, finalize
    h2 = zl.ZipLine(64, 128, 2)
    assert h2.launches_per_call == 4                                 # the filter route: head, filter, tail, one last kernel
    h2.destroy()
    h.destroy()


def test_host_buffer_entry_point_and_streams():
    w = zi.CONFIGS["c2"].with_(B=64)
    ts = zi.generate(w)
    h = zl.ZipLine(w.n, w.R, 64, 0)
    pinned = torch.from_numpy(ts).pin_memory()
    sel = h.select_batched_host(pinned)
    assert_same(ts, 0, (sel.idx.numpy(), sel.barrier.numpy(), sel.wait.numpy(), sel.status.numpy()))
    s = torch.cuda.Stream()
    d = torch.from_numpy(ts).cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(s):
        sel2 = h.select_batched(d[:10])
    s.synchronize()
    assert (sel2.wait.cpu() == sel.wait[:10]).all() and (sel2.idx.cpu() == sel.idx[:10]).all()
    h.destroy()


def test_read_probe_runs_on_any_layout():
    # the load-only measurement kernel: even and odd row lengths, counts beyond the row are clamped
    for R in (64, 77, 1024):
        ts = torch.arange(40 * R, dtype=torch.int64, device="cuda").reshape(40, R)
        count = torch.tensor([0, 1, R - 1, R, R + 50] * 8, dtype=torch.int32, device="cuda")
        sink = torch.zeros(1, dtype=torch.int64, device="cuda")
        zl.zl_probe_read_batched(ts, count, sink)
        zl.zl_probe_read_batched(ts[1:, :], count[1:], sink)           # rows that start 8 bytes off a 16-byte boundary when R is odd
        torch.cuda.synchronize()
    with pytest.raises(ValueError):
        zl.zl_probe_read_batched(ts, count[:3], sink)


# ---------------------------------------------------------------- per-step intermediates
def test_trace_matches_oracle_trace():
    rng = np.random.default_rng(17)
    for n, R, hi in ((4, 8, 50), (16, 64, 10 ** 6), (7, 33, 3), (1, 20, 10), (30, 1, 10), (64, 64, 100)):
        B = 5
        inc = rng.integers(0, hi, size=(B, n, R))
        ts = (rng.integers(0, 3 * hi, size=(B, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        tr = zl.zl_trace_batched(torch.from_numpy(ts).cuda())
        torch.cuda.synchronize()
        for b in range(B):
            ref = o.trace(ts[b])
            for k in ref:
                assert (tr[k][b].cpu().numpy() == ref[k]).all(), (k, n, R, b)


# ---------------------------------------------------------------- the three RANGE routes
def _routes(ts_np):
    B, n, R = ts_np.shape
    h = zl.ZipLine(n, R, B, 0)
    sel = h.select_batched(torch.from_numpy(ts_np).cuda())
    torch.cuda.synchronize()
    filtered, refined, overflow = h.filter_counts(B)
    h.destroy()
    return sel, np.array(filtered), np.array(refined), np.array(overflow)


def test_range_routes_are_all_exercised_and_exact():
    # few survivors: finished by the single-CTA tail
    ts = zi.generate(zi.CONFIGS["c4"].with_(B=3, n=256, R=512))
    sel, filtered, refined, overflow = _routes(ts)
    assert (overflow == 0).all() and (filtered <= 2048).all() and (filtered > 0).all()
    assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))
    # one common period per half of the workers: many elements raise the running maximum, so the
    # instance goes through cell scan, refinement and the bucket sweep
    ts = zi.generate(zi.CONFIGS["c5"].with_(B=3, n=512, R=1024))
    sel, filtered, refined, overflow = _routes(ts)
    assert (overflow == 0).all() and (filtered > 2048).all() and (refined > 0).all() and (refined <= filtered).all()
    assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))
    # identical rows: every element survives, the lists overflow, the segment sweep takes over
    row = np.cumsum(np.arange(1, 401))
    ts = np.broadcast_to(row, (2, 200, 400)).astype(np.int64).copy()
    sel, filtered, refined, overflow = _routes(ts)
    assert (overflow == 1).all()
    assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))


def test_mixed_batch_of_routes():
    # one batch holding a light, a heavy and an overflowing instance: the per-call flags must not let one starve another
    n, R = 256, 512
    light = zi.generate(zi.CONFIGS["c4"].with_(B=1, n=n, R=R))[0]
    heavy = zi.generate(zi.CONFIGS["c5"].with_(B=1, n=n, R=R))[0]
    same = np.broadcast_to(np.cumsum(np.arange(1, R + 1)) * 1000, (n, R)).astype(np.int64)
    ts = np.stack([light, heavy, same, light + 7, heavy + 11])
    sel, filtered, refined, overflow = _routes(ts)
    assert overflow.tolist() == [0, 0, 1, 0, 0]
    assert_same(ts, 0, (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy()))


# ---------------------------------------------------------------- the SUM routes
def _sum_routes(ts_np, options=None):
    B, n, R = ts_np.shape
    h = zl.ZipLine(n, R, B, 1)
    for k, v in (options or {}).items():
        h.set_option(k, v)
    sel = h.select_batched(torch.from_numpy(ts_np).cuda())
    torch.cuda.synchronize()
    buckets, tiles, overflow = h.filter_counts(B)
    h.destroy()
    got = (sel.idx.cpu().numpy(), sel.barrier.cpu().numpy(), sel.wait.cpu().numpy(), sel.status.cpu().numpy())
    return got, np.array(buckets), np.array(tiles), np.array(overflow)


def test_sum_routes_are_all_exercised_and_exact():
    # one bucket: the whole instance fits a shared-memory batch
    ts = zi.generate(zi.CONFIGS["c2"].with_(B=5, n=24, R=100))
    got, buckets, tiles, overflow = _sum_routes(ts, {"no_small": 1})
    assert (buckets == 1).all() and (tiles == 1).all() and (overflow == 0).all()
    assert_same(ts, 1, got)
    # several tiles of buckets, ragged last tile, rows of very different speeds
    ts = zi.generate(zi.CONFIGS["c4"].with_(B=3, n=200, R=700))
    got, buckets, tiles, overflow = _sum_routes(ts)
    assert (buckets > 30).all() and (tiles >= 3).all() and (overflow == 0).all()
    assert_same(ts, 1, got)
    # start offsets and two speeds (the rows do not start together)
    ts = zi.generate(zi.CONFIGS["c5"].with_(B=2, n=300, R=500))
    got, buckets, tiles, overflow = _sum_routes(ts)
    assert (buckets > 15).all() and (overflow == 0).all()
    assert_same(ts, 1, got)
    # rows far from arithmetic (quadratic growth): the early buckets overflow, the segment sweep takes over
    row = np.cumsum(np.arange(1, 401)) * 1000
    ts = np.broadcast_to(row, (2, 200, 400)).astype(np.int64).copy()
    ts += np.arange(200)[None, :, None]
    got, buckets, tiles, overflow = _sum_routes(ts)
    assert (overflow == 1).all()
    assert_same(ts, 1, got)


def test_sum_bucket_counts_around_tile_boundaries():
    # instance sizes chosen so that the number of buckets walks across multiples of the tile size (15 buckets):
    # the index table stores such a boundary twice, and the last tile may hold one bucket or fifteen
    seen = set()
    for k, R in enumerate((330, 352, 374, 396, 680, 704, 726, 1050)):
        n = 120
        ts = zi.generate(zi.CONFIGS["c3"].with_(B=2, n=n, R=R), first_instance=10 * k)
        got, buckets, tiles, overflow = _sum_routes(ts)
        assert (overflow == 0).all()
        seen.update(int(b) % 15 for b in buckets)
        assert_same(ts, 1, got)
    assert len(seen) >= 4                      # several different fillings of the last tile were exercised


def test_sum_buckets_with_heavy_ties_and_odd_shapes():
    rng = np.random.default_rng(4242)
    # many equal timestamps inside a bucket (slots fuller than the rank step allows: the comparison network takes over),
    # rows of odd length, a row count that is not a multiple of the CTA's threads
    for n, R, B, hi in ((77, 333, 3, 3), (130, 257, 2, 40), (513, 45, 2, 2000), (45, 1001, 2, 10 ** 6)):
        inc = rng.integers(0, hi, size=(B, n, R))
        ts = (rng.integers(0, 3 * hi, size=(B, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        got, buckets, tiles, overflow = _sum_routes(ts)
        assert_same(ts, 1, got)


@pytest.mark.parametrize("objective", OBJ)
def test_small_instances_one_launch_and_single_bucket_routes(objective):
    # instances of at most 4096 timestamps: one kernel does the whole search (route 3); with that route off they are
    # sorted whole by one CTA of the bucket route (route 2)
    rng = np.random.default_rng(99)
    for n, R, B, hi in ((16, 64, 300, 10 ** 5), (4096, 1, 2, 1000), (1, 4096, 2, 50), (63, 65, 5, 7), (2, 2048, 3, 10 ** 9), (1, 1, 3, 5)):
        inc = rng.integers(0, hi, size=(B, n, R))
        ts = (rng.integers(0, 3 * hi, size=(B, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        h = zl.ZipLine(n, R, B, objective)
        assert h.route == 3 and h.launches_per_call == 1
        h.set_option("no_small", 1)
        assert h.route == 2
        h.destroy()
        h = zl.ZipLine(n, R, 5000, objective)                # a batch of thousands: the bucket route
        assert h.route == 2
        h.destroy()
        assert_same(ts, objective, gpu_select(ts, objective))
        assert_same(ts, objective, gpu_select(ts, objective, options={"no_small": 1}))
    # errors per instance come out of the one kernel too
    ts = np.cumsum(np.ones((3, 4, 6), dtype=np.int64), axis=2) * 10
    ts[1, 2, 3] = 5
    ts[2, 0, 0] = -4
    idx, barrier, wait, status = gpu_select(ts, objective, flags=zl.ZL_FLAG_CHECK_SORTED)
    assert status.tolist() == [0, zl.binding.ZL_ERR_UNSORTED, zl.binding.ZL_ERR_INVALID_ARG]
    assert (idx[1:] == -1).all() and (barrier[1:] == np.iinfo(np.int64).min).all()


def test_range_filter_route_starts_above_the_small_sizes():
    h = zl.ZipLine(64, 65, 1, 0)
    assert h.route == 1                        # 4160 timestamps: the filter route
    h.destroy()


def test_sum_mixed_batch_of_routes():
    # a regular, an overflowing and a wide-span instance in one batch
    n, R = 128, 512
    regular = zi.generate(zi.CONFIGS["c4"].with_(B=1, n=n, R=R))[0]
    quad = (np.cumsum(np.arange(1, R + 1)) * 2000)[None, :] + np.arange(n)[:, None]
    wide = regular * 50_000
    ts = np.stack([regular, quad, wide, regular + 5]).astype(np.int64)
    got, buckets, tiles, overflow = _sum_routes(ts)
    assert overflow.tolist() == [0, 1, 0, 0] and buckets[2] == 0
    assert_same(ts, 1, got)


# ---------------------------------------------------------------- closed forms at a size no CPU check needs
def test_common_period_closed_forms_at_scale():
    # rows c_p + i * m with one period: RANGE = m - largest circular gap of the offsets, SUM = min_q sum_p ((c_q - c_p) mod m)
    rng = np.random.default_rng(2024)
    for n, R, m in ((1500, 600, 1_000_003), (4000, 64, 50_021), (300, 3000, 997)):
        B = 2
        c = rng.integers(0, m, size=(B, n))
        ts = (c[:, :, None] + m * np.arange(R)[None, None, :]).astype(np.int64)
        for objective in OBJ:
            idx, barrier, wait, status = gpu_select(ts, objective)
            assert (status == 0).all()
            for b in range(B):
                if objective == 0:
                    u = np.unique(c[b])
                    gaps = np.diff(np.concatenate([u, [u[0] + m]]))
                    expect = 0 if len(u) == 1 else m - int(gaps.max())
                else:
                    expect = int(((c[b][:, None] - c[b][None, :]) % m).sum(axis=1).min())
                assert int(wait[b]) == expect, (n, R, m, objective, b)
                chosen = ts[b][np.arange(n), idx[b]]
                assert chosen.max() == barrier[b]
                assert wait[b] == (barrier[b] - chosen.min() if objective == 0 else (barrier[b] - chosen).sum())


# ---------------------------------------------------------------- extreme shapes
@pytest.mark.parametrize("objective", OBJ)
def test_extreme_aspect_ratios(objective):
    rng = np.random.default_rng(900 + objective)
    nmax = zl.zl_max_workers()
    for n, R, B, hi in ((nmax, 3, 2, 1000), (nmax, 1, 1, 50), (2, 50_000, 2, 100), (1, 100_000, 1, 7),
                        (3000, 7, 2, 10 ** 5), (5, 4097, 3, 10 ** 4)):
        inc = rng.integers(0, hi, size=(B, n, R))
        ts = (rng.integers(0, 3 * hi, size=(B, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        assert_same(ts, objective, gpu_select(ts, objective))
    with pytest.raises(zl.ZipLineError):
        zl.ZipLine(nmax + 1, 2, 1, objective)
