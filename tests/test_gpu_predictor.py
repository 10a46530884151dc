"""Phase 1 of ZipLine (constant-interval prediction) and both phases in one call, against the oracle."""
import numpy as np
import pytest
import torch

import oracle as o

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2001_01347_b200 as zl


def _cluster(rng, B, n):
    last = rng.integers(10 ** 9, 10 ** 9 + 10 ** 6, size=(B, n))
    iv = np.rint(np.exp(rng.normal(np.log(100_000), 0.5, size=(B, n)))).astype(np.int64)
    return last.astype(np.int64), iv


@pytest.mark.parametrize("n,R", [(4, 8), (33, 17), (128, 256), (1000, 15), (300, 150)])
def test_prediction_equals_oracle_elementwise(n, R):
    rng = np.random.default_rng(n * 1000 + R)
    last, iv = _cluster(rng, 3, n)
    iv[0, 0] = 0                                               # a stalled worker: all predictions equal
    got = zl.zl_predict_batched(torch.from_numpy(last).cuda(), torch.from_numpy(iv).cuda(), R).cpu().numpy()
    for b in range(3):
        assert (got[b] == o.predict(last[b], iv[b], R)).all()


@pytest.mark.parametrize("objective", [0, 1])
def test_both_phases_in_one_call(objective):
    rng = np.random.default_rng(5 + objective)
    for n, R, B in ((16, 64, 9), (257, 100, 3), (1024, 128, 2)):
        last, iv = _cluster(rng, B, n)
        h = zl.ZipLine(n, R, B, objective, 0, zl.ZL_FLAG_PREDICTOR)
        sel = h.predict_select_batched(torch.from_numpy(last).cuda(), torch.from_numpy(iv).cuda())
        torch.cuda.synchronize()
        for b in range(B):
            w, t, idx = o.sweep_window(o.predict(last[b], iv[b], R), objective)
            assert int(sel.status[b]) == 0
            assert (int(sel.wait[b]), int(sel.barrier[b])) == (w, t)
            assert (sel.idx[b].cpu().numpy() == idx).all()
        h.destroy()


def _check_fused(last, iv, R, options=None):
    """RANGE on predicted rows: both phases in one call (the matrix is never written for the filter route) must equal
    prediction followed by the search, and the oracle."""
    B, n = last.shape
    h = zl.ZipLine(n, R, B, 0, 0, zl.ZL_FLAG_PREDICTOR)
    for k, v in (options or {}).items():
        h.set_option(k, v)
    d_last, d_iv = torch.from_numpy(last).cuda(), torch.from_numpy(iv).cuda()
    ref = h.select_batched(zl.zl_predict_batched(d_last, d_iv, R))
    sel = h.predict_select_batched(d_last, d_iv)               # last, so that the counters below describe it
    torch.cuda.synchronize()
    for a, b in ((sel.idx, ref.idx), (sel.barrier, ref.barrier), (sel.wait, ref.wait), (sel.status, ref.status)):
        assert (a == b).all()
    for b in range(B):
        w, t, idx = o.sweep_window(o.predict(last[b], iv[b], R), 0)
        assert int(sel.status[b]) == 0
        assert (int(sel.wait[b]), int(sel.barrier[b])) == (w, t), b
        assert (sel.idx[b].cpu().numpy() == idx).all(), b
    counts = h.filter_counts(B)
    h.destroy()
    return counts


def test_fused_prediction_and_search_routes():
    rng = np.random.default_rng(77)
    # a heterogeneous cluster: few survivors, the single-CTA tail
    last, iv = _cluster(rng, 3, 300)
    iv[0, 5] = 0                                               # a stalled worker
    iv[1, :7] = 1                                              # very fast workers: the first exhausted row comes early
    filtered, refined, overflow = _check_fused(last, iv, 150)
    assert max(overflow) == 0 and max(filtered) <= 2048
    # a group of slow workers with nearly the same period: many elements raise the running maximum (cell scan,
    # refinement, buckets)
    B, n, R = 2, 512, 1024
    last = rng.integers(0, 10 ** 6, size=(B, n)).astype(np.int64)
    iv = np.where(np.arange(n) < n - 64, 80_000, 240_000).astype(np.int64)[None, :].repeat(B, 0)
    iv = iv + rng.integers(-2_000, 2_000, size=(B, n))         # nearly, not exactly, common periods
    filtered, refined, overflow = _check_fused(last, iv, R)
    assert max(overflow) == 0 and min(filtered) > 2048
    # identical workers: every element ties with n - 1 others, the lists overflow, the segment sweep takes over
    last = np.full((2, 200), 5_000, dtype=np.int64)
    iv = np.full((2, 200), 1_000, dtype=np.int64)
    filtered, refined, overflow = _check_fused(last, iv, 400)
    assert min(overflow) == 1
    # the segment sweep alone, and time spans beyond 32 bits (wide keys)
    last, iv = _cluster(rng, 2, 96)
    _check_fused(last, iv, 300, options={"no_filter": 1})
    _check_fused(last, iv * 200_000, 300)
    # n = 1 and R = 1
    _check_fused(np.array([[7]], dtype=np.int64), np.array([[3]], dtype=np.int64), 5000)
    _check_fused(rng.integers(0, 1000, size=(2, 5000)).astype(np.int64)[:, :4096], rng.integers(0, 1000, size=(2, 4096)).astype(np.int64), 2)


def test_fused_bad_inputs_mark_the_instance():
    rng = np.random.default_rng(78)
    last, iv = _cluster(rng, 4, 64)
    last[1, 10] = -1
    iv[2, 3] = -7
    iv[3, 63] = 2 ** 55                                        # the last prediction would pass 2^62
    h = zl.ZipLine(64, 128, 4, 0, 0, zl.ZL_FLAG_PREDICTOR)
    sel = h.predict_select_batched(torch.from_numpy(last).cuda(), torch.from_numpy(iv).cuda())
    torch.cuda.synchronize()
    bad = zl.binding.ZL_ERR_INVALID_ARG
    assert sel.status.tolist() == [0, bad, bad, bad]
    assert (sel.idx[1:] == -1).all() and (sel.wait[1:] == np.iinfo(np.int64).min).all()
    w, t, idx = o.sweep_window(o.predict(last[0], iv[0], 128), 0)
    assert (int(sel.wait[0]), int(sel.barrier[0])) == (w, t) and (sel.idx[0].cpu().numpy() == idx).all()
    h.destroy()


def test_bad_predictor_inputs_mark_the_instance():
    last = np.array([[100, 200, 300], [100, -5, 300], [100, 200, 2 ** 61]], dtype=np.int64)
    iv = np.array([[10, 20, 30], [10, 20, 30], [10, 20, 2 ** 60]], dtype=np.int64)
    h = zl.ZipLine(3, 4, 3, 0, 0, zl.ZL_FLAG_PREDICTOR)
    sel = h.predict_select_batched(torch.from_numpy(last).cuda(), torch.from_numpy(iv).cuda())
    torch.cuda.synchronize()
    assert sel.status.tolist() == [0, zl.binding.ZL_ERR_INVALID_ARG, zl.binding.ZL_ERR_INVALID_ARG]
    assert (sel.idx[1:] == -1).all()
    h.destroy()
    plain = zl.ZipLine(3, 4, 3)                                # no predictor buffer: the call is refused
    with pytest.raises(zl.ZipLineError):
        plain.predict_select_batched(torch.from_numpy(last).cuda(), torch.from_numpy(iv).cuda())
    plain.destroy()
