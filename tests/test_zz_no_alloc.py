"""The entry point that allocates nothing, for callers that cannot call cudaMalloc.

A server thread living inside a process whose framework already owns all device memory, or a
loop that must never take the driver's allocation lock, cannot create a handle (zl_create
allocates the search's scratch).  zl_select_batched_noalloc keeps that scratch in a fixed array
inside the library.  This file checks, through the C ABI, that it returns exactly what the
handle-based entry point returns, twice in a row (the array keeps the previous call's contents),
and that it refuses batches beyond its stated maximum.  It is collected after every other test
file on purpose.
"""
import numpy as np
import pytest
import torch

import oracle as o
import zl_inputs as zi

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2001_01347_b200 as zl


def _empty_selection(B, n):
    return zl.Selection(torch.full((B, n), -7, dtype=torch.int32, device="cuda"),
                        torch.full((B,), -7, dtype=torch.int64, device="cuda"),
                        torch.full((B,), -7, dtype=torch.int64, device="cuda"),
                        torch.full((B,), -7, dtype=torch.int32, device="cuda"))


@pytest.mark.parametrize("objective", [0, 1])
def test_noalloc_matches_handle_path_on_two_calls_in_a_row(objective):
    # two different shapes back to back: the second call finds the first call's records in the array
    shapes = [zi.CONFIGS["c4"].with_(B=3, n=96, R=300), zi.CONFIGS["c2"].with_(B=40)]
    for w in shapes:
        ts = torch.from_numpy(zi.generate(w)).cuda()
        h = zl.ZipLine(w.n, w.R, w.B, objective)
        ref = h.select_batched(ts)
        torch.cuda.synchronize()
        got = zl.zl_select_batched_noalloc(ts, _empty_selection(w.B, w.n), objective)
        torch.cuda.synchronize()
        # integer results: exact equality is the tolerance every parity test here uses
        assert (got.status == 0).all() and (ref.status == 0).all()
        assert torch.equal(got.idx, ref.idx)
        assert torch.equal(got.barrier, ref.barrier)
        assert torch.equal(got.wait, ref.wait)
        h.destroy()


@pytest.mark.parametrize("objective", [0, 1])
def test_noalloc_against_the_oracle_with_a_bad_instance_and_the_sortedness_check(objective):
    w = zi.CONFIGS["c2"].with_(B=5, n=12, R=40)
    ts = zi.generate(w)
    ts[3, 7, 0] = -9                      # a negative timestamp: this instance alone is refused
    got = zl.zl_select_batched_noalloc(torch.from_numpy(ts).cuda(), _empty_selection(w.B, w.n), objective)
    torch.cuda.synchronize()
    status = got.status.cpu().numpy()
    assert status.tolist() == [0, 0, 0, zl.binding.ZL_ERR_INVALID_ARG, 0]
    assert (got.idx.cpu().numpy()[3] == -1).all()
    for b in (0, 1, 2, 4):
        wt, bar, ix = o.sweep(ts[b], objective)
        assert (int(got.wait[b]), int(got.barrier[b])) == (wt, bar) and (got.idx[b].cpu().numpy() == ix).all()
    # with the sortedness check: a row that goes backwards is reported for its instance only
    ts2 = zi.generate(w)
    ts2[1, 2, 5] = ts2[1, 2, 3] - 1
    got = zl.zl_select_batched_noalloc(torch.from_numpy(ts2).cuda(), _empty_selection(w.B, w.n), objective, zl.ZL_FLAG_CHECK_SORTED)
    torch.cuda.synchronize()
    assert got.status.cpu().tolist() == [0, zl.binding.ZL_ERR_UNSORTED, 0, 0, 0]
    for b in (0, 2, 3, 4):
        wt, bar, ix = o.sweep(ts2[b], objective)
        assert (int(got.wait[b]), int(got.barrier[b])) == (wt, bar) and (got.idx[b].cpu().numpy() == ix).all()


def test_noalloc_rejects_batches_beyond_the_fixed_scratch():
    B = zl.zl_noalloc_max_batch() + 1
    ts = torch.from_numpy(np.cumsum(np.ones((B, 2, 3), dtype=np.int64), axis=2)).cuda()
    with pytest.raises(zl.ZipLineError) as e:
        zl.zl_select_batched_noalloc(ts, _empty_selection(B, 2))
    assert e.value.code == zl.binding.ZL_ERR_UNSUPPORTED
    assert 0 < zl.zl_noalloc_scratch_bytes() < 1 << 20
