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
