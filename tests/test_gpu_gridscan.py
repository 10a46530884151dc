"""The paper's heuristic baselines (Algorithm 1: GridScan, FullGridScan) on the GPU against the oracle."""
import numpy as np
import pytest
import torch

import oracle as o
import zl_inputs as zi

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2001_01347_b200 as zl


def _check(ts, full):
    idx, barrier, wait = zl.zl_gridscan_batched(torch.from_numpy(ts).cuda(), full)
    torch.cuda.synchronize()
    idx, barrier, wait = idx.cpu().numpy(), barrier.cpu().numpy(), wait.cpu().numpy()
    for b in range(ts.shape[0]):
        w, t, ix = o.gridscan(ts[b], full)
        assert (int(wait[b]), int(barrier[b])) == (w, t), (b, full)
        assert (idx[b] == ix).all()
    return wait


@pytest.mark.parametrize("full", [False, True])
def test_random_small_instances_with_ties(full):
    rng = np.random.default_rng(31 + full)
    for n, R, hi in ((1, 1, 5), (2, 3, 4), (5, 6, 3), (7, 9, 50), (33, 17, 10 ** 6), (3, 40, 5)):
        inc = rng.integers(0, hi, size=(12, n, R))
        ts = (rng.integers(0, 3 * hi, size=(12, n, 1)) + np.cumsum(inc, axis=2)).astype(np.int64)
        _check(ts, full)


@pytest.mark.parametrize("full", [False, True])
def test_paper_table_shapes_and_quality_against_the_exact_search(full):
    for name in ("t2_n10_R15", "t2_n10_R150", "t2_n100_R15"):
        w = zi.CONFIGS[name].with_(B=6)
        ts = zi.generate(w)
        wait = _check(ts, full)
        h = zl.ZipLine(w.n, w.R, 6, 0)
        exact = h.select_batched(torch.from_numpy(ts).cuda()).wait.cpu().numpy()
        h.destroy()
        assert (wait >= exact).all()                       # the heuristics never beat the optimum
