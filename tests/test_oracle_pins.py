"""Pins for the CPU oracle: everything here runs without a GPU.

The oracle is checked against things that are not the oracle: hand-worked
examples, a pure-Python enumeration of all R^n combinations written straight
from the definition (Section III), the textbook smallest-range-over-k-lists
routine, a closed form, and invariants of the definition.
"""
import heapq
import itertools

import numpy as np
import pytest

import oracle as o
from conftest import load_hand_examples

OBJ = [o.RANGE, o.SUM]


# ------------------------------------------------------------------ independent references
def brute_python(M, objective):
    """All R^n choices, straight from the definition; ties -> smallest barrier, then largest indices."""
    n, R = len(M), len(M[0])
    best = None
    for j in itertools.product(range(R), repeat=n):
        Z = [M[p][j[p]] for p in range(n)]
        mx = max(Z)
        d = mx - min(Z) if objective == o.RANGE else sum(mx - z for z in Z)
        key = (d, mx, tuple(-x for x in j))
        if best is None or key < best:
            best = key
    return best[0], best[1], [-x for x in best[2]]


def smallest_range_heap(M):
    """Textbook k-pointer routine: advance the list that holds the current minimum."""
    n, R = len(M), len(M[0])
    heap = [(M[p][0], p, 0) for p in range(n)]
    heapq.heapify(heap)
    cur_max = max(M[p][0] for p in range(n))
    best = None
    while True:
        t, p, i = heap[0]
        if best is None or cur_max - t < best:
            best = cur_max - t
        if i + 1 == R:
            return best
        heapq.heapreplace(heap, (M[p][i + 1], p, i + 1))
        cur_max = max(cur_max, M[p][i + 1])


def random_instance(rng, regime):
    n = int(rng.integers(1, 6))
    R = int(rng.integers(1, 7))
    if n ** 1 and R ** n > 8000:
        R = max(1, int(8000 ** (1.0 / n)))
    if regime == "dense":          # small ints, many ties, zero-length iterations allowed
        inc = rng.integers(0, 4, size=(n, R))
        off = rng.integers(0, 5, size=(n, 1))
    elif regime == "sparse":
        inc = rng.integers(0, 10 ** 9, size=(n, R))
        off = rng.integers(0, 10 ** 9, size=(n, 1))
    else:                          # strictly increasing, moderate
        inc = rng.integers(1, 50, size=(n, R))
        off = rng.integers(0, 60, size=(n, 1))
    return (off + np.cumsum(inc, axis=1)).astype(np.int64)


# ------------------------------------------------------------------ hand examples
@pytest.mark.parametrize("ex", load_hand_examples(), ids=lambda e: e[0])
@pytest.mark.parametrize("fn", [o.enumerate_all, o.sweep, o.sweep_window], ids=lambda f: f.__name__)
def test_hand_examples(ex, fn):
    _, M, rng_exp, sum_exp = ex
    for obj, exp in ((o.RANGE, rng_exp), (o.SUM, sum_exp)):
        w, b, idx = fn(M, obj)
        assert (w, b, list(idx)) == (exp[0], exp[1], exp[2])


@pytest.mark.parametrize("ex", load_hand_examples(), ids=lambda e: e[0])
def test_hand_examples_python_brute(ex):
    _, M, rng_exp, sum_exp = ex
    assert brute_python(M, o.RANGE) == (rng_exp[0], rng_exp[1], rng_exp[2])
    assert brute_python(M, o.SUM) == (sum_exp[0], sum_exp[1], sum_exp[2])


def test_first_of_two_equal_minima_is_chosen():
    # Fig. 3 caption: two equal minima, the earlier one is taken.
    M = [[10, 30, 50, 70], [12, 32, 55, 72]]
    for fn in (o.enumerate_all, o.sweep, o.sweep_window):
        assert fn(M, o.RANGE)[:2] == (2, 12)
    assert o.alg2(M)[:2] == (2, 12)


# ------------------------------------------------------------------ brute force on tiny inputs
@pytest.mark.parametrize("regime", ["dense", "sparse", "strict"])
@pytest.mark.parametrize("objective", OBJ)
def test_all_functions_equal_brute_force(regime, objective):
    rng = np.random.default_rng(1234 + objective + 17 * len(regime))
    for _ in range(400):
        M = random_instance(rng, regime)
        ref = brute_python(M.tolist(), objective)
        for fn in (o.enumerate_all, o.sweep, o.sweep_window):
            w, b, idx = fn(M, objective)
            assert (w, b, list(idx)) == ref, (fn.__name__, M.tolist())


@pytest.mark.parametrize("regime", ["dense", "sparse", "strict"])
def test_algorithm2_listing_and_heap_agree_on_wait_and_barrier(regime):
    rng = np.random.default_rng(99 + len(regime))
    for _ in range(600):
        M = random_instance(rng, regime)
        w, b, _ = o.sweep(M, o.RANGE)
        w2, b2, idx2 = o.alg2(M)
        assert (w2, b2) == (w, b), M.tolist()
        Z = [M[p][idx2[p]] for p in range(M.shape[0])]
        assert max(Z) - min(Z) == w and max(Z) == b     # Z* of the listing is a true minimiser
        assert smallest_range_heap(M.tolist()) == w


def test_medium_sizes_window_equals_plain_sweep():
    rng = np.random.default_rng(5)
    for n, R in ((7, 40), (33, 17), (64, 64), (1, 50), (50, 1)):
        inc = rng.integers(0, 1000, size=(n, R))
        M = rng.integers(0, 3000, size=(n, 1)) + np.cumsum(inc, axis=1)
        for obj in OBJ:
            a = o.sweep(M, obj)
            b = o.sweep_window(M, obj)
            assert a[:2] == b[:2] and list(a[2]) == list(b[2])
        assert smallest_range_heap(M.tolist()) == o.sweep(M, o.RANGE)[0]


# ------------------------------------------------------------------ closed form
def test_common_period_closed_form():
    # rows e^p_i = c_p + i*m with one period m and R >= 2: the best window misses only the
    # largest circular gap between the distinct offsets.
    rng = np.random.default_rng(7)
    for _ in range(200):
        n = int(rng.integers(1, 9))
        m = int(rng.integers(5, 400))
        R = int(rng.integers(2, 9))
        c = rng.integers(0, m, size=n)
        M = c[:, None] + m * np.arange(R)[None, :]
        u = np.unique(c)
        gaps = np.diff(np.concatenate([u, [u[0] + m]]))
        expect = 0 if len(u) == 1 else m - int(gaps.max())
        assert o.sweep(M, o.RANGE)[0] == expect
        assert o.sweep_window(M, o.RANGE)[0] == expect


def test_common_period_closed_form_for_the_total_wait():
    # same rows, SUM objective, R >= 3: while every row still has elements the total wait at time T is
    # sum_p ((T - c_p) mod m), candidates are the element times, so the minimum is min_q sum_p ((c_q - c_p) mod m);
    # after the rows run out the wait only grows.  The barrier is congruent to a minimising offset.
    rng = np.random.default_rng(8)
    for _ in range(200):
        n = int(rng.integers(1, 9))
        m = int(rng.integers(5, 400))
        R = int(rng.integers(3, 9))
        c = rng.integers(0, m, size=n)
        M = c[:, None] + m * np.arange(R)[None, :]
        totals = ((c[:, None] - c[None, :]) % m).sum(axis=1)           # totals[q] = sum_p ((c_q - c_p) mod m)
        expect = int(totals.min())
        for fn in (o.sweep, o.sweep_window):
            wait, barrier, idx = fn(M, o.SUM)
            assert wait == expect
            assert barrier % m in set((c[totals == expect] % m).tolist())
            assert barrier <= int(c.max()) + m                           # the first minimum comes within one period


# ------------------------------------------------------------------ invariants of the definition
def _rand_rows(rng, n, R, hi=500):
    return rng.integers(0, hi, size=(n, 1)) + np.cumsum(rng.integers(0, hi, size=(n, R)), axis=1)


@pytest.mark.parametrize("objective", OBJ)
def test_invariants(objective):
    rng = np.random.default_rng(2024)
    for _ in range(150):
        n, R = int(rng.integers(1, 12)), int(rng.integers(1, 12))
        M = _rand_rows(rng, n, R)
        w, b, idx = o.sweep(M, objective)
        # bracket: chosen element <= barrier < next element; someone finishes exactly at the barrier
        chosen = M[np.arange(n), idx]
        assert (chosen <= b).all() and chosen.max() == b
        for p in range(n):
            if idx[p] + 1 < R:
                assert M[p, idx[p] + 1] > b
        assert b >= M[:, 0].max()
        # the reported wait is the objective of the reported selection
        assert w == (b - chosen.min() if objective == o.RANGE else int((b - chosen).sum()))
        # uniform shift
        c = 10 ** 15
        w2, b2, idx2 = o.sweep(M + c, objective)
        assert (w2, b2 - c, list(idx2)) == (w, b, list(idx))
        # permuting workers permutes idx only
        perm = rng.permutation(n)
        w3, b3, idx3 = o.sweep(M[perm], objective)
        assert (w3, b3) == (w, b) and list(idx3) == list(idx[perm])
        # one more, later, element per row can only keep or lower the wait
        ext = np.concatenate([M, M.max() + 1 + rng.integers(0, 50, size=(n, 1))], axis=1)
        assert o.sweep(ext, objective)[0] <= w


def test_objectives_bracket_each_other():
    rng = np.random.default_rng(11)
    for _ in range(200):
        n, R = int(rng.integers(1, 10)), int(rng.integers(1, 10))
        M = _rand_rows(rng, n, R)
        wr = o.sweep(M, o.RANGE)[0]
        ws = o.sweep(M, o.SUM)[0]
        assert 0 <= wr <= ws <= max(n - 1, 1) * wr or (n == 1 and wr == ws == 0)


def test_all_equal_timestamps_give_zero_wait():
    M = np.full((5, 6), 42, dtype=np.int64)
    for obj in OBJ:
        for fn in (o.enumerate_all, o.sweep, o.sweep_window):
            w, b, idx = fn(M, obj)
            assert (w, b, list(idx)) == (0, 42, [5] * 5)


def test_unsorted_row_is_rejected():
    with pytest.raises(ValueError):
        o.sweep([[3, 2, 5], [1, 2, 3]], o.RANGE)


def test_large_magnitudes():
    base = 2 ** 61
    M = np.array([[base, base + 10, base + 30], [base + 4, base + 29, base + 31]], dtype=np.int64)
    assert o.sweep(M, o.RANGE)[:2] == (1, base + 30)
    assert o.sweep(M, o.SUM)[:2] == (1, base + 30)
    assert brute_python(M.tolist(), o.RANGE)[:2] == (1, base + 30)


# ------------------------------------------------------------------ the per-position trace
def test_trace_matches_the_selection():
    rng = np.random.default_rng(3)
    for _ in range(200):
        n, R = int(rng.integers(1, 7)), int(rng.integers(1, 9))
        M = _rand_rows(rng, n, R, hi=int(rng.choice([3, 40, 10 ** 6])))
        tr = o.trace(M)
        # Omega is a sorted permutation of the matrix
        assert (np.diff(tr["om_t"]) >= 0).all()
        assert (M[tr["om_p"], tr["om_i"]] == tr["om_t"]).all()
        assert len(set(zip(tr["om_p"].tolist(), tr["om_i"].tolist()))) == n * R
        # S is the sum over started workers of their latest element (direct recomputation)
        k = int(rng.integers(0, n * R))
        last = {}
        for q in range(k + 1):
            last[int(tr["om_p"][q])] = int(tr["om_t"][q])
        assert tr["S"][k] == sum(last.values()) and tr["cnt"][k] == len(last)
        # every array at every position, straight from its definition (no running state)
        N = n * R
        INF, NINF = np.iinfo(np.int64).max, np.iinfo(np.int64).min
        t0 = int(M[:, 0].max())
        for q in range(N):
            wp, wi, wt = int(tr["om_p"][q]), int(tr["om_i"][q]), int(tr["om_t"][q])
            assert tr["delta"][q] == (wt if wi == 0 else wt - int(M[wp, wi - 1]))
            assert tr["first"][q] == (1 if wi == 0 else 0)
            assert tr["next"][q] == (INF if wi == R - 1 else int(M[wp, wi + 1]))
            before = [INF if int(tr["om_i"][j]) == R - 1 else int(M[int(tr["om_p"][j]), int(tr["om_i"][j]) + 1]) for j in range(q)]
            pm = max(before) if before else NINF
            assert tr["PM"][q] == pm
            latest = {}
            for j in range(q + 1):
                latest[int(tr["om_p"][j])] = int(tr["om_t"][j])
            assert tr["S"][q] == sum(latest.values()) and tr["cnt"][q] == len(latest)
            g = max(wt, t0, pm)
            assert tr["d_range"][q] == (INF if g == INF else g - wt)
            assert tr["w_sum"][q] == (n * wt - sum(latest.values()) if len(latest) == n else INF)
        # minimum over positions reproduces the selection, with the first-minimum rule
        w, b, _ = o.sweep(M, o.RANGE)
        d = tr["d_range"]
        kmin = int(np.argmin(d))
        assert d[kmin] == w and tr["om_t"][kmin] + d[kmin] == b
        w, b, _ = o.sweep(M, o.SUM)
        ws = tr["w_sum"]
        kmin = int(np.argmin(ws))
        assert ws[kmin] == w and tr["om_t"][kmin] == b


# ------------------------------------------------------------------ the predictor (phase 1)
def test_predictor_rows_are_arithmetic_from_the_last_timestamp():
    rng = np.random.default_rng(21)
    last = rng.integers(0, 10 ** 12, size=9)
    iv = rng.integers(0, 10 ** 6, size=9)
    out = o.predict(last, iv, 7)
    assert out.shape == (9, 7)
    assert (out[:, 0] == last + iv).all()
    assert (np.diff(out, axis=1) == iv[:, None]).all()
    with pytest.raises(ValueError):
        o.predict([5], [-1], 3)
    with pytest.raises(ValueError):
        o.predict([2 ** 61], [2 ** 61], 3)


def test_predictor_then_search_matches_the_common_period_closed_form():
    # all workers predicted with one interval m: the best window misses only the largest circular gap of the phases
    rng = np.random.default_rng(22)
    for _ in range(100):
        n, m, R = int(rng.integers(1, 9)), int(rng.integers(5, 400)), int(rng.integers(2, 9))
        phase = rng.integers(0, m, size=n)
        last = 10 ** 9 + phase                      # latest observed end of each worker
        M = o.predict(last, np.full(n, m), R)
        u = np.unique(phase)
        gaps = np.diff(np.concatenate([u, [u[0] + m]]))
        expect = 0 if len(u) == 1 else m - int(gaps.max())
        w, b, idx = o.sweep(M, o.RANGE)
        assert w == expect
        assert (M[np.arange(n), idx] <= b).all() and M[np.arange(n), idx].max() == b


# ------------------------------------------------------------------ Algorithm 1 (GridScan) and FullGridScan
def gridscan_python(M, full):
    """Algorithm 1 written out from the listing: nearest point of every other row to each designated point."""
    n, R = len(M), len(M[0])
    pb = min(range(n), key=lambda p: (M[p][0], p))
    best = None
    for q in (range(n) if full else [pb]):
        for j in range(R):
            e = M[q][j]
            z = []
            for p in range(n):
                if p == q:
                    z.append(j)
                else:
                    z.append(min(range(R), key=lambda i: (abs(M[p][i] - e), i)))
            vals = [M[p][z[p]] for p in range(n)]
            d = max(vals) - min(vals)
            if best is None or d < best[0]:
                best = (d, max(vals), z)
    return best


@pytest.mark.parametrize("full", [False, True])
@pytest.mark.parametrize("regime", ["dense", "sparse", "strict"])
def test_gridscan_matches_the_listing_and_never_beats_the_optimum(full, regime):
    rng = np.random.default_rng(400 + full + len(regime))
    misses = 0
    for _ in range(300):
        M = random_instance(rng, regime)
        w, b, idx = o.gridscan(M, full)
        assert (w, b, list(idx)) == gridscan_python(M.tolist(), full)
        chosen = M[np.arange(M.shape[0]), idx]
        assert chosen.max() - chosen.min() == w and chosen.max() == b
        opt = o.sweep(M, o.RANGE)[0]
        assert w >= opt
        misses += w > opt
    if full and regime != "dense":
        assert misses < 300                     # FullGridScan finds the optimum at least sometimes


def test_fullgridscan_is_never_worse_than_gridscan():
    rng = np.random.default_rng(77)
    for _ in range(200):
        M = random_instance(rng, "strict")
        assert o.gridscan(M, True)[0] <= o.gridscan(M, False)[0]
    # a hand case: rows [0,10,20], [4,14,24], [9,19,29]; designated row 0; e=0 -> {0,4,9} d=9; e=10 -> {10,14,9} d=5
    assert o.gridscan([[0, 10, 20], [4, 14, 24], [9, 19, 29]])[:2] == (5, 14)
