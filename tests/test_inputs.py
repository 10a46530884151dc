"""The seeded input generator: determinism and the structure the recipe promises."""
import numpy as np

import zl_inputs as zi


def test_deterministic_and_order_independent():
    w = zi.CONFIGS["c3"].with_(B=6)
    a = zi.generate(w)
    b = zi.generate(w)
    assert (a == b).all()
    # instance k alone equals instance k of the batch (counter-based draws)
    c = zi.generate(w, B=2, first_instance=3)
    assert (c == a[3:5]).all()


def test_shapes_and_monotone_rows():
    for name in ("c1", "c2", "c3", "t2_n10_R15", "t2_n100_R150"):
        w = zi.CONFIGS[name]
        a = zi.generate(w, B=min(w.B, 8))
        assert a.shape == (min(w.B, 8), w.n, w.R) and a.dtype == np.int64
        assert (np.diff(a, axis=2) >= 1).all() if w.R > 1 else True
        assert (a > 0).all()


def test_c1_is_seed_zero_and_small_enough_for_enumeration():
    a = zi.generate(zi.CONFIGS["c1"])
    assert a.shape == (1, 4, 8)
    means = np.diff(a[0], axis=1).mean(axis=1)
    assert ((means > 50_000) & (means < 800_000)).all()      # lognormal around 200 ms


def test_c3_has_ten_percent_stragglers():
    w = zi.CONFIGS["c3"].with_(B=4)
    a = zi.generate(w)
    means = np.diff(a, axis=2).mean(axis=2)                   # [B, n]
    for b in range(4):
        slow = (means[b] > 2.0 * np.median(means[b])).sum()
        assert 10 <= slow <= 16                               # ceil(128/10) = 13 workers x3


def test_c5_offsets_and_bimodal_means():
    w = zi.CONFIGS["c5"].with_(n=64, R=128, B=2)
    a = zi.generate(w)
    means = np.diff(a, axis=2).mean(axis=2)
    assert (np.abs(means[:, :32] - 80_000) < 4_000).all()
    assert (np.abs(means[:, 32:] - 240_000) < 12_000).all()
    first = a[:, :, 0] - np.diff(a, axis=2)[:, :, 0]          # roughly the start offset
    assert first.min() > -60_000 and first.max() < 1_060_000


def test_epoch_shift_is_exact():
    w = zi.CONFIGS["c2"].with_(B=3)
    a = zi.generate(w)
    b = zi.generate(w.with_(epoch_us=1_700_000_000_000_000))
    assert (b - a == 1_700_000_000_000_000).all()
