"""The oracle's histogram normaliser (the paper codes each layer with a 256-state coder,
Section III-A, and does not say how counts become slots: any valid normalisation decodes
identically, only the size changes)."""
import numpy as np
import pytest

import oracle


@pytest.mark.parametrize("R", [2, 6, 8, 12, 14])
def test_normalised_frequencies_are_valid(R):
    rng = np.random.default_rng(R)
    L = 1 << R
    for trial in range(50):
        A = int(rng.integers(1, min(256, L) + 1))
        counts = np.zeros(256, dtype=np.uint64)
        k = int(rng.integers(1, A + 1))
        idx = rng.choice(A, size=k, replace=False)
        counts[idx] = (rng.pareto(0.7, size=k) * 50 + 1).astype(np.uint64)
        f = oracle.normalize_freqs(counts, A, R)
        assert int(f.sum()) == L
        assert ((f > 0) == (counts[:A] > 0)).all()
        exact = counts[:A].astype(np.float64) * L / counts.sum()
        big = exact >= 1
        if (f[~big & (counts[:A] > 0)] == 1).all() and (~big).sum() == 0:
            assert (np.abs(f[big] - exact[big]) < 1.0 + 1e-9).all()


def test_known_small_cases():
    assert oracle.normalize_freqs([3, 1], 2, 2).tolist() == [3, 1]
    assert oracle.normalize_freqs([1, 1, 1], 3, 2).tolist() == [2, 1, 1]          # tie -> lower symbol
    assert oracle.normalize_freqs([1000, 1, 1, 1], 4, 2).tolist() == [1, 1, 1, 1]  # overshoot path
    assert oracle.normalize_freqs([0, 5, 0], 3, 4).tolist() == [0, 16, 0]
    with pytest.raises(oracle.OracleError):
        oracle.normalize_freqs([1, 1, 1, 1, 1], 5, 2)
    with pytest.raises(oracle.OracleError):
        oracle.normalize_freqs([0, 0], 2, 4)


def test_histogram_is_a_plain_count():
    rng = np.random.default_rng(3)
    for n in (0, 1, 255, 100_003):
        sym = rng.integers(0, 256, size=n, dtype=np.uint8)
        if n > 10:
            sym[::3] = 7                                   # a peak, as in weight symbols
        h = oracle.histogram(sym)
        assert h.shape == (256,) and int(h.sum()) == n
        assert (h == np.bincount(sym, minlength=256)).all()
