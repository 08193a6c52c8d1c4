"""Pins for the oracle's spread and decode table (paper Section II-A, Fig. 2)."""
import itertools

import numpy as np
import pytest

import oracle
from conftest import read_golden


def _ints(s):
    return [int(x) for x in s.split()]


@pytest.mark.parametrize("name", ["trace_T1.txt", "trace_T2.txt"])
def test_table_matches_hand_trace(name):
    g = read_golden(name)
    R = int(g["table_log"])
    T = oracle.Table(_ints(g["freqs"]), R)
    ent = T.entries()
    assert [e[0] for e in ent] == _ints(g["slot"])
    for i in range(1 << R):
        assert list(ent[i]) == _ints(g[f"entry {i}"])


def _random_freqs(rng, A, R):
    L = 1 << R
    cuts = np.sort(rng.choice(np.arange(1, L), size=A - 1, replace=False)) if A > 1 else np.array([], int)
    return np.diff(np.concatenate([[0], cuts, [L]])).astype(np.uint32)


@pytest.mark.parametrize("R", [1, 2, 3, 5, 6, 7, 8, 11, 12, 14])
def test_table_invariants(R):
    """Each symbol owns f_s states; nb takes one of two values; for every symbol the
    ranges [newX, newX + 2^nb) of its states tile [0, l) exactly, which is what makes
    every (state, symbol) pair encodable in exactly one way."""
    rng = np.random.default_rng(R)
    L = 1 << R
    for trial in range(4):
        A = int(min(L, rng.integers(1, 40)))
        f = _random_freqs(rng, A, R)
        if trial == 3:                       # skewed: one symbol owns almost everything
            f = np.ones(A, dtype=np.uint32); f[A // 2] = L - (A - 1)
        ent = oracle.Table(f, R).entries()
        for s in range(A):
            mine = [(nb, nx) for (sy, nb, nx) in ent if sy == s]
            assert len(mine) == f[s]
            if f[s] == 0:
                continue
            hi = R - int(np.floor(np.log2(int(f[s]))))
            assert {nb for nb, _ in mine} <= {hi, hi - 1}
            cover = np.zeros(L, dtype=np.int32)
            for nb, nx in mine:
                assert nx % (1 << nb) == 0 and nx + (1 << nb) <= L
                cover[nx:nx + (1 << nb)] += 1
            assert (cover == 1).all()


@pytest.mark.parametrize("R", [2, 3, 4])
def test_table_is_duda_decoding_function(R):
    """Brute force against the defining relation of ANS: state x in [l, 2l) decodes to
    (s, x_s) with s the symbol spread at x and x_s = f_s + (number of smaller states
    carrying s); the table's (nb, newX) must be the unique renormalisation of x_s back
    into [l, 2l)."""
    L = 1 << R
    for f in itertools.product(range(0, L + 1), repeat=3):
        if sum(f) != L:
            continue
        ent = oracle.Table(f, R).entries()
        slot = [e[0] for e in ent]
        for i, (s, nb, nx) in enumerate(ent):
            xs = f[s] + sum(1 for y in range(i) if slot[y] == s)
            assert f[s] <= xs < 2 * f[s]
            k = 0
            while (xs << k) < L:
                k += 1
            assert nb == k and nx == (xs << k) - L
        # bit-reversal spread: slot handed out j-th sits at the R-bit reversal of j
        order = sorted(range(L), key=lambda i: int(format(i, f"0{R}b")[::-1], 2))
        expect = [s for s in range(3) for _ in range(f[s])]
        assert [slot[i] for i in order] == expect


def test_lut_fits_three_bytes_per_state_up_to_256_states():
    """Section II-A: symbol, nb_bits and newX each fit one byte, 3*l bytes in all."""
    g = read_golden("paper_lut_size.txt")
    l = int(g["states"])
    R = l.bit_length() - 1
    rng = np.random.default_rng(0)
    A = (1 << int(g["symbol_bits"])) - 1
    f = _random_freqs(rng, A, R)
    ent = oracle.Table(f, R).entries()
    assert all(0 <= s < 256 and 0 <= nb < 256 and 0 <= nx < 256 for s, nb, nx in ent)
    assert max(nx + (1 << nb) for _, nb, nx in ent) <= 1 << int(g["adder_bits"])
    assert 3 * len(ent) == int(g["lut_bytes"])
    for R8 in (7, 8):
        ent = oracle.Table(_random_freqs(rng, 31, R8), R8).entries()
        assert all(nx < 256 and nb < 256 for _, nb, nx in ent)


def test_bad_frequencies_rejected():
    with pytest.raises(oracle.OracleError):
        oracle.Table([3, 2], 2)
    with pytest.raises(oracle.OracleError):
        oracle.Table([1, 1], 2)


def test_single_symbol_layer_reads_no_bits():
    ent = oracle.Table([0, 16, 0], 4).entries()
    assert all(s == 1 and nb == 0 for s, nb, _ in ent)
    assert sorted(nx for _, _, nx in ent) == list(range(16))
