"""Pins for the multi-lane containers (paper Section III-B: one table, a vector of
states, one state per stream)."""
import numpy as np
import pytest

import oracle
from conftest import read_golden


def _ints(s):
    return [int(x) for x in s.split()]


def _source(rng, n, A=15, zp=7, th=0.3):
    p = th ** np.abs(np.arange(A) - zp); p /= p.sum()
    return rng.choice(A, size=n, p=p).astype(np.uint8)


def _table(msg, A, R):
    return oracle.Table(oracle.normalize_freqs(oracle.histogram(msg), A, R), R)


@pytest.mark.parametrize("layout", [oracle.INTERLEAVED, oracle.PRIVATE, oracle.QUADS])
@pytest.mark.parametrize("n,C,G", [(2, 64, 1), (3, 64, 1), (127, 1000, 1), (129, 1000, 1), (1001, 333, 2),
                                   (0, 64, 1), (1, 64, 1), (31, 64, 1), (32, 64, 1), (33, 64, 1),
                                   (4096, 1024, 1), (5000, 1024, 2), (777, 4096, 4), (65536 + 17, 16384, 1)])
def test_container_round_trip(layout, n, C, G):
    rng = np.random.default_rng(n + C + G)
    msg = _source(rng, max(n, 1))
    T = _table(msg, 15, 12)
    msg = msg[:n]
    P = oracle.pack(T, msg, C, G, layout)
    assert P.sub_offsets.size == P.n_sub + 1 and P.sub_offsets[-1] == P.stream.size
    assert all(int(o) % 16 == 0 for o in P.sub_offsets)
    out, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and (out == msg).all()


@pytest.mark.parametrize("layout", [oracle.INTERLEAVED, oracle.PRIVATE])
def test_lanes_equal_plain_single_lane_coding(layout):
    """Lane lambda of a chunk carries the chunk's symbols lambda, lambda + W, ... and its
    initial state is what the plain one-lane coder gives for that sub-sequence; for the
    private container its words are that coder's bytes."""
    rng = np.random.default_rng(11)
    n, C, G = 3000, 2048, 2
    W = 32 * G
    msg = _source(rng, n)
    T = _table(msg, 15, 10)
    P = oracle.pack(T, msg, C, G, layout)
    for c in range(P.n_chunks):
        chunk = msg[c * C:(c + 1) * C]
        for lam in range(W):
            sub, k = c * G + lam // 32, lam % 32
            init, data, nbits = oracle.encode_plain(T, chunk[lam::W])
            meta = int(P.lane_meta[sub, k])
            assert (meta & 0xFFFF) == init
            if layout == oracle.PRIVATE:
                b0 = int(P.sub_offsets[sub]) + 4 * (meta >> 16)
                words = (nbits + 31) // 32
                got = bytes(P.stream[b0:b0 + 4 * words])
                assert got == bytes(data) + bytes(4 * words - len(data))


def test_same_symbols_for_every_chunking():
    rng = np.random.default_rng(2)
    msg = _source(rng, 20000)
    T = _table(msg, 15, 11)
    for layout in (oracle.INTERLEAVED, oracle.PRIVATE, oracle.QUADS):
        for C, G in [(1024, 1), (4096, 1), (4096, 4), (16384, 2), (65536, 8), (1001, 1), (4099, 2)]:
            out, rc = oracle.unpack(T, oracle.pack(T, msg, C, G, layout))
            assert rc == oracle.OK and (out == msg).all()


@pytest.mark.parametrize("name", ["trace_T1.txt", "trace_T2.txt"])
def test_interleaved_units_of_a_single_active_lane(name):
    """Lane 0 of a chunk carrying the hand trace's message must start from the trace's
    initial state and its first 16-bit unit must be the trace's bits."""
    g = read_golden(name)
    T = oracle.Table(_ints(g["freqs"]), int(g["table_log"]))
    msg = _ints(g["message"])
    # message symbol t sits at chunk position 32 t, i.e. in lane 0; the other lanes hold
    # copies of the first symbol.  Lane 0 refills first in round 0 and the whole trace
    # needs fewer than 16 bits, so the sub-stream's first unit is lane 0's bit string.
    n = 32 * (len(msg) - 1) + 1
    sym = np.full(n, msg[0], dtype=np.uint8)
    sym[::32] = msg
    P = oracle.pack(T, sym, n, 1, oracle.INTERLEAVED)
    assert int(P.lane_meta[0, 0]) == int(g["init_state"])
    want = bytes.fromhex(g["interleaved_units_hex"].replace(" ", ""))
    assert bytes(P.stream[:2]) == want
    out, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and out[::32].tolist() == msg


def test_interleaved_unit_order_is_the_refill_schedule():
    """Independent replay in Python: walk the rounds, let every lane that holds < 16
    bits take the next unit, and check that each lane ends up with its own bit string."""
    rng = np.random.default_rng(4)
    n, C = 1500, 1500
    msg = _source(rng, n, th=0.5)
    T = _table(msg, 15, 9)
    P = oracle.pack(T, msg, C, 1, oracle.INTERLEAVED)
    units = np.frombuffer(bytes(P.stream), dtype="<u2")
    per_lane_units = [[] for _ in range(32)]
    per_lane_nb = []
    for k in range(32):
        _, nb, _ = oracle.encode_lane_fields(T, msg[k::32])
        per_lane_nb.append(nb.tolist())
    have = [0] * 32
    u = 0
    for r in range((n + 31) // 32):
        for k in range(32):
            if r < len(per_lane_nb[k]) and have[k] < 16:
                per_lane_units[k].append(int(units[u])); u += 1; have[k] += 16
        for k in range(32):
            if r < len(per_lane_nb[k]):
                have[k] -= per_lane_nb[k][r]
                assert have[k] >= 0
    assert (u * 2 + 15) // 16 * 16 == P.stream.size
    for k in range(32):
        _, data, nbits = oracle.encode_plain(T, msg[k::32])
        mine = b"".join(int(x).to_bytes(2, "little") for x in per_lane_units[k])
        assert mine[:len(data)] == bytes(data) and not any(mine[len(data):])


def test_container_overhead_is_small_for_long_chunks():
    """Section III-B: splitting into parallel streams costs little (< 1 % for the paper's
    per-input-channel streams).  Report-style check: at 16 K symbols per chunk the
    containers stay within a few percent of the single-lane coded size."""
    rng = np.random.default_rng(9)
    msg = _source(rng, 1 << 18, th=0.25)
    T = _table(msg, 15, 12)
    single = oracle.encode_plain(T, msg)[2] / 8
    a = oracle.pack(T, msg, 16384, 1, oracle.INTERLEAVED).total_bytes()
    b = oracle.pack(T, msg, 16384, 1, oracle.PRIVATE).total_bytes()
    assert single < a < 1.05 * single
    assert single < b < 1.08 * single
    assert single < oracle.pack(T, msg, 16384, 1, oracle.QUADS).total_bytes() < 1.08 * single


@pytest.mark.parametrize("layout", [oracle.INTERLEAVED, oracle.PRIVATE, oracle.QUADS])
def test_corruption_is_reported(layout):
    rng = np.random.default_rng(6)
    msg = _source(rng, 8192)
    T = _table(msg, 15, 12)
    P = oracle.pack(T, msg, 4096, 1, layout)
    flagged = 0
    for pos in range(3, P.stream.size, 97):
        Q = oracle.Packed(P.layout, P.stream.copy(), P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        Q.stream[pos] ^= 0x5A
        out, rc = oracle.unpack(T, Q)
        flagged += (rc == oracle.ERR_CORRUPT)
    assert flagged > 0
    Q = oracle.Packed(P.layout, P.stream, P.sub_offsets, P.lane_meta.copy(), P.n, P.chunk, P.groups)
    Q.lane_meta[0, 5] ^= 1
    assert oracle.unpack(T, Q)[1] == oracle.ERR_CORRUPT


def test_threaded_unpack_equals_serial():
    rng = np.random.default_rng(8)
    msg = _source(rng, 100_000)
    T = _table(msg, 15, 12)
    for layout in (oracle.INTERLEAVED, oracle.PRIVATE, oracle.QUADS):
        P = oracle.pack(T, msg, 4096, 1, layout)
        a, rca = oracle.unpack(T, P, threads=1)
        b, rcb = oracle.unpack(T, P, threads=4)
        assert rca == rcb == oracle.OK and (a == b).all() and (a == msg).all()


def _quads_lanes(nc, W):
    """Which chunk positions each lane owns, by dealing the chunk out four symbols at a time."""
    lanes = [[] for _ in range(W)]
    for q in range(nc):
        lanes[(q // 4) % W].append(q)
    return lanes


@pytest.mark.parametrize("n,C,G", [(3000, 2048, 2), (1000, 1000, 1), (517, 300, 4), (130, 130, 1)])
def test_quads_lanes_equal_plain_single_lane_coding(n, C, G):
    """A quads lane carries the symbols dealt to it four at a time; its initial state is the
    plain one-lane coder's for that sub-sequence and its words are that coder's fields, each
    written most significant bit first from the top of a 32-bit little-endian word."""
    rng = np.random.default_rng(n)
    W = 32 * G
    msg = _source(rng, n)
    T = _table(msg, 15, 10)
    P = oracle.pack(T, msg, C, G, oracle.QUADS)
    for c in range(P.n_chunks):
        chunk = msg[c * C:(c + 1) * C]
        owned = _quads_lanes(chunk.size, W)
        assert sorted(q for l in owned for q in l) == list(range(chunk.size))
        for lam in range(W):
            sub, k = c * G + lam // 32, lam % 32
            init, nb, val = oracle.encode_lane_fields(T, chunk[owned[lam]])
            meta = int(P.lane_meta[sub, k])
            assert (meta & 0xFFFF) == init
            bits = "".join(format(int(v), "b").zfill(int(b)) if b else "" for b, v in zip(nb, val))
            words = (len(bits) + 31) // 32
            bits = bits.ljust(32 * words, "0")
            want = b"".join(int(bits[32 * i:32 * i + 32], 2).to_bytes(4, "little") for i in range(words))
            b0 = int(P.sub_offsets[sub]) + 4 * (meta >> 16)
            assert bytes(P.stream[b0:b0 + 4 * words]) == want
            nxt = int(P.lane_meta[sub, k + 1]) >> 16 if k < 31 else None
            if nxt is not None:
                assert nxt - (meta >> 16) == words


@pytest.mark.parametrize("name", ["trace_T1.txt", "trace_T2.txt"])
def test_quads_word_of_the_hand_trace(name):
    """Lane 0 of a one-chunk quads layer carrying the hand trace's message: the trace's
    initial state, and the word worked out by hand in the fixture."""
    g = read_golden(name)
    T = oracle.Table(_ints(g["freqs"]), int(g["table_log"]))
    msg = _ints(g["message"])
    # lane 0 owns chunk positions 0..3, 128..131, ...; the other lanes hold the first symbol
    pos = [(t // 4) * 128 + t % 4 for t in range(len(msg))]
    sym = np.full(pos[-1] + 1, msg[0], dtype=np.uint8)
    sym[pos] = msg
    P = oracle.pack(T, sym, sym.size, 1, oracle.QUADS)
    assert (int(P.lane_meta[0, 0]) & 0xFFFF) == int(g["init_state"]) and int(P.lane_meta[0, 0]) >> 16 == 0
    assert bytes(P.stream[:4]) == bytes.fromhex(g["quads_word_hex"].replace(" ", ""))
    out, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and out[pos].tolist() == msg and (out == sym).all()
