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


# ---- strips container -----------------------------------------------------------------------
STRIP_CASES = [(0, 512, 1), (1, 512, 1), (6, 512, 1), (130, 512, 1), (511, 512, 1), (512, 512, 1), (513, 512, 1),
               (5000, 1024, 2), (4096, 1024, 1), (777, 4096, 4), (65536 + 17, 16384, 2), (3000, 2048, 2),
               (1000, 32, 1), (1000, 192, 2), (40001, 16384, 4), (33, 96, 3)]


@pytest.mark.parametrize("n,C,G", STRIP_CASES)
def test_strips_round_trip(n, C, G):
    rng = np.random.default_rng(n + C + G)
    msg = _source(rng, max(n, 1))
    T = _table(msg, 15, 12)
    msg = msg[:n]
    P = oracle.pack(T, msg, C, G, oracle.STRIPS)
    assert P.sub_offsets.size == P.n_sub + 1 and P.sub_offsets[-1] == P.stream.size
    assert all(int(o) % 16 == 0 for o in P.sub_offsets) and P.lane_meta.size == 0
    out, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and (out == msg).all()


def test_strips_chunk_must_be_a_multiple_of_the_lanes():
    T = oracle.Table([3, 1], 2)
    for C, G in ((1000, 1), (48, 1), (96, 2), (32 * 4097, 1)):
        with pytest.raises(oracle.OracleError):
            oracle.pack(T, np.zeros(10, dtype=np.uint8), C, G, oracle.STRIPS)


@pytest.mark.parametrize("n,C,G", [(3000, 2048, 2), (1000, 1024, 1), (517, 512, 4), (130, 4096, 1), (40000, 16384, 2)])
def test_strips_equal_plain_single_lane_coding(n, C, G):
    """Independent build of every sub-stream in Python.  Sub-stream g owns the strip
    [g*32*S, (g+1)*32*S) of its chunk; the strip is dealt to 32 lanes round-robin;
    a lane's string is the plain one-lane coder's initial state in R bits followed by that
    coder's fields, most significant bit first; the sub-stream is the 32 lengths as
    little-endian uint16, then the strings back to back in 32-bit little-endian words filled
    from the top bit, zero-padded to 16 bytes."""
    rng = np.random.default_rng(n)
    W, R = 32 * G, 10
    S = C // W
    msg = _source(rng, n)
    T = _table(msg, 15, R)
    P = oracle.pack(T, msg, C, G, oracle.STRIPS)
    for c in range(P.n_chunks):
        chunk = msg[c * C:(c + 1) * C]
        for g in range(G):
            sub = c * G + g
            strip = chunk[g * 32 * S:(g + 1) * 32 * S]
            lens, bits = [], ""
            for k in range(32):
                mine = strip[k::32]
                s = ""
                if mine.size:
                    init, nb, val = oracle.encode_lane_fields(T, mine)
                    s = format(init, "b").zfill(R)
                    s += "".join(format(int(v), "b").zfill(int(b)) if b else "" for b, v in zip(nb, val))
                lens.append(len(s))
                bits += s
            words = (len(bits) + 31) // 32
            bits = bits.ljust(32 * words, "0")
            want = b"".join(int(x).to_bytes(2, "little") for x in lens)
            want += b"".join(int(bits[32 * i:32 * i + 32], 2).to_bytes(4, "little") for i in range(words))
            want += bytes(-len(want) % 16)
            b0, b1 = int(P.sub_offsets[sub]), int(P.sub_offsets[sub + 1])
            assert bytes(P.stream[b0:b1]) == want


def _body_bits(stream, nbits):
    words = np.frombuffer(bytes(stream[64:64 + 4 * ((nbits + 31) // 32)]), dtype="<u4")
    return "".join(format(int(w), "032b") for w in words)[:nbits]


@pytest.mark.parametrize("name", ["trace_T1.txt", "trace_T2.txt"])
def test_strips_bytes_of_the_hand_trace(name):
    """Lane 0 of a one-strip layer carrying the hand trace's message (positions 0, 32, 64, ...;
    the other positions hold the first symbol): its length and bits are the ones worked out by
    hand in the fixture; for T1 so are the other lanes' and the first word."""
    g = read_golden(name)
    R = int(g["table_log"])
    T = oracle.Table(_ints(g["freqs"]), R)
    msg = _ints(g["message"])
    pos = [32 * t for t in range(len(msg))]
    sym = np.full(pos[-1] + 1, msg[0], dtype=np.uint8)
    sym[pos] = msg
    P = oracle.pack(T, sym, 512, 1, oracle.STRIPS)
    lens = np.frombuffer(bytes(P.stream[:64]), dtype="<u2").astype(int)
    want = g["strips_lane_bits"]
    assert lens[0] == len(want) and _body_bits(P.stream, len(want)) == want
    if "strips_other_lane_bits" in g:
        other = g["strips_other_lane_bits"]
        assert (lens[1:] == len(other)).all()
        assert _body_bits(P.stream, int(lens.sum())) == want + other * 31
        assert bytes(P.stream[64:68]) == bytes.fromhex(g["strips_first_word_hex"].replace(" ", ""))
        assert P.stream.size == int(g["strips_sub_stream_bytes"])
    out, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and out[pos].tolist() == msg and (out == sym).all()


def test_strips_same_symbols_for_every_chunking_and_threads():
    rng = np.random.default_rng(21)
    msg = _source(rng, 50000)
    T = _table(msg, 15, 11)
    for C, G in [(1024, 1), (4096, 1), (4096, 4), (16384, 2), (65536, 8), (32, 1), (131072, 1), (480, 3)]:
        P = oracle.pack(T, msg, C, G, oracle.STRIPS)
        for th in (1, 4):
            out, rc = oracle.unpack(T, P, threads=th)
            assert rc == oracle.OK and (out == msg).all()


def test_strips_with_one_group_own_the_symbols_of_the_private_lanes():
    """With 32 lanes per chunk the strip is the whole chunk, so lane k owns the very symbols it
    owns in the private container: same initial states, same number of bits."""
    rng = np.random.default_rng(23)
    msg = _source(rng, 9000)
    T = _table(msg, 15, 9)
    Pp = oracle.pack(T, msg, 4096, 1, oracle.PRIVATE)
    Ps = oracle.pack(T, msg, 4096, 1, oracle.STRIPS)
    for sub in range(Pp.n_sub):
        b0 = int(Ps.sub_offsets[sub])
        lens = np.frombuffer(bytes(Ps.stream[b0:b0 + 64]), dtype="<u2").astype(int)
        body = _body_bits(Ps.stream[b0:], int(lens.sum()))
        chunk = msg[sub * 4096:(sub + 1) * 4096]
        start = 0
        for k in range(32):
            mine = body[start:start + lens[k]]
            start += lens[k]
            if not lens[k]:
                assert chunk[k::32].size == 0
                continue
            assert int(mine[:9], 2) == (int(Pp.lane_meta[sub, k]) & 0xFFFF)
            assert lens[k] - 9 == oracle.encode_plain(T, chunk[k::32])[2]


def test_strips_corruption_is_reported():
    rng = np.random.default_rng(16)
    msg = _source(rng, 8192)
    T = _table(msg, 15, 12)
    P = oracle.pack(T, msg, 4096, 1, oracle.STRIPS)
    flagged = 0
    positions = list(range(3, P.stream.size, 97))
    for pos in positions:
        Q = oracle.Packed(P.layout, P.stream.copy(), P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        Q.stream[pos] ^= 0x5A
        flagged += (oracle.unpack(T, Q)[1] == oracle.ERR_CORRUPT)
    assert flagged > len(positions) // 2
    for k in (0, 7, 31):                                   # a wrong length is always caught
        Q = oracle.Packed(P.layout, P.stream.copy(), P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        Q.stream[2 * k] ^= 1
        assert oracle.unpack(T, Q)[1] == oracle.ERR_CORRUPT
    Q = oracle.Packed(P.layout, P.stream, P.sub_offsets.copy(), P.lane_meta, P.n, P.chunk, P.groups)
    Q.sub_offsets[1] -= 16                                 # truncated sub-stream
    Q.sub_offsets[2:] -= 16
    Q.stream = np.delete(P.stream, np.s_[int(P.sub_offsets[1]) - 16:int(P.sub_offsets[1])])
    assert oracle.unpack(T, Q)[1] == oracle.ERR_CORRUPT


def test_strips_overhead_per_lane_is_the_state_and_a_length():
    """Coded size = the plain coder's bits of every lane + (R + 16) bits per lane + word and
    16-byte padding per sub-stream; slimmer than the quads container at the same lanes."""
    rng = np.random.default_rng(19)
    n, C, G, R = 1 << 17, 16384, 2, 8
    msg = _source(rng, n, A=7, zp=3, th=0.1)
    T = _table(msg, 7, R)
    P = oracle.pack(T, msg, C, G, oracle.STRIPS)
    S = C // (32 * G)
    bits = 0
    for sub in range(P.n_sub):
        strip = msg[sub * 32 * S:(sub + 1) * 32 * S]
        for k in range(32):
            bits += oracle.encode_plain(T, strip[k::32])[2] + R + 16
    pad = 0
    for sub in range(P.n_sub):
        b0, b1 = int(P.sub_offsets[sub]), int(P.sub_offsets[sub + 1])
        body = int(np.frombuffer(bytes(P.stream[b0:b0 + 64]), dtype="<u2").astype(int).sum())
        assert 0 <= (b1 - b0 - 64) * 8 - body < 128 + 32
        pad += (b1 - b0 - 64) * 8 - body
    assert P.stream.size * 8 == bits + pad
    assert P.total_bytes() < oracle.pack(T, msg, C, G, oracle.QUADS).total_bytes()


# ---- channels container (the paper's grouping by input channel, Section III-B) ------------------
@pytest.mark.parametrize("O,I,H,W", [(8, 64, 3, 3), (5, 32, 1, 1), (16, 96, 7, 7), (3, 128, 3, 3), (64, 64, 1, 1)])
def test_channels_lane_is_an_input_channel(O, I, H, W):
    """A conv tensor stored O x I x H x W as one chunk with I lanes and pieces of H*W symbols:
    lane c's string is the plain one-lane coder's state and fields for tensor[:, c, :, :] read in
    memory order; the sub-stream bytes are built here independently (lengths, strings from the
    top bit of 32-bit little-endian words, zero padding to 16 bytes)."""
    rng = np.random.default_rng(O * I + H)
    R = 9
    w = _source(rng, O * I * H * W).reshape(O, I, H, W)
    T = _table(w.ravel(), 15, R)
    P = oracle.pack(T, w.ravel(), w.size, I // 32, oracle.CHANNELS, piece=H * W)
    assert P.n_sub == I // 32 and P.lane_meta.size == 0
    for g in range(I // 32):
        lens, bits = [], ""
        for k in range(32):
            mine = np.ascontiguousarray(w[:, 32 * g + k]).ravel()
            init, nb, val = oracle.encode_lane_fields(T, mine)
            s = format(init, "b").zfill(R) + "".join(format(int(v), "b").zfill(int(b)) if b else "" for b, v in zip(nb, val))
            lens.append(len(s))
            bits += s
        words = (len(bits) + 31) // 32
        bits = bits.ljust(32 * words, "0")
        want = b"".join(int(x).to_bytes(2, "little") for x in lens)
        want += b"".join(int(bits[32 * i:32 * i + 32], 2).to_bytes(4, "little") for i in range(words))
        want += bytes(-len(want) % 16)
        assert bytes(P.stream[int(P.sub_offsets[g]):int(P.sub_offsets[g + 1])]) == want
    out, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and (out == w.ravel()).all()


def test_channels_with_pieces_of_one_symbol_and_32_lanes_is_the_strips_container():
    rng = np.random.default_rng(31)
    msg = _source(rng, 32 * 300)
    T = _table(msg, 15, 10)
    a = oracle.pack(T, msg, 3200, 1, oracle.CHANNELS, piece=1)
    b = oracle.pack(T, msg, 3200, 1, oracle.STRIPS)
    assert bytes(a.stream) == bytes(b.stream) and (a.sub_offsets == b.sub_offsets).all()


def test_channels_chunks_threads_sizes_and_corruption():
    rng = np.random.default_rng(33)
    O, I, E = 24, 64, 9
    w = _source(rng, O * I * E)
    T = _table(w, 15, 11)
    for C in (w.size, 8 * I * E, I * E):                   # one chunk per layer, or chunks of whole rows
        P = oracle.pack(T, w, C, I // 32, oracle.CHANNELS, piece=E)
        for th in (1, 3):
            out, rc = oracle.unpack(T, P, threads=th)
            assert rc == oracle.OK and (out == w).all()
    for C, n, E2 in ((w.size + 1, w.size, 9), (w.size, w.size - 64, 9), (w.size, w.size, 7)):
        with pytest.raises(oracle.OracleError):            # sizes that are no multiple of lanes * piece
            oracle.pack(T, w[:n], C, I // 32, oracle.CHANNELS, piece=E2)
    P = oracle.pack(T, w, w.size, I // 32, oracle.CHANNELS, piece=E)
    flagged = 0
    positions = list(range(3, P.stream.size, 131))
    for pos in positions:
        Q = oracle.Packed(P.layout, P.stream.copy(), P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups, P.piece)
        Q.stream[pos] ^= 0x5A
        flagged += (oracle.unpack(T, Q)[1] == oracle.ERR_CORRUPT)
    assert flagged > len(positions) // 2
