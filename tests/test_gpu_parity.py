"""GPU vs oracle, element by element, through the C ABI.  Streams are encoded by the ORACLE;
the library only decodes them.  Integer symbols, fp32 and bf16 outputs are compared as bit
patterns: the decode is integer work and the dequantiser is one IEEE multiply plus one
round-to-nearest-even, so the tolerance is zero."""
import numpy as np
import pytest
import torch

import oracle
import synthgen as sg
import paper_2406_06237_b200 as ans
from paper_2406_06237_b200.runtime import DeviceBatch
from helpers import (bits_view, expected_bits, oracle_expected, oracle_pack_spec, parallel_map, tiny_spec,
                     to_packed_layer)

pytestmark = pytest.mark.gpu
LAYOUTS = [ans.ANS_LAYOUT_INTERLEAVED, ans.ANS_LAYOUT_PRIVATE, ans.ANS_LAYOUT_QUADS]
OWN_WORDS = [ans.ANS_LAYOUT_PRIVATE, ans.ANS_LAYOUT_QUADS]


def run_and_compare(specs, layout, lanes=32, per_layer=False, threads=8, chunk=None, table_log=None):
    def prep(spec):
        sym = sg.draw_symbols(spec, threads=1)
        T, P, f256 = oracle_pack_spec(spec, sym, layout, lanes, chunk, table_log)
        want_sym, want = oracle_expected(spec, T, P)
        assert (want_sym == sym).all()
        return to_packed_layer(spec, P, f256, table_log), want_sym, want

    prepared = parallel_map(prep, specs, threads)
    db = DeviceBatch([p[0] for p in prepared])
    # canaries: outputs start poisoned so that an element the kernel skips cannot pass by luck
    for o in db.out_sets[0]:
        o.view(torch.uint8).fill_(0xA5)
    (db.decode_per_layer if per_layer else db.decode)()
    assert db.read_status() == 0
    for i, (pl, want_sym, want) in enumerate(prepared):
        got = bits_view(db.output(i))
        assert got.shape == want.shape
        bad = np.flatnonzero(got != expected_bits(want))
        assert bad.size == 0, f"layer {i} ({specs[i].name}): {bad.size} mismatches, first at {bad[:5]}"
    return db, prepared


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("lanes", [32, 64, 128, 256])
def test_config1_single_conv_fp32(layout, lanes):
    db, prepared = run_and_compare(sg.workload_conv3x3(), layout, lanes)
    assert (db.decode_symbols(0).cpu().numpy() == prepared[0][1]).all()
    assert db.read_status() == 0


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("n", [0, 1, 31, 32, 33, 63, 64, 65, 2047, 2048, 2049, 4096 + 17, 3 * 4096])
def test_edge_sizes(layout, n):
    for dt in ("u8", "bf16", "f32"):
        run_and_compare([tiny_spec(n, out_dtype=dt, chunk=4096)], layout, 64)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("R", [1, 2, 3, 6, 7, 8, 11, 12, 13, 14])
def test_table_sizes(layout, R):
    b = 1 if R == 1 else min(8, R)
    specs = [tiny_spec(50_000 + R, bitwidth=b, pzp=p, table_log=R, chunk=16384, out_dtype=dt, index=i)
             for i, (p, dt) in enumerate([(0.55, "bf16"), (0.9, "u8"), (0.97, "f32")])]
    run_and_compare(specs, layout, 32)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_single_symbol_layer_and_odd_chunks(layout):
    """A layer whose every weight is the zero-point has one symbol with f = l: every
    transition reads zero bits and the streams hold only padding."""
    A, zp = sg.alphabet_for_bits(4)
    spec = sg.LayerSpec("const", (10_000,), 4, A, zp, 1e-9, 0.5, 10, 1000, "bf16", sg.stream_key(5, 0))
    sym = sg.draw_symbols(spec)
    assert (sym == zp).all()
    run_and_compare([spec], layout, 32)
    # chunk sizes that are not multiples of the lane count or of 16
    run_and_compare([tiny_spec(7001, chunk=c, out_dtype=dt, index=c) for c, dt in
                     [(999, "u8"), (1001, "bf16"), (77, "f32"), (4099, "u8")]], layout, 64)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_batch_with_mixed_layers_one_launch(layout):
    specs = [tiny_spec(20_000, 2, 0.8, 9, 4096, "bf16", index=0), tiny_spec(0, 4, 0.6, 12, 4096, "f32", index=1),
             tiny_spec(4096, 8, 0.9, 14, 1024, "u8", index=2), tiny_spec(123_457, 6, 0.7, 11, 16384, "bf16", index=3),
             tiny_spec(1, 1, 0.6, 1, 64, "f32", index=4), tiny_spec(70_000, 3, 0.95, 12, 32768, "bf16", index=5)]
    run_and_compare(specs, layout, 32)
    run_and_compare(specs, layout, 128, per_layer=True)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_batch_of_more_layers_than_the_kernel_parameters_hold(layout):
    """Beyond 96 layers the CTAs search the descriptors for their layer instead of the launch
    parameters, and walk the plan's own numbering; empty layers and one-chunk layers mixed in."""
    dts = ("bf16", "u8", "f32")
    specs = [tiny_spec(0 if i % 17 == 5 else 900 + 611 * (i % 13) + (40_000 if i % 29 == 0 else 0),
                       1 + i % 6, 0.55 + 0.04 * (i % 10), 6 + i % 7, 1024 << (i % 3), dts[i % 3], index=i)
             for i in range(131)]
    run_and_compare(specs, layout, 32)
    run_and_compare(specs[:100], layout, 64)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("shift", [1, 2, 3, 5])
def test_symbols_into_a_buffer_of_any_alignment(layout, shift):
    """ans_decode_layer asks no alignment of the symbol buffer: the vector stores of the fast
    paths must give way to byte stores, and nothing outside the buffer may be touched."""
    for n, chunk, lanes in [(70_001, 4096, 32), (1_200_000, 2048, 64)]:
        spec = tiny_spec(n, 3, 0.7, 8, chunk, "u8", index=shift)
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, layout, lanes)
        db = DeviceBatch([to_packed_layer(spec, P, f256)])
        buf = torch.full((n + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        ans.ans_decode_layer(db.h_descs[0][0], buf.data_ptr() + shift, db.status.data_ptr(),
                             torch.cuda.current_stream().cuda_stream)
        assert db.read_status() == 0
        got = buf.cpu().numpy()
        assert (got[shift:shift + n] == sym).all()
        assert (got[:shift] == 0xA5).all() and (got[shift + n:] == 0xA5).all()


def _channels_last(sym, shape):
    """The OHWI flattening of symbols drawn for an OIHW tensor: a permutation of the input."""
    return np.ascontiguousarray(sym.reshape(shape).transpose(0, 2, 3, 1)).ravel()


@pytest.mark.parametrize("layout", LAYOUTS)
def test_streams_grouped_by_input_channel(layout):
    """The paper's own grouping (Section III-B): one chunk per layer, as many lanes as the conv has
    input channels, weights stored channels-last, so that lane c carries input channel c.  Lane
    counts that are no power of two and up to the largest allowed ride along."""
    shapes = [(64, 64, 1, 1), (64, 64, 3, 3), (256, 96, 1, 1), (128, 512, 1, 1), (96, 2048, 1, 1), (32, 160, 3, 3)]
    prepared = []
    for i, shape in enumerate(shapes):
        spec = tiny_spec(int(np.prod(shape)), 3 + i % 3, 0.8, 8, int(np.prod(shape)), ("bf16", "f32", "u8")[i % 3],
                         index=i)
        sym = _channels_last(sg.draw_symbols(spec), shape)
        if layout == ans.ANS_LAYOUT_PRIVATE:             # lane c holds exactly input channel c
            per_channel = sym.reshape(-1, shape[1])
            assert (per_channel[:, 5] == sym[5::shape[1]]).all()
        T, P, f256 = oracle_pack_spec(spec, sym, layout, shape[1])
        want_sym, want = oracle_expected(spec, T, P)
        assert (want_sym == sym).all()
        prepared.append((to_packed_layer(spec, P, f256), want))
    db = DeviceBatch([p[0] for p in prepared])
    db.decode()
    assert db.read_status() == 0
    for i, (pl, want) in enumerate(prepared):
        assert np.array_equal(bits_view(db.output(i)), expected_bits(want)), f"layer {i}"


@pytest.mark.parametrize("layout", LAYOUTS)
def test_config2_resnet18_bf16(layout):
    run_and_compare(sg.workload_resnet18(), layout, 32)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("lanes", [32, 128])
def test_config3_resnet50_bf16(layout, lanes):
    run_and_compare(sg.workload_resnet50(), layout, lanes)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("chunk", [1024, 4096, 16384, 65536])
@pytest.mark.parametrize("R", [11, 12, 14])
def test_config4_sweep_reduced(layout, chunk, R):
    """The granularity sweep at reduced size (the full 2^28 runs in test_gpu_full_size): 2^22
    symbols, and 2^24 for the 64 K-symbol chunks, so that every cell has the 256 sub-streams and
    more from which a launch takes the many-warp shape the full size runs in."""
    n = (1 << 24) + 12345 if chunk == 65536 else (1 << 22) + 12345
    run_and_compare(sg.workload_sweep(table_log=R, chunk=chunk, n=n), layout, 32)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_config5_reduced(layout):
    run_and_compare(sg.workload_large(n_mats=2, dim=2048), layout, 32)


@pytest.mark.parametrize("layout", OWN_WORDS)
@pytest.mark.parametrize("lanes", [32, 64, 128, 256])
@pytest.mark.parametrize("R", [1, 5, 8, 9, 12])
def test_private_layers_of_many_substreams(layout, lanes, R):
    """Private layers that average 64 or more work items and have at most 512 states, and quads
    layers of any kind, are walked one symbol per look-up, every lane storing straight to the
    output: whole blocks, the rows after them, a ragged end, chunks that start off a quad's
    alignment, every output type and every lane count."""
    b = 1 if R == 1 else min(5, R)
    g = lanes // 32
    specs = [tiny_spec(300_017 // g * g + 5, b, 0.6, R, 999, "u8", index=0),
             tiny_spec(400_001, b, 0.75, R, 1001 * g, "bf16", index=1),
             tiny_spec(270_000 * g, b, 0.9, R, 777 * g, "f32", index=2),
             tiny_spec(1_100_000, b, 0.5, R, 4096, "bf16", index=3)]
    db, prepared = run_and_compare(specs, layout, lanes)
    assert (db.decode_symbols(1).cpu().numpy() == prepared[1][1]).all()
    assert db.read_status() == 0
    run_and_compare(specs[:2], layout, lanes, per_layer=True)


@pytest.mark.parametrize("layout", OWN_WORDS)
def test_private_many_long_substreams_read_from_global_memory(layout):
    """Sub-streams too long for the shared-memory staging buffer are read word by word from
    global memory; with many of them the layer still takes the one-symbol-per-look-up walk."""
    run_and_compare([tiny_spec(260 * 65536 + 321, 5, 0.15, 8, 65536, "u8")], layout, 32)


@pytest.mark.parametrize("layout", OWN_WORDS)
def test_private_many_substreams_corruption_is_flagged(layout):
    spec = tiny_spec(600_000, 3, 0.7, 8, 2048, "bf16")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, layout, 32)
    rng = np.random.default_rng(1)
    flagged = 0
    for trial in range(4):
        s = P.stream.copy()
        pos = rng.integers(0, s.size, size=8)
        s[pos] ^= rng.integers(1, 256, size=8).astype(np.uint8)
        P2 = oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        db = DeviceBatch([to_packed_layer(spec, P2, f256)])
        db.decode()
        st = db.read_status()
        _, orc = oracle.unpack(T, P2)
        assert (st != 0) == (orc != oracle.OK)
        flagged += st != 0
    assert flagged > 0
    m = P.lane_meta.copy(); m[5, 7] += 1 << 16            # a lane's first word moved
    db = DeviceBatch([to_packed_layer(spec, oracle.Packed(P.layout, P.stream, P.sub_offsets, m, P.n, P.chunk,
                                                          P.groups), f256)])
    db.decode()
    assert db.read_status() != 0


@pytest.mark.parametrize("layout", LAYOUTS)
def test_corrupt_streams_are_flagged_not_fatal(layout):
    """Corruption is planted on the host.  Reads are clamped to the stream and every loop is
    counted, so a bad stream yields wrong symbols and a status bit, never a fault."""
    spec = tiny_spec(40_000, 4, 0.6, 12, 4096, "bf16")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, layout, 32)

    def decode(P2):
        db = DeviceBatch([to_packed_layer(spec, P2, f256)])
        guard = torch.full((1 << 16,), 0x5A, dtype=torch.uint8, device="cuda")
        db.decode()
        st = db.read_status()
        assert (guard == 0x5A).all()
        return st, bits_view(db.output(0))

    st, good = decode(P)
    assert st == 0
    flagged = 0
    rng = np.random.default_rng(0)
    for trial in range(6):
        s = P.stream.copy()
        pos = rng.integers(0, s.size, size=8)
        s[pos] ^= rng.integers(1, 256, size=8).astype(np.uint8)
        st, _ = decode(oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups))
        _, orc = oracle.unpack(T, oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups))
        assert (st != 0) == (orc != oracle.OK)
        flagged += st != 0
    assert flagged > 0
    m = P.lane_meta.copy(); m[1, 3] ^= 1
    st, _ = decode(oracle.Packed(P.layout, P.stream, P.sub_offsets, m, P.n, P.chunk, P.groups))
    assert st & 1
    o = P.sub_offsets.copy(); o[2] += 1 << 40            # offset far outside the stream
    st, _ = decode(oracle.Packed(P.layout, P.stream, o, P.lane_meta, P.n, P.chunk, P.groups))
    assert st & 2
    short = P.stream[:P.stream.size - 16].copy()         # truncated stream
    st, _ = decode(oracle.Packed(P.layout, short, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups))
    assert st & 2


DEQUANT_EDGES = [(0, 1.0), (7, 0.02), (127, 0.1 / 256), (3, 0.05), (15, 1.0 / 3.0), (31, 3.0e-39),
                 (1, 257.0 / 65536.0), (127, 1.0 + 2.0 ** -8), (0, 1.0 + 3 * 2.0 ** -8), (255, 1.0 + 2.0 ** -8),
                 (0, -0.75), (200, 1.0e30), (128, 2.0 ** -140)]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("out_dtype", ["f32", "bf16"])
def test_dequantiser_edge_cases_reach_the_kernel(layout, out_dtype):
    """Every one of the 256 symbols goes through a layer for each (zero_point, scale) pair that
    pins the oracle's dequantiser (Section II-B): scales whose products are exact bf16 ties with
    an even and with an odd kept mantissa, subnormal products (no flush to zero), products that
    are not representable (1/3), the extreme zero-points.  One batched launch holds all pairs; the
    output must equal the oracle's, bit for bit."""
    rng = np.random.default_rng(7)
    base = np.concatenate([np.arange(256, dtype=np.uint8), rng.integers(0, 256, size=5000, dtype=np.uint8)])
    prepared = []
    for i, (zp, scale) in enumerate(DEQUANT_EDGES):
        sym = np.roll(base, 17 * i)
        spec = sg.LayerSpec(f"edge{i}", (sym.size,), 8, 256, zp, 0.5, scale, 10 + i % 3, 1024, out_dtype,
                            sg.stream_key(11, i))
        T, P, f256 = oracle_pack_spec(spec, sym, layout, 32)
        want_sym, want = oracle_expected(spec, T, P)
        assert (want_sym == sym).all()
        prepared.append((to_packed_layer(spec, P, f256), want))
    # the oracle's values are themselves what the test expects them to be: ties and subnormals
    b = oracle.dequant(np.array([1, 2, 3], np.uint8), 0, 1.0 + 2.0 ** -8, "bf16")
    assert b.tolist() == [0x3F80, 0x4000, 0x4041]
    tiny = oracle.dequant(np.array([32, 33], np.uint8), 31, 3.0e-39, "f32")
    assert tiny[0] != 0.0 and tiny[0] < 1.2e-38 and tiny[1] == np.float32(2) * np.float32(3.0e-39)
    db = DeviceBatch([p[0] for p in prepared])
    for o in db.out_sets[0]:
        o.view(torch.uint8).fill_(0xA5)
    db.decode()
    assert db.read_status() == 0
    for i, (pl, want) in enumerate(prepared):
        assert np.array_equal(bits_view(db.output(i)), expected_bits(want)), f"pair {DEQUANT_EDGES[i]}"
    db.decode_per_layer()                                # the single-layer entry point takes the same values
    assert db.read_status() == 0
    for i, (pl, want) in enumerate(prepared):
        assert np.array_equal(bits_view(db.output(i)), expected_bits(want)), f"pair {DEQUANT_EDGES[i]}"


@pytest.mark.parametrize("layout", LAYOUTS)
def test_substream_ends_off_a_16_byte_boundary_are_flagged(layout):
    """An offsets table whose entries are not multiples of 16 (planted on the host) must be
    flagged as a bad length; the sub-streams it touches are not read at all."""
    spec = tiny_spec(40_000, 4, 0.6, 12, 4096, "bf16")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, layout, 32)
    for which, delta in [(3, 4), (len(P.sub_offsets) - 1, -1), (1, 8), (2, -12)]:
        o = P.sub_offsets.copy()
        o[which] = np.uint64(int(o[which]) + delta)
        db = DeviceBatch([to_packed_layer(spec, oracle.Packed(P.layout, P.stream, o, P.lane_meta, P.n, P.chunk,
                                                              P.groups), f256)])
        guard = torch.full((1 << 16,), 0x5A, dtype=torch.uint8, device="cuda")
        db.decode()
        assert db.read_status() & 2
        assert (guard == 0x5A).all()
    db = DeviceBatch([to_packed_layer(spec, P, f256)])   # and the context is still good
    db.decode()
    assert db.read_status() == 0


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("idle", [False, True])
@pytest.mark.parametrize("big", [False, True])
def test_launches_queued_back_to_back_with_the_descriptor_flags(layout, idle, big):
    """ANS_DESC_INPUTS_SETTLED / ANS_DESC_OUTPUT_IDLE on the general kernel: launches queued behind a
    device-side spin, rotating over three output sets, every set poisoned first and compared with the
    oracle afterwards; small layers (CTAs of four warps) and one big enough for the many-warp shape."""
    if big:
        specs = [tiny_spec(6_000_000, 3, 0.7, 8, 16384, "bf16", index=0)]
    else:
        specs = [tiny_spec(200_000, 3, 0.8, 9, 8192, "bf16", index=0), tiny_spec(50_001, 5, 0.6, 11, 4096, "f32", index=1),
                 tiny_spec(0, 2, 0.8, 6, 4096, "u8", index=2), tiny_spec(99_999, 2, 0.9, 7, 16384, "u8", index=3)]
    prepared = []
    for spec in specs:
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, layout, 32)
        prepared.append((to_packed_layer(spec, P, f256), oracle_expected(spec, T, P)[1]))
    db = DeviceBatch([p[0] for p in prepared], n_out_sets=3, inputs_settled=True, output_idle=idle)
    for outs in db.out_sets:
        for o in outs:
            o.view(torch.uint8).fill_(0xA5)
    torch.cuda.synchronize()
    torch.cuda._sleep(20_000_000)
    for i in range(12):
        db.decode(i % 3)
    assert db.read_status() == 0
    for k in range(3):
        for i, (pl, want) in enumerate(prepared):
            assert (bits_view(db.output(i, k)) == expected_bits(want)).all(), (k, i)


def test_bitwidth_check():
    spec = tiny_spec(5000, 4, 0.6, 12, 4096, "u8")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, ans.ANS_LAYOUT_INTERLEAVED, 32)
    pl = to_packed_layer(spec, P, f256)
    pl.bitwidth, pl.zero_point = 2, 1                    # alphabet 15 does not fit 2 bits
    db = DeviceBatch([pl])
    db.decode()
    assert db.read_status() & 4


@pytest.mark.parametrize("layout", LAYOUTS)
def test_host_buffer_entry_point(layout):
    spec = tiny_spec(100_000, 3, 0.7, 12, 16384, "bf16")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, layout, 32)
    _, want = oracle_expected(spec, T, P)
    pl = to_packed_layer(spec, P, f256)
    db = DeviceBatch([pl])                               # for the table only
    d = db.h_descs[0][0]
    need = ans.ans_host_scratch_bytes(d, pl.stream.nbytes)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    out = np.zeros(spec.n, dtype=np.uint16)
    rc = ans.ans_decode_dequant_host(d, pl.stream, pl.sub_offsets, pl.lane_meta, out, scratch.data_ptr(), need,
                                     torch.cuda.current_stream().cuda_stream)
    assert rc == ans.ANS_OK and (out == want).all()
    bad = pl.stream.copy(); bad[100] ^= 0xFF
    rc = ans.ans_decode_dequant_host(d, bad, pl.sub_offsets, pl.lane_meta, out, scratch.data_ptr(), need,
                                     torch.cuda.current_stream().cuda_stream)
    assert rc == ans.ANS_ERR_CORRUPT


def test_device_tables_match_oracle_tables():
    """ans_build_decode_tables against the oracle's table, entry by entry, and the pre-walked
    entries against a walk of the oracle's table."""
    specs = [tiny_spec(30_000, b, p, R, 4096, index=i) for i, (b, p, R) in
             enumerate([(1, 0.6, 1), (2, 0.9, 2), (4, 0.6, 6), (5, 0.85, 8), (8, 0.95, 12), (3, 0.7, 12), (8, 0.5, 14)])]
    layers = []
    tabs = []
    for spec in specs:
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, ans.ANS_LAYOUT_PRIVATE, 32)
        layers.append(to_packed_layer(spec, P, f256)); tabs.append(T)
    db = DeviceBatch(layers)
    raw = db.tables.cpu().numpy()
    for spec, T, off in zip(specs, tabs, db.table_offsets):
        L = 1 << spec.table_log
        blob = raw[int(off):int(off) + ans.ans_table_bytes(spec.table_log)]
        hdr = blob[:16].view(np.uint32)
        single = blob[1040:1040 + 4 * L].view(np.uint32)
        multi = blob[1040 + 4 * L:1040 + 8 * L].view(np.uint32)
        ent = T.entries()
        assert hdr[1] == spec.table_log and hdr[2] == spec.alphabet
        dom = [s for s in range(spec.alphabet) if 2 * int(T.freqs[s]) > L]
        assert hdr[3] == (dom[0] if dom else 0xFFFFFFFF)
        for i, (s, nb, nx) in enumerate(ent):
            assert single[i] == (s | nb << 8 | nx << 16)
            cur, run = i, 0
            while run < 15 and ent[cur][1] == 0:
                assert ent[cur][0] == dom[0]
                cur, run = ent[cur][2], run + 1
            s2, nb2, nx2 = ent[cur]
            assert multi[i] == (s2 | nb2 << 8 | run << 12 | nx2 << 16)
