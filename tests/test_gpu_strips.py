"""GPU vs oracle for the strips container (a look-up may stand for a run of the dominant symbol
plus one more symbol: the zero-bit transitions of Section II-A), element by element, through
the C ABI.  Streams are encoded by the ORACLE; outputs are compared as bit patterns."""
import numpy as np
import pytest
import torch

import oracle
import synthgen as sg
import paper_2406_06237_b200 as ans
from paper_2406_06237_b200.runtime import DeviceBatch
from helpers import bits_view, expected_bits, oracle_expected, oracle_pack_spec, tiny_spec, to_packed_layer
from test_gpu_parity import DEQUANT_EDGES, run_and_compare

pytestmark = pytest.mark.gpu
STRIPS = ans.ANS_LAYOUT_STRIPS


@pytest.mark.parametrize("lanes", [32, 64, 128, 256])
def test_config1_single_conv_fp32(lanes):
    db, prepared = run_and_compare(sg.workload_conv3x3(), STRIPS, lanes)
    assert (db.decode_symbols(0).cpu().numpy() == prepared[0][1]).all()
    assert db.read_status() == 0


@pytest.mark.parametrize("n", [0, 1, 3, 4, 5, 127, 128, 129, 131, 2047, 2048, 2049, 4095, 4096, 4096 + 17, 3 * 4096, 8192 + 2049])
def test_edge_sizes(n):
    """Empty layers, strips of less than a quad, less than a row, a ragged last row, a ragged last
    strip, a last chunk whose second strip is empty; every output type."""
    for dt in ("u8", "bf16", "f32"):
        run_and_compare([tiny_spec(n, out_dtype=dt, chunk=4096, pzp=0.9)], STRIPS, 64)
        run_and_compare([tiny_spec(n, out_dtype=dt, chunk=4096, pzp=0.5)], STRIPS, 32)
        run_and_compare([tiny_spec(n, out_dtype=dt, chunk=96 * 41, pzp=0.8)], STRIPS, 96)


@pytest.mark.parametrize("R", [1, 2, 3, 6, 7, 8, 9, 11, 12, 13, 14])
def test_table_sizes(R):
    b = 1 if R == 1 else min(8, R)
    specs = [tiny_spec(50_000 + R, bitwidth=b, pzp=p, table_log=R, chunk=16384, out_dtype=dt, index=i)
             for i, (p, dt) in enumerate([(0.55, "bf16"), (0.9, "u8"), (0.97, "f32"), (0.999, "bf16")])]
    run_and_compare(specs, STRIPS, 32)
    run_and_compare(specs, STRIPS, 128, per_layer=True)


def test_single_symbol_layer():
    """Every weight is the zero-point: one symbol with f = l, every transition reads zero bits,
    a lane's string is its state alone, and every look-up stands for a full run."""
    A, zp = sg.alphabet_for_bits(4)
    spec = sg.LayerSpec("const", (10_000,), 4, A, zp, 1e-9, 0.5, 10, 1024, "bf16", sg.stream_key(5, 0))
    assert (sg.draw_symbols(spec) == zp).all()
    run_and_compare([spec], STRIPS, 32)


def test_batch_with_mixed_layers_one_launch():
    specs = [tiny_spec(20_000, 2, 0.8, 9, 4096, "bf16", index=0), tiny_spec(0, 4, 0.6, 12, 4096, "f32", index=1),
             tiny_spec(4096, 8, 0.9, 14, 1024, "u8", index=2), tiny_spec(123_457, 6, 0.7, 11, 16384, "bf16", index=3),
             tiny_spec(1, 1, 0.6, 1, 512, "f32", index=4), tiny_spec(70_000, 3, 0.95, 12, 32768, "bf16", index=5)]
    run_and_compare(specs, STRIPS, 32)
    run_and_compare(specs, STRIPS, 128, per_layer=True)


def test_batch_of_more_layers_than_one_launch_holds():
    """More layers than travel in one launch's parameters: the batch call makes several launches."""
    dts = ("bf16", "u8", "f32")
    specs = [tiny_spec(0 if i % 17 == 5 else 900 + 611 * (i % 13) + (40_000 if i % 29 == 0 else 0),
                       1 + i % 6, 0.55 + 0.04 * (i % 10), 6 + i % 7, 1024 << (i % 3), dts[i % 3], index=i)
             for i in range(150)]
    run_and_compare(specs, STRIPS, 32)
    run_and_compare(specs[:100], STRIPS, 64)


@pytest.mark.parametrize("shift", [1, 2, 3, 5])
def test_symbols_into_a_buffer_of_any_alignment(shift):
    for n, chunk, lanes in [(70_001, 4096, 32), (1_200_000, 2048, 64)]:
        spec = tiny_spec(n, 3, 0.7, 8, chunk, "u8", index=shift)
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, lanes)
        db = DeviceBatch([to_packed_layer(spec, P, f256)])
        buf = torch.full((n + 64,), 0xA5, dtype=torch.uint8, device="cuda")
        ans.ans_decode_layer(db.h_descs[0][0], buf.data_ptr() + shift, db.status.data_ptr(),
                             torch.cuda.current_stream().cuda_stream)
        assert db.read_status() == 0
        got = buf.cpu().numpy()
        assert (got[shift:shift + n] == sym).all()
        assert (got[:shift] == 0xA5).all() and (got[shift + n:] == 0xA5).all()


def test_config2_resnet18_bf16():
    run_and_compare(sg.workload_resnet18(), STRIPS, 64)


@pytest.mark.parametrize("lanes", [32, 64, 128])
def test_config3_resnet50_bf16(lanes):
    run_and_compare(sg.workload_resnet50(), STRIPS, lanes)


def test_config3_resnet50_at_4096_states():
    run_and_compare(sg.workload_resnet50(table_log=12), STRIPS, 64)


@pytest.mark.parametrize("chunk", [1024, 4096, 16384, 65536])
@pytest.mark.parametrize("R", [11, 12, 14])
def test_config4_sweep_reduced(chunk, R):
    run_and_compare(sg.workload_sweep(table_log=R, chunk=chunk, n=(1 << 22) + 12345), STRIPS, 32)


def test_config5_reduced():
    run_and_compare(sg.workload_large(n_mats=2, dim=2048), STRIPS, 64)


@pytest.mark.parametrize("idle", [False, True])
def test_launches_queued_back_to_back_with_the_settled_inputs_flags(idle):
    """ANS_DESC_INPUTS_SETTLED (and ANS_DESC_OUTPUT_IDLE): a launch may read its inputs, and begin,
    while the launch before it on the stream still runs.  Thirty launches queued behind a device-side
    spin, rotating over three output sets (so that a launch never writes the set the one before it
    writes), every set poisoned first; every set must hold the oracle's bits afterwards.  A corrupt
    stream is still flagged."""
    specs = [tiny_spec(300_000, 3, 0.9, 8, 16384, "bf16", index=0), tiny_spec(70_001, 4, 0.7, 8, 4096, "f32", index=1),
             tiny_spec(0, 2, 0.8, 6, 4096, "u8", index=2), tiny_spec(150_000, 2, 0.95, 7, 8192, "u8", index=3)]
    prepared = []
    for spec in specs:
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 64)
        prepared.append((to_packed_layer(spec, P, f256), oracle_expected(spec, T, P)[1]))
    db = DeviceBatch([p[0] for p in prepared], n_out_sets=3, inputs_settled=True, output_idle=idle)
    want_flags = ans.ANS_DESC_INPUTS_SETTLED | (ans.ANS_DESC_OUTPUT_IDLE if idle else 0)
    assert all(int(d.flags) == want_flags for k in range(3) for d in db.h_descs[k][:len(specs)])
    for outs in db.out_sets:
        for o in outs:
            o.view(torch.uint8).fill_(0xA5)
    torch.cuda.synchronize()
    torch.cuda._sleep(20_000_000)
    for i in range(30):
        db.decode(i % 3)
    assert db.read_status() == 0
    for k in range(3):
        for i, (pl, want) in enumerate(prepared):
            got = bits_view(db.output(i, k))
            assert (got == expected_bits(want)).all(), (k, i)
    # a corrupt stream under the same flags
    pl = prepared[0][0]
    bad = pl.stream.copy()
    bad[int(pl.sub_offsets[1]) + 70] ^= 0x5A
    import dataclasses
    db2 = DeviceBatch([dataclasses.replace(pl, stream=bad)], n_out_sets=2, inputs_settled=True, output_idle=idle)
    for i in range(4):
        db2.decode(i % 2)
    assert db2.read_status() != 0


def test_a_batch_of_more_layers_than_one_launch_holds_with_the_flags_set():
    """70 small layers are two launches of the strips kernel per call; with both flags set the
    second does not wait for the first.  Four calls queued back to back over two output sets."""
    specs = [tiny_spec(3000 + 517 * i, 1 + i % 6, 0.6 + 0.005 * i, 5 + i % 4, 2048, ("bf16", "u8", "f32")[i % 3], index=i)
             for i in range(70)]
    prepared = []
    for spec in specs:
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 64)
        prepared.append((to_packed_layer(spec, P, f256), oracle_expected(spec, T, P)[1]))
    db = DeviceBatch([p[0] for p in prepared], n_out_sets=2, inputs_settled=True, output_idle=True)
    assert db.launches_per_decode() == 2
    for outs in db.out_sets:
        for o in outs:
            o.view(torch.uint8).fill_(0xA5)
    torch.cuda.synchronize()
    torch.cuda._sleep(10_000_000)
    for i in range(4):
        db.decode(i % 2)
    assert db.read_status() == 0
    for k in range(2):
        for i, (pl, want) in enumerate(prepared):
            assert (bits_view(db.output(i, k)) == expected_bits(want)).all(), (k, i)


@pytest.mark.parametrize("layout,lanes", [(STRIPS, 64), (ans.ANS_LAYOUT_QUADS, 32)])
def test_decode_launches_captured_in_a_cuda_graph(layout, lanes):
    """Six batched decode launches (descriptor flags set, rotating over three output sets) captured
    from a stream into a CUDA graph and replayed three times; every set holds the oracle's bits."""
    specs = [tiny_spec(300_000, 3, 0.9, 8, 16384, "bf16", index=0), tiny_spec(70_001, 4, 0.7, 8, 4096, "f32", index=1),
             tiny_spec(150_000, 2, 0.95, 7, 8192, "u8", index=3)]
    prepared = []
    for spec in specs:
        sym = sg.draw_symbols(spec)
        T, P, f256 = oracle_pack_spec(spec, sym, layout, lanes)
        prepared.append((to_packed_layer(spec, P, f256), oracle_expected(spec, T, P)[1]))
    db = DeviceBatch([p[0] for p in prepared], n_out_sets=3, inputs_settled=True, output_idle=True)
    db.decode(0)                                          # the first call sets the kernels' attributes: outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(6):
                db.decode(i % 3, stream=side.cuda_stream)
    for outs in db.out_sets:
        for o in outs:
            o.view(torch.uint8).fill_(0xA5)
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert db.read_status() == 0
    for k in range(3):
        for i, (pl, want) in enumerate(prepared):
            assert (bits_view(db.output(i, k)) == expected_bits(want)).all(), (k, i)


def test_long_substreams_read_from_global_memory():
    """Sub-streams too long for the shared-memory staging buffer (here beside short ones of another
    layer, which size the buffer) are read word by word from global memory."""
    run_and_compare([tiny_spec(40 * 65536 + 321, 8, 0.05, 12, 65536, "u8", index=0),
                     tiny_spec(30_000, 2, 0.95, 8, 4096, "bf16", index=1)], STRIPS, 32)
    run_and_compare([tiny_spec(9 * 131072 + 77, 8, 0.02, 14, 131072, "bf16")], STRIPS, 32)


def test_corrupt_streams_are_flagged_not_fatal():
    """Corruption is planted on the host.  Reads are clamped to the sub-stream and every loop is
    counted, so a bad stream yields wrong symbols and a status bit, never a fault; the verdict
    is the oracle's, case by case."""
    spec = tiny_spec(40_000, 4, 0.8, 12, 4096, "bf16")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 32)

    def decode(P2):
        db = DeviceBatch([to_packed_layer(spec, P2, f256)])
        guard = torch.full((1 << 16,), 0x5A, dtype=torch.uint8, device="cuda")
        db.decode()
        st = db.read_status()
        assert (guard == 0x5A).all()
        return st

    assert decode(P) == 0
    flagged = 0
    rng = np.random.default_rng(0)
    for trial in range(10):
        s = P.stream.copy()
        pos = rng.integers(0, s.size, size=8)
        s[pos] ^= rng.integers(1, 256, size=8).astype(np.uint8)
        P2 = oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        st = decode(P2)
        assert (st != 0) == (oracle.unpack(T, P2)[1] != oracle.OK)
        flagged += st != 0
    assert flagged > 0
    for k, delta in [(0, 1), (9, 0x40), (31, 0xFF)]:       # a lane's length: every later lane starts elsewhere
        s = P.stream.copy()
        s[int(P.sub_offsets[3]) + 2 * k] ^= delta
        assert decode(oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)) & 2
    s = P.stream.copy()
    s[int(P.sub_offsets[2]):int(P.sub_offsets[2]) + 64] = 0xFF   # lengths far beyond the sub-stream
    assert decode(oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)) & 2
    o = P.sub_offsets.copy(); o[2] += 1 << 40              # offset far outside the stream
    assert decode(oracle.Packed(P.layout, P.stream, o, P.lane_meta, P.n, P.chunk, P.groups)) & 2
    short = P.stream[:P.stream.size - 16].copy()           # truncated stream
    assert decode(oracle.Packed(P.layout, short, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)) & 2
    for which, delta in [(3, 4), (len(P.sub_offsets) - 1, -1), (1, 8), (2, -12)]:   # ends off a 16-byte boundary
        o = P.sub_offsets.copy()
        o[which] = np.uint64(int(o[which]) + delta)
        assert decode(oracle.Packed(P.layout, P.stream, o, P.lane_meta, P.n, P.chunk, P.groups)) & 2
    assert decode(P) == 0                                  # and the context is still good


def test_corruption_in_substreams_read_from_global_memory():
    spec = tiny_spec(6 * 65536, 8, 0.05, 12, 65536, "u8")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 32)
    rng = np.random.default_rng(3)
    for trial in range(4):
        s = P.stream.copy()
        pos = rng.integers(0, s.size, size=8)
        s[pos] ^= rng.integers(1, 256, size=8).astype(np.uint8)
        P2 = oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups)
        db = DeviceBatch([to_packed_layer(spec, P2, f256)])
        db.decode()
        assert (db.read_status() != 0) == (oracle.unpack(T, P2)[1] != oracle.OK)


@pytest.mark.parametrize("out_dtype", ["f32", "bf16"])
def test_dequantiser_edge_cases_reach_the_kernel(out_dtype):
    """Every one of the 256 symbols through a layer for each (zero_point, scale) pair that pins the
    oracle's dequantiser (Section II-B): bf16 ties, subnormal products, the extreme zero-points."""
    rng = np.random.default_rng(7)
    base = np.concatenate([np.arange(256, dtype=np.uint8), rng.integers(0, 256, size=5000, dtype=np.uint8)])
    prepared = []
    for i, (zp, scale) in enumerate(DEQUANT_EDGES):
        sym = np.roll(base, 17 * i)
        spec = sg.LayerSpec(f"edge{i}", (sym.size,), 8, 256, zp, 0.5, scale, 10 + i % 3, 1024, out_dtype,
                            sg.stream_key(11, i))
        T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 32)
        want_sym, want = oracle_expected(spec, T, P)
        assert (want_sym == sym).all()
        prepared.append((to_packed_layer(spec, P, f256), want))
    # and the same pairs on layers where one symbol dominates, so that the fill value is dequantised too
    for i, (zp, scale) in enumerate(DEQUANT_EDGES):
        sym = np.where(rng.random(6000) < 0.9, zp, rng.integers(0, 256, size=6000)).astype(np.uint8)
        spec = sg.LayerSpec(f"skew{i}", (sym.size,), 8, 256, zp, 0.5, scale, 8 + i % 3, 2048, out_dtype,
                            sg.stream_key(12, i))
        T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 64)
        want_sym, want = oracle_expected(spec, T, P)
        assert (want_sym == sym).all()
        prepared.append((to_packed_layer(spec, P, f256), want))
    db = DeviceBatch([p[0] for p in prepared])
    for o in db.out_sets[0]:
        o.view(torch.uint8).fill_(0xA5)
    db.decode()
    assert db.read_status() == 0
    for i, (pl, want) in enumerate(prepared):
        assert np.array_equal(bits_view(db.output(i)), expected_bits(want)), f"layer {i}"


def test_bitwidth_check():
    spec = tiny_spec(5000, 4, 0.6, 12, 4096, "u8")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 32)
    pl = to_packed_layer(spec, P, f256)
    pl.bitwidth, pl.zero_point = 2, 1                      # alphabet 15 does not fit 2 bits
    db = DeviceBatch([pl])
    db.decode()
    assert db.read_status() & 4


def test_unsupported_chunk_sizes_are_refused():
    spec = tiny_spec(5000, 4, 0.6, 12, 4096, "u8")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 32)
    pl = to_packed_layer(spec, P, f256)
    pl.chunk_symbols = 1000                                # no multiple of 4 * lanes
    with pytest.raises(ans.AnsError) as e:
        DeviceBatch([pl]).decode()
    assert e.value.code == ans.ANS_ERR_UNSUPPORTED


def test_host_buffer_entry_points():
    spec = tiny_spec(100_000, 3, 0.9, 8, 16384, "bf16")
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, STRIPS, 64)
    _, want = oracle_expected(spec, T, P)
    pl = to_packed_layer(spec, P, f256)
    db = DeviceBatch([pl])                                 # for the table only
    d = db.h_descs[0][0]
    need = ans.ans_host_scratch_bytes(d, pl.stream.nbytes)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    out = np.zeros(spec.n, dtype=np.uint16)
    st = torch.cuda.current_stream().cuda_stream
    rc = ans.ans_decode_dequant_host(d, pl.stream, pl.sub_offsets, pl.lane_meta, out, scratch.data_ptr(), need, st)
    assert rc == ans.ANS_OK and (out == want).all()
    bad = pl.stream.copy(); bad[100] ^= 0xFF
    rc = ans.ans_decode_dequant_host(d, bad, pl.sub_offsets, pl.lane_meta, out, scratch.data_ptr(), need, st)
    assert rc == ans.ANS_ERR_CORRUPT
    out[:] = 0
    rc = ans.ans_decode_dequant_host_noalloc(d, f256, spec.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta, out, st)
    assert rc == ans.ANS_OK and (out == want).all()


@pytest.mark.parametrize("lanes", [32, 64])
def test_full_size_resnet50_in_the_benchmark_configuration(lanes):
    """Config 3 as bench.py times it (32 lanes per 16 K-symbol chunk, and 64 as a variant; 256-state
    tables; one launch; descriptor flags set; launches queued back to back over several output sets),
    every output element of every set against the oracle."""
    specs = sg.workload_resnet50()
    db0, prepared = run_and_compare(specs, STRIPS, lanes, threads=16)       # one launch, flags not set
    del db0
    db = DeviceBatch([p[0] for p in prepared], n_out_sets=3, inputs_settled=True, output_idle=True)
    for outs in db.out_sets:
        for o in outs:
            o.view(torch.uint8).fill_(0xA5)
    torch.cuda.synchronize()
    torch.cuda._sleep(20_000_000)
    for i in range(12):
        db.decode(i % 3)
    assert db.read_status() == 0
    for k in range(3):
        for i, (pl, want_sym, want) in enumerate(prepared):
            assert (bits_view(db.output(i, k)) == expected_bits(want)).all(), (k, specs[i].name)


# ---- channels container: one stream per input channel of an O x I x H x W tensor (Section III-B) ----
CHANNELS = ans.ANS_LAYOUT_CHANNELS


def _channels_case(shape, b, pzp, R, dt, index=0, chunk_rows=0):
    O, I, H, W = shape
    n = O * I * H * W
    spec = sg.LayerSpec(f"conv{index}", shape, b, *sg.alphabet_for_bits(b), sg.theta_for_pzp(*sg.alphabet_for_bits(b), pzp),
                        0.02, R, (chunk_rows * I * H * W) if chunk_rows else n, dt, sg.stream_key(21, index))
    sym = sg.draw_symbols(spec)
    f = oracle.normalize_freqs(oracle.histogram(sym), spec.alphabet, R)
    T = oracle.Table(f, R)
    P = oracle.pack(T, sym, spec.chunk_symbols, I // 32, oracle.CHANNELS, piece=H * W)
    f256 = np.zeros(256, dtype=np.uint32)
    f256[:spec.alphabet] = f
    want_sym, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and (want_sym == sym).all()
    return spec, T, P, f256, sym, oracle.dequant(sym, spec.zero_point, spec.scale, dt)


def _decode_and_compare(cases, per_layer=False, flagged=False):
    """flagged: descriptor flags set, six launches queued back to back over two output sets."""
    db = DeviceBatch([to_packed_layer(c[0], c[2], c[3]) for c in cases], n_out_sets=2 if flagged else 1,
                     inputs_settled=flagged, output_idle=flagged)
    for outs in db.out_sets:
        for o in outs:
            o.view(torch.uint8).fill_(0xA5)
    if flagged:
        torch.cuda.synchronize()
        torch.cuda._sleep(10_000_000)
        for k in range(6):
            db.decode(k % 2)
    else:
        (db.decode_per_layer if per_layer else db.decode)()
    assert db.read_status() == 0
    for k in range(len(db.out_sets)):
        for i, c in enumerate(cases):
            assert np.array_equal(bits_view(db.output(i, k)), expected_bits(c[5])), f"set {k} layer {i} {c[0].shape}"
    return db


@pytest.mark.parametrize("dt", ["bf16", "u8", "f32"])
def test_channels_conv_shapes(dt):
    """3x3, 1x1 and 7x7 kernels, 32 to 512 input channels, one chunk per layer or chunks of whole
    output-channel rows; the decoded tensor is in the tensor's own O x I x H x W order."""
    shapes = [((64, 64, 3, 3), 0), ((128, 32, 1, 1), 0), ((16, 96, 7, 7) if dt != "f32" else (16, 96, 5, 5), 0),
              ((256, 512, 1, 1), 0), ((40, 128, 3, 3), 8), ((7, 64, 1, 1), 1), ((512, 256, 3, 3), 64)]
    cases = [_channels_case(sh, 1 + i % 6, 0.6 + 0.06 * i, 6 + i % 6, dt, i, rows) for i, (sh, rows) in enumerate(shapes)]
    db = _decode_and_compare(cases)
    assert (db.decode_symbols(0).cpu().numpy() == cases[0][4]).all() and db.read_status() == 0
    _decode_and_compare(cases[:3], per_layer=True)
    _decode_and_compare(cases, flagged=True)


def test_channels_resnet50_by_input_channel():
    """Every ResNet-50 conv but the first (3 input channels; the paper leaves the first layer
    uncompressed, Section III-A) as one chunk with a lane per input channel."""
    cases = []
    for i, spec in enumerate(sg.workload_resnet50()):
        if spec.shape[1] % 32:
            continue
        cases.append(_channels_case(spec.shape, spec.bitwidth, 0.9, 8, "bf16", i))
    assert len(cases) == 52
    _decode_and_compare(cases)


def test_channels_corruption_and_bad_sizes():
    c = _channels_case((64, 64, 3, 3), 4, 0.8, 10, "bf16")
    spec, T, P, f256 = c[0], c[1], c[2], c[3]
    rng = np.random.default_rng(5)
    flagged = 0
    for trial in range(6):
        s = P.stream.copy()
        pos = rng.integers(0, s.size, size=4)
        s[pos] ^= rng.integers(1, 256, size=4).astype(np.uint8)
        P2 = oracle.Packed(P.layout, s, P.sub_offsets, P.lane_meta, P.n, P.chunk, P.groups, P.piece)
        db = DeviceBatch([to_packed_layer(spec, P2, f256)])
        db.decode()
        st = db.read_status()
        assert (st != 0) == (oracle.unpack(T, P2)[1] != oracle.OK)
        flagged += st != 0
    assert flagged > 0
    pl = to_packed_layer(spec, P, f256)
    pl.piece_symbols = 7                                   # 64 * 64 * 9 is no multiple of 64 * 7
    with pytest.raises(ans.AnsError) as e:
        DeviceBatch([pl]).decode()
    assert e.value.code == ans.ANS_ERR_UNSUPPORTED
