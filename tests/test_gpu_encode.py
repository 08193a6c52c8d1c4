"""The compress side on the device against the oracle: histogram, its entropy (Section II-C:
the entropy H_W of the quantised weights that Eq. 3 regularises), normalisation to 2^R states,
and the encoder for the strips container (Section II-A), whose bytes must be the oracle's."""
import numpy as np
import pytest
import torch

import oracle
import synthgen as sg
import paper_2406_06237_b200 as ans
from paper_2406_06237_b200.runtime import DeviceBatch
from helpers import bits_view, expected_bits, oracle_pack_spec, tiny_spec, to_packed_layer

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _stream():
    return torch.cuda.current_stream().cuda_stream


@pytest.mark.parametrize("n,shift", [(0, 0), (1, 0), (15, 3), (16, 0), (17, 1), (1000, 5), (1 << 20, 0), ((1 << 22) + 13, 7)])
def test_histogram_equals_the_oracle(n, shift):
    rng = np.random.default_rng(n)
    sym = rng.integers(0, 256, size=n + 16, dtype=np.uint8)
    sym[::3] = 7
    d = _dev(sym)
    counts = torch.full((256,), 12345, dtype=torch.int64, device="cuda")
    ans.ans_histogram_device(d.data_ptr() + shift, n, counts.data_ptr(), _stream())
    torch.cuda.synchronize()
    want = oracle.histogram(sym[shift:shift + n])
    assert (counts.cpu().numpy().astype(np.uint64) == want).all()


@pytest.mark.parametrize("b,pzp,R", [(1, 0.6, 1), (2, 0.9, 2), (4, 0.6, 6), (5, 0.85, 8), (8, 0.95, 12), (3, 0.7, 12),
                                     (8, 0.5, 14), (8, 0.01, 8), (6, 0.999, 5)])
def test_normalised_frequencies_and_entropy_equal_the_oracle(b, pzp, R):
    spec = tiny_spec(200_000, b, pzp, R, 4096)
    sym = sg.draw_symbols(spec)
    d = _dev(sym)
    counts = torch.zeros(256, dtype=torch.int64, device="cuda")
    freqs = torch.full((256,), 99, dtype=torch.int32, device="cuda")
    ent = torch.zeros(2, dtype=torch.float64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ans.ans_histogram_device(d.data_ptr(), sym.size, counts.data_ptr(), _stream())
    ans.ans_normalize_freqs_device(counts.data_ptr(), spec.alphabet, R, freqs.data_ptr(), status.data_ptr(), _stream())
    ans.ans_entropy_device(counts.data_ptr(), spec.alphabet, ent.data_ptr(), _stream())
    torch.cuda.synchronize()
    c = oracle.histogram(sym)
    present = int((c > 0).sum())
    if present > (1 << R):
        assert int(status.item()) & 1
        return
    want = oracle.normalize_freqs(c, spec.alphabet, R)
    got = freqs.cpu().numpy().astype(np.uint32)
    assert int(status.item()) == 0 and (got[:spec.alphabet] == want).all() and not got[spec.alphabet:].any()
    p = c[c > 0].astype(np.float64) / sym.size
    h = float(-(p * np.log2(p)).sum())
    e = ent.cpu().numpy()
    assert abs(e[0] - h) <= 1e-12 * max(1.0, h) and abs(e[1] - h * sym.size) <= 1e-9 * max(1.0, h * sym.size)


def test_normaliser_corner_cases():
    """Ties between remainders go to the lower symbol; an overshoot (many rare symbols that each
    keep one state) is taken from the largest shares; an empty histogram is flagged."""
    cases = [([5, 5, 5, 5, 5, 5, 5], 7, 3), ([1000, 1, 1, 1, 1, 1, 1, 1, 1, 1, 1, 1, 1, 1, 1, 1], 16, 4),
             ([10, 10, 10, 1, 1, 1, 1, 1], 8, 3), ([3, 3, 2], 3, 2), ([1, 0, 0, 7], 4, 5)]
    for counts, A, R in cases:
        c = np.zeros(256, dtype=np.uint64)
        c[:len(counts)] = counts
        d = _dev(c.view(np.int64))
        freqs = torch.zeros(256, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ans.ans_normalize_freqs_device(d.data_ptr(), A, R, freqs.data_ptr(), status.data_ptr(), _stream())
        torch.cuda.synchronize()
        want = oracle.normalize_freqs(c[:A], A, R)
        assert int(status.item()) == 0 and (freqs.cpu().numpy()[:A].astype(np.uint32) == want).all(), (counts, R)
    d = _dev(np.zeros(256, dtype=np.int64))
    freqs = torch.zeros(256, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ans.ans_normalize_freqs_device(d.data_ptr(), 4, 3, freqs.data_ptr(), status.data_ptr(), _stream())
    torch.cuda.synchronize()
    assert int(status.item()) & 1


def _encode_on_device(spec, sym, lanes, f256):
    """histogram-independent part: table from f256, then the device encoder."""
    R, C = spec.table_log, spec.chunk_symbols
    n = sym.size
    tbytes = ans.ans_table_bytes(R)
    tables = torch.zeros(max(tbytes, 256), dtype=torch.uint8, device="cuda")
    ans.ans_build_decode_tables(f256[None, :], [spec.alphabet], [R], tables.data_ptr(), tables.numel(), _stream())
    n_sub = -(-n // C) * (lanes // 32)
    cap = ans.ans_host_pack_bound(n, C, lanes, ans.ANS_LAYOUT_STRIPS)
    out = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    offs = torch.full((n_sub + 1,), -1, dtype=torch.int64, device="cuda")
    need = ans.ans_encode_scratch_bytes(n, C, lanes)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    d = _dev(sym) if n else torch.zeros(1, dtype=torch.uint8, device="cuda")
    ans.ans_encode_layer_device(d.data_ptr(), n, tables.data_ptr(), R, C, lanes, ans.ANS_LAYOUT_STRIPS, out.data_ptr(),
                                cap, offs.data_ptr(), scratch.data_ptr(), need, status.data_ptr(), _stream())
    torch.cuda.synchronize()
    o = offs.cpu().numpy().astype(np.uint64)
    total = int(o[-1])
    assert (out[cap:].cpu().numpy() == 0xA5).all()
    return out[:total].cpu().numpy(), o, int(status.item())


@pytest.mark.parametrize("n,C,lanes,R,b,pzp", [(36864, 4096, 32, 12, 4, 0.6), (5000, 1024, 64, 8, 3, 0.9),
                                               (100_003, 16384, 128, 11, 6, 0.8), (33, 128, 32, 6, 2, 0.7),
                                               (70_000, 65536, 256, 14, 8, 0.3), (4097, 4096, 32, 12, 1, 0.6),
                                               (130, 512, 32, 5, 3, 0.7), (1_300_000, 16384, 64, 8, 4, 0.93),
                                               (0, 4096, 32, 8, 4, 0.6), (1, 32, 32, 1, 1, 0.6)])
def test_device_encoder_writes_the_oracles_bytes(n, C, lanes, R, b, pzp):
    spec = tiny_spec(max(n, 1), bitwidth=b, pzp=pzp, table_log=R, chunk=C)
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, oracle.STRIPS, lanes)
    sym = sym[:n]
    P = oracle.pack(T, sym, C, lanes // 32, oracle.STRIPS)
    got, offs, status = _encode_on_device(spec, sym, lanes, f256)
    assert status == 0
    assert (offs == P.sub_offsets).all()
    assert got.size == P.stream.size and (got == P.stream).all()


@pytest.mark.parametrize("shape,b,pzp,R,rows", [((64, 64, 3, 3), 3, 0.8, 8, 0), ((128, 32, 1, 1), 4, 0.6, 10, 0),
                                                ((16, 96, 7, 7), 2, 0.9, 6, 0), ((40, 128, 3, 3), 5, 0.7, 12, 8),
                                                ((512, 256, 3, 3), 3, 0.93, 8, 64)])
def test_device_encoder_writes_the_oracles_bytes_for_the_channels_container(shape, b, pzp, R, rows):
    """One stream per input channel of an O x I x H x W tensor (Section III-B), encoded on the
    device: bytes and offsets equal to the oracle's."""
    O, I, H, Wd = shape
    n, E = O * I * H * Wd, H * Wd
    C = n if not rows else rows * I * E
    spec = tiny_spec(n, bitwidth=b, pzp=pzp, table_log=R, chunk=C)
    sym = sg.draw_symbols(spec)
    f = oracle.normalize_freqs(oracle.histogram(sym), spec.alphabet, R)
    T = oracle.Table(f, R)
    P = oracle.pack(T, sym, C, I // 32, oracle.CHANNELS, piece=E)
    f256 = np.zeros(256, dtype=np.uint32)
    f256[:spec.alphabet] = f
    tables = torch.zeros(max(ans.ans_table_bytes(R), 256), dtype=torch.uint8, device="cuda")
    ans.ans_build_decode_tables(f256[None, :], [spec.alphabet], [R], tables.data_ptr(), tables.numel(), _stream())
    n_sub = -(-n // C) * (I // 32)
    cap = ans.ans_host_pack_bound(n, C, I, ans.ANS_LAYOUT_CHANNELS)
    out = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    offs = torch.full((n_sub + 1,), -1, dtype=torch.int64, device="cuda")
    need = ans.ans_encode_scratch_bytes(n, C, I)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ans.ans_encode_channels_device(_dev(sym).data_ptr(), n, tables.data_ptr(), R, C, I, E, out.data_ptr(), cap,
                                   offs.data_ptr(), scratch.data_ptr(), need, status.data_ptr(), _stream())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o = offs.cpu().numpy().astype(np.uint64)
    assert (o == P.sub_offsets).all()
    got = out[:int(o[-1])].cpu().numpy()
    assert got.size == P.stream.size and (got == P.stream).all()
    assert (out[cap:].cpu().numpy() == 0xA5).all()
    # sizes the container does not take are refused
    with pytest.raises(ans.AnsError):
        ans.ans_encode_channels_device(_dev(sym).data_ptr(), n, tables.data_ptr(), R, C, I, 0, out.data_ptr(), cap,
                                       offs.data_ptr(), scratch.data_ptr(), need, status.data_ptr(), _stream())
    with pytest.raises(ans.AnsError):
        ans.ans_encode_channels_device(_dev(sym).data_ptr(), n - 1, tables.data_ptr(), R, C, I, E, out.data_ptr(), cap,
                                       offs.data_ptr(), scratch.data_ptr(), need, status.data_ptr(), _stream())


@pytest.mark.parametrize("n,C,lanes,R,b,pzp", [(36864, 4096, 32, 12, 4, 0.6), (5000, 1024, 64, 8, 3, 0.9),
                                               (100_003, 16384, 128, 11, 6, 0.8), (33, 128, 32, 6, 2, 0.7),
                                               (70_001, 65536, 256, 14, 8, 0.3), (4097, 4096, 32, 12, 1, 0.6),
                                               (131, 512, 32, 5, 3, 0.7), (1_300_002, 32768, 32, 8, 3, 0.7),
                                               (0, 4096, 32, 8, 4, 0.6), (1, 32, 32, 1, 1, 0.6), (7, 1000, 96, 4, 2, 0.6)])
def test_device_encoder_writes_the_oracles_bytes_for_the_quads_container(n, C, lanes, R, b, pzp):
    """Bytes, offsets and lane metadata (initial state, first word) equal to the oracle's."""
    spec = tiny_spec(max(n, 1), bitwidth=b, pzp=pzp, table_log=R, chunk=C)
    sym = sg.draw_symbols(spec)
    T, _, f256 = oracle_pack_spec(spec, sym, oracle.QUADS, lanes)
    sym = sym[:n]
    P = oracle.pack(T, sym, C, lanes // 32, oracle.QUADS)
    tables = torch.zeros(max(ans.ans_table_bytes(R), 256), dtype=torch.uint8, device="cuda")
    ans.ans_build_decode_tables(f256[None, :], [spec.alphabet], [R], tables.data_ptr(), tables.numel(), _stream())
    n_sub = -(-n // C) * (lanes // 32)
    cap = ans.ans_host_pack_bound(n, C, lanes, ans.ANS_LAYOUT_QUADS)
    out = torch.full((cap + 64,), 0xA5, dtype=torch.uint8, device="cuda")
    offs = torch.full((n_sub + 1,), -1, dtype=torch.int64, device="cuda")
    meta = torch.full((max(n_sub, 1), 32), -1, dtype=torch.int32, device="cuda")
    need = ans.ans_encode_scratch_bytes(n, C, lanes)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    d = _dev(sym) if n else torch.zeros(1, dtype=torch.uint8, device="cuda")
    ans.ans_encode_quads_device(d.data_ptr(), n, tables.data_ptr(), R, C, lanes, out.data_ptr(), cap, offs.data_ptr(),
                                meta.data_ptr(), scratch.data_ptr(), need, status.data_ptr(), _stream())
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o = offs.cpu().numpy().astype(np.uint64)
    assert (o == P.sub_offsets).all()
    got = out[:int(o[-1])].cpu().numpy()
    assert got.size == P.stream.size and (got == P.stream).all()
    if n:
        assert (meta.cpu().numpy().view(np.uint32)[:n_sub] == P.lane_meta.reshape(n_sub, 32)).all()
    assert (out[cap:].cpu().numpy() == 0xA5).all()


def test_compress_then_decode_on_the_device():
    """The whole loop without the host: histogram, normalise, build the table, encode, decode +
    dequantise; the output is the oracle's dequantisation of the symbols."""
    spec = tiny_spec(500_000, 5, 0.9, 8, 16384, "bf16")
    sym = sg.draw_symbols(spec)
    d = _dev(sym)
    counts = torch.zeros(256, dtype=torch.int64, device="cuda")
    freqs = torch.zeros(256, dtype=torch.int32, device="cuda")
    ans.ans_histogram_device(d.data_ptr(), sym.size, counts.data_ptr(), _stream())
    ans.ans_normalize_freqs_device(counts.data_ptr(), spec.alphabet, 8, freqs.data_ptr(), 0, _stream())
    torch.cuda.synchronize()
    f256 = freqs.cpu().numpy().astype(np.uint32)
    got, offs, status = _encode_on_device(spec, sym, 64, f256)
    assert status == 0
    T = oracle.Table(f256[:spec.alphabet], 8)
    P = oracle.Packed(oracle.STRIPS, got, offs, np.zeros((offs.size - 1, 0), np.uint32), sym.size, 16384, 2)
    osym, rc = oracle.unpack(T, P)
    assert rc == oracle.OK and (osym == sym).all()
    db = DeviceBatch([to_packed_layer(spec, P, f256)])
    db.decode()
    assert db.read_status() == 0
    want = oracle.dequant(sym, spec.zero_point, spec.scale, "bf16")
    assert np.array_equal(bits_view(db.output(0)), expected_bits(want))


def test_encoder_flags_what_it_cannot_code():
    spec = tiny_spec(10_000, 4, 0.6, 8, 4096)
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, oracle.STRIPS, 32)
    bad = sym.copy()
    bad[1234] = 200                                        # a symbol without a state
    _, _, status = _encode_on_device(spec, bad, 32, f256)
    assert status & 4
    # a stream buffer that is too small: flagged, nothing written past it
    tables = torch.zeros(ans.ans_table_bytes(8), dtype=torch.uint8, device="cuda")
    ans.ans_build_decode_tables(f256[None, :], [spec.alphabet], [8], tables.data_ptr(), tables.numel(), _stream())
    cap = 1024
    out = torch.full((cap + 4096,), 0xA5, dtype=torch.uint8, device="cuda")
    offs = torch.zeros(4, dtype=torch.int64, device="cuda")
    need = ans.ans_encode_scratch_bytes(sym.size, 4096, 32)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ans.ans_encode_layer_device(_dev(sym).data_ptr(), sym.size, tables.data_ptr(), 8, 4096, 32, ans.ANS_LAYOUT_STRIPS,
                                out.data_ptr(), cap, offs.data_ptr(), scratch.data_ptr(), need, status.data_ptr(), _stream())
    torch.cuda.synchronize()
    assert int(status.item()) & 2 and (out[cap:].cpu().numpy() == 0xA5).all()
    assert (offs.cpu().numpy().astype(np.uint64) == P.sub_offsets).all()
