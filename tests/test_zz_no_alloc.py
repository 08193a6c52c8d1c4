"""The allocation-free host-buffer call, ans_decode_dequant_host_noalloc.

Some users of this library run where device memory may not be allocated: a plug-in inside an
application that owns the whole memory budget, a real-time loop that may not enter the
allocator.  For them the library carries a fixed working area of its own, and this call decodes
one layer from host buffers to a host buffer inside it.  Checked here, through the C ABI:
the call gives bit for bit what the ordinary host-buffer call gives and what the CPU oracle
gives, on streams the oracle encoded, in every container, twice in a row (the second call
finds the first call's bytes in the shared area); it takes no device memory; it refuses
what does not fit."""
import numpy as np
import pytest
import torch

import oracle
import synthgen as sg
import paper_2406_06237_b200 as ans
from paper_2406_06237_b200.runtime import DeviceBatch, pack_layer
from helpers import expected_bits, oracle_expected, oracle_pack_spec, tiny_spec, to_packed_layer

pytestmark = pytest.mark.gpu
NP_DTYPE = {"u8": np.uint8, "bf16": np.uint16, "f32": np.uint32}


def _both_ways(spec, layout, lanes):
    """One layer, encoded by the oracle, through the ordinary host-buffer call and through the
    allocation-free one; both must equal the oracle's decode + dequantise."""
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, layout, lanes)
    want_sym, want = oracle_expected(spec, T, P)
    assert (want_sym == sym).all()
    pl = to_packed_layer(spec, P, f256)
    st = torch.cuda.current_stream().cuda_stream
    # the existing entry point: caller-allocated table and scratch
    db = DeviceBatch([pl])
    d = db.h_descs[0][0]
    need = ans.ans_host_scratch_bytes(d, pl.stream.nbytes)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    ordinary = np.zeros(spec.n, dtype=NP_DTYPE[spec.out_dtype])
    assert ans.ans_decode_dequant_host(d, pl.stream, pl.sub_offsets, pl.lane_meta, ordinary, scratch.data_ptr(),
                                       need, st) == ans.ANS_OK
    # the allocation-free entry point: host buffers only, and no device memory taken by it
    got = np.full(spec.n, 0xA5, dtype=NP_DTYPE[spec.out_dtype])
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    rc = ans.ans_decode_dequant_host_noalloc(d, pl.freqs, spec.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta,
                                             got, st)
    free_after = torch.cuda.mem_get_info()[0]
    assert rc == ans.ANS_OK
    assert free_after == free_before, "the allocation-free call changed the device's free memory"
    assert np.array_equal(got, ordinary)                  # bit-exact, as everywhere else in this suite
    assert np.array_equal(got, expected_bits(want))       # and equal to the oracle
    return pl, d


def test_two_calls_in_a_row_match_the_ordinary_call_and_the_oracle():
    # the first call on the device looks up the working area's address (module load happens here,
    # before any free-memory reading is compared)
    warm = tiny_spec(4096, 3, 0.7, 8, 1024, "u8", index=9)
    sym = sg.draw_symbols(warm)
    T, P, f256 = oracle_pack_spec(warm, sym, ans.ANS_LAYOUT_QUADS, 32)
    pl = to_packed_layer(warm, P, f256)
    d = DeviceBatch([pl]).h_descs[0][0]
    out = np.zeros(warm.n, dtype=np.uint8)
    assert ans.ans_decode_dequant_host_noalloc(d, pl.freqs, warm.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta,
                                               out, torch.cuda.current_stream().cuda_stream) == ans.ANS_OK
    assert (out == sym).all()
    # different layers back to back, in every container: each call finds the previous call's
    # bytes in the shared working area and must not be disturbed by them
    _both_ways(tiny_spec(200_000, 3, 0.7, 12, 16384, "bf16", index=1), ans.ANS_LAYOUT_QUADS, 32)
    _both_ways(tiny_spec(200_000, 3, 0.7, 12, 16384, "bf16", index=1), ans.ANS_LAYOUT_QUADS, 32)
    _both_ways(tiny_spec(70_001, 4, 0.6, 11, 4096, "f32", index=2), ans.ANS_LAYOUT_INTERLEAVED, 64)
    _both_ways(tiny_spec(333_333, 2, 0.9, 8, 16384, "bf16", index=4), ans.ANS_LAYOUT_QUADS, 128)
    pl, d = _both_ways(tiny_spec(150_000, 6, 0.9, 12, 16384, "u8", index=3), ans.ANS_LAYOUT_PRIVATE, 32)
    # a corrupt stream after good ones: flagged, and the status word is clean again afterwards
    bad = pl.stream.copy(); bad[17] ^= 0xFF
    out = np.zeros(pl.n_symbols, dtype=np.uint8)
    st = torch.cuda.current_stream().cuda_stream
    assert ans.ans_decode_dequant_host_noalloc(d, pl.freqs, pl.alphabet, bad, pl.sub_offsets, pl.lane_meta, out,
                                               st) == ans.ANS_ERR_CORRUPT
    assert ans.ans_decode_dequant_host_noalloc(d, pl.freqs, pl.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta,
                                               out, st) == ans.ANS_OK


def test_a_layer_beyond_the_fixed_area_is_refused():
    limit = ans.ans_noalloc_max_bytes()
    assert limit == 8 << 20
    spec = tiny_spec(3_000_000, 3, 0.7, 12, 32768, "f32")      # 12 MB of fp32 output
    sym = sg.draw_symbols(spec)
    pl = pack_layer(sym, spec.alphabet, spec.table_log, spec.chunk_symbols, 32, ans.ANS_LAYOUT_PRIVATE,
                    spec.bitwidth, spec.zero_point, spec.scale, ans.ANS_F32)
    d = ans.ans_layer_desc()
    d.n_symbols, d.chunk_symbols, d.lanes, d.table_log = pl.n_symbols, pl.chunk_symbols, pl.lanes, pl.table_log
    d.bitwidth, d.zero_point, d.scale, d.out_dtype, d.layout = pl.bitwidth, pl.zero_point, pl.scale, ans.ANS_F32, pl.layout
    out = np.zeros(spec.n, dtype=np.uint32)
    with pytest.raises(ans.AnsError) as e:
        ans.ans_decode_dequant_host_noalloc(d, pl.freqs, spec.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta, out)
    assert e.value.code == ans.ANS_ERR_BUFFER_TOO_SMALL
    # sizes that would wrap the layout arithmetic are refused the same way, not decoded
    for n, sb in [(1 << 62, pl.stream.nbytes), (pl.n_symbols, (1 << 64) - 200), ((1 << 64) - 1, (1 << 64) - 1)]:
        d.n_symbols = n
        rc = ans.lib().ans_decode_dequant_host_noalloc(d, pl.freqs.ctypes.data, spec.alphabet, pl.stream.ctypes.data,
                                                       sb, pl.sub_offsets.ctypes.data, pl.lane_meta.ctypes.data,
                                                       out.ctypes.data, None)
        assert rc == ans.ANS_ERR_BUFFER_TOO_SMALL
    # an empty layer is fine, but its descriptor is still checked
    d.n_symbols = 0
    assert ans.ans_decode_dequant_host_noalloc(d, pl.freqs, spec.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta,
                                               out) == ans.ANS_OK
    d.table_log = 99
    with pytest.raises(ans.AnsError):
        ans.ans_decode_dequant_host_noalloc(d, pl.freqs, spec.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta, out)
