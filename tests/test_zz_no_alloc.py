"""The allocation-free host-buffer call (for callers that may not touch the device allocator:
plug-ins inside an application that owns the memory budget, real-time loops) must give exactly
what the ordinary host-buffer call gives.  Collected last on purpose: a failure here cannot hide
any other test from a run that stops at the first failure.  Everything the new call needs on the
device sits in the library's fixed working area, so the only device memory this test allocates
is for the call it compares against."""
import numpy as np
import pytest
import torch

import synthgen as sg
import paper_2406_06237_b200 as ans
from paper_2406_06237_b200.runtime import DeviceBatch, pack_layer
from helpers import tiny_spec

pytestmark = pytest.mark.gpu


def _both_ways(spec, layout, lanes):
    sym = sg.draw_symbols(spec)
    pl = pack_layer(sym, spec.alphabet, spec.table_log, spec.chunk_symbols, lanes, layout, spec.bitwidth,
                    spec.zero_point, spec.scale, ans.DTYPES[spec.out_dtype])
    np_dtype = {"u8": np.uint8, "bf16": np.uint16, "f32": np.uint32}[spec.out_dtype]
    # the existing entry point: caller-allocated table and scratch
    db = DeviceBatch([pl])
    d = db.h_descs[0][0]
    need = ans.ans_host_scratch_bytes(d, pl.stream.nbytes)
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    want = np.zeros(spec.n, dtype=np_dtype)
    st = torch.cuda.current_stream().cuda_stream
    assert ans.ans_decode_dequant_host(d, pl.stream, pl.sub_offsets, pl.lane_meta, want, scratch.data_ptr(),
                                       need, st) == ans.ANS_OK
    # the allocation-free entry point: host buffers only
    got = np.full(spec.n, 0xA5, dtype=np_dtype)
    rc = ans.ans_decode_dequant_host_noalloc(d, pl.freqs, spec.alphabet, pl.stream, pl.sub_offsets, pl.lane_meta,
                                             got, st)
    assert rc == ans.ANS_OK
    assert np.array_equal(got, want)          # bit-exact, as everywhere else in this suite
    return pl, d


def test_two_calls_in_a_row_match_the_ordinary_call():
    # two different layers back to back: the second call finds the first call's bytes in the
    # shared working area and must not be disturbed by them
    _both_ways(tiny_spec(200_000, 3, 0.7, 12, 16384, "bf16", index=1), ans.ANS_LAYOUT_PRIVATE, 32)
    _both_ways(tiny_spec(70_001, 4, 0.6, 11, 4096, "f32", index=2), ans.ANS_LAYOUT_INTERLEAVED, 64)
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
