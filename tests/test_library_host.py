"""CPU-only checks of the CUDA library: it loads, exports what the header declares, its host
packer writes the same bytes as the oracle's encoder, and argument errors are reported
before any CUDA call."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import synthgen as sg
import paper_2406_06237_b200 as ans
from helpers import oracle_pack_spec, tiny_spec

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "ans_b200.h")).read()
    declared = set(re.findall(r"^\s*(?:int|const char\*)\s+(ans_\w+)\s*\(", hdr, flags=re.M))
    assert declared and declared == set(ans.binding.EXPORTS)
    L = ans.lib()
    for name in declared:
        assert getattr(L, name) is not None
    assert ans.ans_version() >= 100
    assert "invalid" in ans.ans_strerror(ans.ANS_ERR_INVALID_ARG)


def test_descriptor_layout_matches_header():
    # 5 pointers, 2 u64, then 4-byte fields: the ctypes mirror must have the C struct's size
    assert ctypes.sizeof(ans.ans_layer_desc) == 5 * 8 + 2 * 8 + 12 * 4
    assert ans.ans_layer_desc.n_symbols.offset == 48 and ans.ans_layer_desc.work_count.offset == 92
    assert ans.ans_layer_desc.piece_symbols.offset == 96


def test_table_bytes():
    for R in range(1, 15):
        b = ans.ans_table_bytes(R)
        assert b % 256 == 0 and b >= 16 + 1024 + 8 * (1 << R)
    with pytest.raises(ans.AnsError):
        ans.ans_table_bytes(15)


@pytest.mark.parametrize("layout", [ans.ANS_LAYOUT_INTERLEAVED, ans.ANS_LAYOUT_PRIVATE, ans.ANS_LAYOUT_QUADS])
@pytest.mark.parametrize("n,C,lanes,R,b", [(36864, 4096, 32, 12, 4), (5000, 1024, 64, 8, 3), (100_003, 16384, 128, 11, 6),
                                           (33, 64, 32, 6, 2), (70_000, 65536, 256, 14, 8), (4097, 4096, 32, 12, 1),
                                           (10_007, 1001, 32, 9, 4), (130, 130, 32, 5, 3),
                                           (50_000, 50_000, 96, 8, 3), (300_000, 300_000, 2048, 8, 4)])
def test_host_packer_equals_oracle_encoder(layout, n, C, lanes, R, b):
    spec = tiny_spec(n, bitwidth=b, pzp=0.7, table_log=R, chunk=C)
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, layout, lanes)
    counts = np.bincount(sym, minlength=256).astype(np.uint64)
    f = ans.ans_host_normalize_freqs(counts[:spec.alphabet], spec.alphabet, R)
    assert (f == f256).all()
    for threads in (1, 3):
        s, o, m = ans.ans_host_pack_layer(sym, f, spec.alphabet, R, C, lanes, layout, threads)
        assert s.size == P.stream.size and (s == P.stream).all()
        assert (o == P.sub_offsets).all() and (m == P.lane_meta).all()


@pytest.mark.parametrize("n,C,lanes,R,b", [(36864, 4096, 32, 12, 4), (5000, 1024, 64, 8, 3), (100_003, 16384, 128, 11, 6),
                                           (33, 128, 32, 6, 2), (70_000, 65536, 256, 14, 8), (4097, 4096, 32, 12, 1),
                                           (130, 512, 32, 5, 3), (300_000, 16384, 64, 8, 4), (0, 4096, 32, 8, 4)])
def test_host_packer_equals_oracle_encoder_strips(n, C, lanes, R, b):
    spec = tiny_spec(max(n, 1), bitwidth=b, pzp=0.9, table_log=R, chunk=C)
    sym = sg.draw_symbols(spec)
    T, P, f256 = oracle_pack_spec(spec, sym, oracle.STRIPS, lanes)
    sym = sym[:n]
    P = oracle.pack(T, sym, C, lanes // 32, oracle.STRIPS)
    for threads in (1, 3):
        s, o, m = ans.ans_host_pack_layer(sym, f256, spec.alphabet, R, C, lanes, ans.ANS_LAYOUT_STRIPS, threads)
        assert s.size == P.stream.size and (s == P.stream).all()
        assert (o == P.sub_offsets).all() and m.size == 0
    with pytest.raises(ans.AnsError):                      # chunk no multiple of 4 * lanes
        ans.ans_host_pack_layer(sym, f256, spec.alphabet, R, 1000, 32, ans.ANS_LAYOUT_STRIPS, 1)


@pytest.mark.parametrize("O,I,E,R,chunk_rows", [(8, 64, 9, 8, 0), (5, 32, 1, 6, 0), (16, 96, 49, 11, 4), (64, 128, 9, 8, 16)])
def test_host_packer_equals_oracle_encoder_channels(O, I, E, R, chunk_rows):
    """ANS_LAYOUT_CHANNELS: a stream per input channel of a tensor stored O x I x (H*W)."""
    spec = tiny_spec(O * I * E, bitwidth=4, pzp=0.85, table_log=R, chunk=O * I * E)
    sym = sg.draw_symbols(spec)
    C = chunk_rows * I * E if chunk_rows else sym.size
    T, _, f256 = oracle_pack_spec(spec, sym, oracle.STRIPS, 32, chunk=32)
    P = oracle.pack(T, sym, C, I // 32, oracle.CHANNELS, piece=E)
    for threads in (1, 3):
        s, o, m = ans.ans_host_pack_channels(sym, f256, spec.alphabet, R, C, I, E, threads)
        assert s.size == P.stream.size and (s == P.stream).all() and (o == P.sub_offsets).all() and m.size == 0
    with pytest.raises(ans.AnsError):                      # the layer is no multiple of lanes * piece
        ans.ans_host_pack_channels(sym[:-1], f256, spec.alphabet, R, C, I, E, 1)
    with pytest.raises(ans.AnsError):                      # the plain call cannot know the piece size
        ans.ans_host_pack_layer(sym, f256, spec.alphabet, R, C, I, ans.ANS_LAYOUT_CHANNELS, 1)


def test_plan_batch_counts_groups_of_four_sub_streams():
    arr = (ans.ans_layer_desc * 3)()
    for d, (n, C, lanes) in zip(arr, [(36864, 4096, 32), (0, 4096, 64), (10, 4, 128)]):
        d.n_symbols, d.chunk_symbols, d.lanes = n, C, lanes
    assert ans.ans_plan_batch(arr) == 3 + 0 + 3
    assert [d.work_begin for d in arr] == [0, 3, 3] and [d.work_count for d in arr] == [3, 0, 3]


def test_argument_errors_come_back_without_a_gpu():
    d = ans.ans_layer_desc()
    d.n_symbols, d.chunk_symbols, d.lanes, d.table_log, d.bitwidth = 100, 64, 32, 12, 4
    d.zero_point, d.scale = 7, 0.5
    with pytest.raises(ans.AnsError) as e:
        ans.ans_decode_dequant(d, 16)           # null table / stream pointers
    assert e.value.code == ans.ANS_ERR_INVALID_ARG
    d.lanes = 48
    with pytest.raises(ans.AnsError) as e:
        ans.ans_decode_dequant(d, 16)
    assert e.value.code in (ans.ANS_ERR_UNSUPPORTED, ans.ANS_ERR_INVALID_ARG)
    f = np.zeros((1, 256), dtype=np.uint32); f[0, 0] = 5
    with pytest.raises(ans.AnsError) as e:
        ans.ans_build_decode_tables(f, [2], [4], 256, 1 << 20)
    assert e.value.code == ans.ANS_ERR_BAD_FREQS
    f[0, 0] = 16
    with pytest.raises(ans.AnsError) as e:
        ans.ans_build_decode_tables(f, [2], [4], 256, 64)      # buffer too small
    assert e.value.code == ans.ANS_ERR_BUFFER_TOO_SMALL
    with pytest.raises(ans.AnsError):
        ans.ans_host_normalize_freqs(np.zeros(4, np.uint64), 4, 8)


def test_no_cpu_fallback_in_product_path():
    """The package must not import the oracle, and the oracle must not import the package."""
    pkg = os.path.join(ROOT, "paper_2406_06237_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                src = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in src.replace("no CPU path", ""), fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c")):
            assert "paper_2406_06237_b200" not in open(os.path.join(ROOT, "oracle", fn)).read()


def test_gemm_block_order_is_the_128_byte_swizzle_of_a_k_major_tile():
    """Rows of 64 bf16 = 128 bytes lie one after the other; inside row r the eight 16-byte pieces
    (8 elements each) are exchanged by r mod 8; elements keep their place inside a piece."""
    from paper_2406_06237_b200.runtime import gemm_block_order
    o = gemm_block_order()
    assert sorted(o.ravel().tolist()) == list(range(4096))
    r, c = np.meshgrid(np.arange(64), np.arange(64), indexing="ij")
    assert (o // 64 == r).all()
    assert ((o % 64) // 8 == ((c // 8) ^ (r % 8))).all()
    assert (o % 8 == c % 8).all()
