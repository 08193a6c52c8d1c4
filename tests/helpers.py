"""Shared by the CPU and GPU tests: oracle-side encoding of synthetic layers."""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np

import oracle
import synthgen as sg


def oracle_pack_spec(spec, symbols, layout, lanes=32, chunk=None, table_log=None):
    """Encode one layer with the ORACLE; returns (oracle.Table, oracle.Packed, freqs256)."""
    R = table_log or spec.table_log
    C = chunk or spec.chunk_symbols
    if symbols.size:
        f = oracle.normalize_freqs(oracle.histogram(symbols), spec.alphabet, R)
    else:                                  # an empty layer still needs some valid table
        f = np.zeros(spec.alphabet, dtype=np.uint32)
        f[0] = 1 << R
    T = oracle.Table(f, R)
    P = oracle.pack(T, symbols, C, lanes // 32, layout)
    f256 = np.zeros(256, dtype=np.uint32)
    f256[:spec.alphabet] = f
    return T, P, f256


def to_packed_layer(spec, P, f256, table_log=None, out_dtype=None):
    """Wrap the oracle's container in the library's host-side record (no re-encoding)."""
    import paper_2406_06237_b200 as ans
    from paper_2406_06237_b200.runtime import PackedLayer
    return PackedLayer(P.stream, P.sub_offsets, P.lane_meta, f256, spec.alphabet, P.n, P.chunk,
                       32 * P.groups, table_log or spec.table_log, spec.bitwidth, spec.zero_point,
                       spec.scale, ans.DTYPES[out_dtype or spec.out_dtype], P.layout, getattr(P, "piece", 1))


def oracle_expected(spec, T, P, threads=1, out_dtype=None):
    """Oracle decode + dequant: (symbols, output array in the layer's dtype bit patterns)."""
    sym, rc = oracle.unpack(T, P, threads=threads)
    assert rc == oracle.OK
    return sym, oracle.dequant(sym, spec.zero_point, spec.scale, out_dtype or spec.out_dtype, threads=threads)


def bits_view(t):
    """torch tensor -> numpy array of raw bit patterns."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.cpu().numpy().view(np.uint32)
    return t.cpu().numpy()


def expected_bits(a):
    return a.view(np.uint32) if a.dtype == np.float32 else a


def parallel_map(fn, items, threads=8):
    with ThreadPoolExecutor(threads) as ex:
        return list(ex.map(fn, items))


def tiny_spec(n, bitwidth=4, pzp=0.6, table_log=12, chunk=4096, out_dtype="bf16", seed=0, scale=0.02, index=0):
    A, zp = sg.alphabet_for_bits(bitwidth)
    return sg.LayerSpec(f"tiny{n}", (n,), bitwidth, A, zp, sg.theta_for_pzp(A, zp, pzp), scale,
                        table_log, chunk, out_dtype, sg.stream_key(seed, index))
