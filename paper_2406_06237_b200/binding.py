"""ctypes binding of libans_b200.so: the same entry points as include/ans_b200.h.

Argument marshalling only.  Every step of the decode path runs in the library's CUDA
kernels; nothing here computes, and there is no CPU fallback: if the shared library is
missing or cannot be loaded, importing this module's functions raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

ANS_OK = 0
ANS_ERR_INVALID_ARG, ANS_ERR_BAD_FREQS, ANS_ERR_UNSUPPORTED = -1, -2, -3
ANS_ERR_BUFFER_TOO_SMALL, ANS_ERR_CUDA, ANS_ERR_CORRUPT = -4, -5, -6
ANS_U8, ANS_F32, ANS_BF16 = 0, 1, 2
ANS_LAYOUT_INTERLEAVED, ANS_LAYOUT_PRIVATE, ANS_LAYOUT_QUADS, ANS_LAYOUT_STRIPS, ANS_LAYOUT_CHANNELS = 0, 1, 2, 3, 4
ANS_DESC_INPUTS_SETTLED, ANS_DESC_OUTPUT_IDLE = 1, 2
DTYPES = {"u8": ANS_U8, "f32": ANS_F32, "bf16": ANS_BF16}
ELEM_SIZE = {ANS_U8: 1, ANS_F32: 4, ANS_BF16: 2}

EXPORTS = [
    "ans_version", "ans_strerror", "ans_last_cuda_error", "ans_table_bytes", "ans_build_decode_tables",
    "ans_plan_batch", "ans_decode_layer", "ans_decode_dequant", "ans_decode_dequant_batch",
    "ans_read_status", "ans_host_scratch_bytes", "ans_decode_dequant_host",
    "ans_host_normalize_freqs", "ans_host_pack_bound", "ans_host_pack_layer", "ans_host_pack_channels",
    "ans_noalloc_max_bytes", "ans_decode_dequant_host_noalloc",
    "ans_histogram_device", "ans_entropy_device", "ans_normalize_freqs_device",
    "ans_encode_scratch_bytes", "ans_encode_layer_device", "ans_encode_channels_device", "ans_encode_quads_device",
    "ans_decode_gemm_bf16",
]


class ans_layer_desc(ctypes.Structure):
    _fields_ = [
        ("d_table", ctypes.c_void_p), ("d_stream", ctypes.c_void_p), ("d_sub_offsets", ctypes.c_void_p),
        ("d_lane_meta", ctypes.c_void_p), ("d_out", ctypes.c_void_p),
        ("stream_bytes", ctypes.c_uint64), ("n_symbols", ctypes.c_uint64), ("chunk_symbols", ctypes.c_uint32), ("lanes", ctypes.c_uint32),
        ("table_log", ctypes.c_int32), ("bitwidth", ctypes.c_int32), ("zero_point", ctypes.c_int32),
        ("scale", ctypes.c_float), ("out_dtype", ctypes.c_int32), ("layout", ctypes.c_int32),
        ("work_begin", ctypes.c_uint32), ("work_count", ctypes.c_uint32),
        ("piece_symbols", ctypes.c_uint32), ("flags", ctypes.c_uint32),
    ]


class AnsError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {ans_strerror(code)} ({code}; cuda {lib().ans_last_cuda_error()})")


_LIB = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Load libans_b200.so (built in-tree by paper_2406_06237_b200.build.build())."""
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: run paper_2406_06237_b200.build.build() "
                              "(needs nvcc); there is no fallback path")
        L = ctypes.CDLL(path)
        vp, i32, u32, u64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_size_t
        P = ctypes.POINTER
        L.ans_version.argtypes = []
        L.ans_strerror.argtypes = [i32]
        L.ans_strerror.restype = ctypes.c_char_p
        L.ans_last_cuda_error.argtypes = []
        L.ans_table_bytes.argtypes = [i32, P(sz)]
        L.ans_build_decode_tables.argtypes = [vp, vp, vp, i32, vp, sz, vp, vp]
        L.ans_plan_batch.argtypes = [P(ans_layer_desc), i32, P(u64)]
        L.ans_decode_layer.argtypes = [P(ans_layer_desc), vp, vp, vp]
        L.ans_decode_dequant.argtypes = [P(ans_layer_desc), vp, vp]
        L.ans_decode_dequant_batch.argtypes = [vp, P(ans_layer_desc), i32, vp, vp]
        L.ans_read_status.argtypes = [vp, vp, P(u32)]
        L.ans_host_scratch_bytes.argtypes = [P(ans_layer_desc), u64, P(sz)]
        L.ans_decode_dequant_host.argtypes = [P(ans_layer_desc), vp, u64, vp, vp, vp, vp, sz, vp]
        L.ans_noalloc_max_bytes.argtypes = [P(sz)]
        L.ans_decode_dequant_host_noalloc.argtypes = [P(ans_layer_desc), vp, i32, vp, u64, vp, vp, vp, vp]
        L.ans_host_normalize_freqs.argtypes = [vp, i32, i32, vp]
        L.ans_host_pack_bound.argtypes = [u64, u32, u32, i32, P(u64)]
        L.ans_host_pack_layer.argtypes = [vp, u64, vp, i32, i32, u32, u32, i32, vp, u64, P(u64), vp, vp, i32]
        L.ans_decode_gemm_bf16.argtypes = [P(ans_layer_desc), vp, i32, i32, i32, vp, vp, vp]
        L.ans_host_pack_channels.argtypes = [vp, u64, vp, i32, i32, u32, u32, u32, vp, u64, P(u64), vp, i32]
        L.ans_histogram_device.argtypes = [vp, u64, vp, vp]
        L.ans_entropy_device.argtypes = [vp, i32, vp, vp]
        L.ans_normalize_freqs_device.argtypes = [vp, i32, i32, vp, vp, vp]
        L.ans_encode_scratch_bytes.argtypes = [u64, u32, u32, P(sz)]
        L.ans_encode_layer_device.argtypes = [vp, u64, vp, i32, u32, u32, i32, vp, u64, vp, vp, sz, vp, vp]
        L.ans_encode_channels_device.argtypes = [vp, u64, vp, i32, u32, u32, u32, vp, u64, vp, vp, sz, vp, vp]
        L.ans_encode_quads_device.argtypes = [vp, u64, vp, i32, u32, u32, vp, u64, vp, vp, vp, sz, vp, vp]
        _LIB = L
    return _LIB


def _check(rc, where):
    if rc != ANS_OK:
        raise AnsError(rc, where)


def ans_version() -> int:
    return lib().ans_version()


def ans_strerror(code: int) -> str:
    return lib().ans_strerror(code).decode()


def ans_last_cuda_error() -> int:
    return lib().ans_last_cuda_error()


def ans_table_bytes(table_log: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().ans_table_bytes(table_log, ctypes.byref(out)), "ans_table_bytes")
    return out.value


def ans_build_decode_tables(norm_freqs: np.ndarray, alphabet, table_log, d_tables: int, d_tables_bytes: int,
                            stream: int = 0) -> np.ndarray:
    """norm_freqs [n_layers, 256] uint32 (host); returns the per-layer byte offsets (host)."""
    f = np.ascontiguousarray(norm_freqs, dtype=np.uint32).reshape(-1, 256)
    a = np.ascontiguousarray(alphabet, dtype=np.int32)
    r = np.ascontiguousarray(table_log, dtype=np.int32)
    n = f.shape[0]
    offs = np.zeros(max(n, 1), dtype=np.uint64)
    _check(lib().ans_build_decode_tables(f.ctypes.data, a.ctypes.data, r.ctypes.data, n, d_tables,
                                         d_tables_bytes, offs.ctypes.data, stream), "ans_build_decode_tables")
    return offs[:n]


def ans_plan_batch(h_descs) -> int:
    total = ctypes.c_uint64()
    _check(lib().ans_plan_batch(h_descs, len(h_descs), ctypes.byref(total)), "ans_plan_batch")
    return total.value


def ans_decode_layer(h_desc: ans_layer_desc, d_symbols_out: int, d_status: int, stream: int = 0) -> None:
    _check(lib().ans_decode_layer(ctypes.byref(h_desc), d_symbols_out, d_status, stream), "ans_decode_layer")


def ans_decode_dequant(h_desc: ans_layer_desc, d_status: int, stream: int = 0) -> None:
    _check(lib().ans_decode_dequant(ctypes.byref(h_desc), d_status, stream), "ans_decode_dequant")


def ans_decode_dequant_batch(d_descs: int, h_descs, d_status: int, stream: int = 0) -> None:
    _check(lib().ans_decode_dequant_batch(d_descs, h_descs, len(h_descs), d_status, stream),
           "ans_decode_dequant_batch")


def ans_read_status(d_status: int, stream: int = 0) -> int:
    """Waits for the stream; returns the status word (0 = sound) and clears it."""
    out = ctypes.c_uint32()
    rc = lib().ans_read_status(d_status, stream, ctypes.byref(out))
    if rc not in (ANS_OK, ANS_ERR_CORRUPT):
        raise AnsError(rc, "ans_read_status")
    return out.value


def ans_host_scratch_bytes(h_desc: ans_layer_desc, stream_bytes: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().ans_host_scratch_bytes(ctypes.byref(h_desc), stream_bytes, ctypes.byref(out)),
           "ans_host_scratch_bytes")
    return out.value


def ans_decode_dequant_host(h_desc, h_stream: np.ndarray, h_sub_offsets: np.ndarray, h_lane_meta: np.ndarray,
                            h_out: np.ndarray, d_scratch: int, d_scratch_bytes: int, stream: int = 0) -> int:
    """Returns ANS_OK or ANS_ERR_CORRUPT; raises on every other error."""
    rc = lib().ans_decode_dequant_host(ctypes.byref(h_desc), h_stream.ctypes.data, h_stream.nbytes,
                                       h_sub_offsets.ctypes.data, h_lane_meta.ctypes.data,
                                       h_out.ctypes.data, d_scratch, d_scratch_bytes, stream)
    if rc not in (ANS_OK, ANS_ERR_CORRUPT):
        raise AnsError(rc, "ans_decode_dequant_host")
    return rc


def ans_noalloc_max_bytes() -> int:
    out = ctypes.c_size_t()
    _check(lib().ans_noalloc_max_bytes(ctypes.byref(out)), "ans_noalloc_max_bytes")
    return out.value


def ans_decode_dequant_host_noalloc(h_desc, freqs: np.ndarray, alphabet: int, h_stream: np.ndarray,
                                    h_sub_offsets: np.ndarray, h_lane_meta: np.ndarray, h_out: np.ndarray,
                                    stream: int = 0) -> int:
    """Decode one layer from host buffers to a host buffer without any device allocation by the
    caller or the library (fixed working area inside the library).  Returns ANS_OK or
    ANS_ERR_CORRUPT; raises AnsError otherwise (ANS_ERR_BUFFER_TOO_SMALL if the layer does not
    fit the area)."""
    f = np.ascontiguousarray(freqs, dtype=np.uint32)
    assert f.size == 256
    rc = lib().ans_decode_dequant_host_noalloc(ctypes.byref(h_desc), f.ctypes.data, alphabet,
                                               h_stream.ctypes.data, h_stream.nbytes,
                                               h_sub_offsets.ctypes.data, h_lane_meta.ctypes.data,
                                               h_out.ctypes.data, stream)
    if rc not in (ANS_OK, ANS_ERR_CORRUPT):
        raise AnsError(rc, "ans_decode_dequant_host_noalloc")
    return rc


def ans_host_normalize_freqs(counts, alphabet: int, table_log: int) -> np.ndarray:
    c = np.ascontiguousarray(counts, dtype=np.uint64)
    f = np.zeros(256, dtype=np.uint32)
    _check(lib().ans_host_normalize_freqs(c.ctypes.data, alphabet, table_log, f.ctypes.data),
           "ans_host_normalize_freqs")
    return f


def ans_host_pack_layer(symbols: np.ndarray, freqs: np.ndarray, alphabet: int, table_log: int,
                        chunk_symbols: int, lanes: int, layout: int, n_threads: int = 0):
    """Returns (stream uint8[], sub_offsets uint64[n_sub+1], lane_meta [n_sub,32])."""
    sym = np.ascontiguousarray(symbols, dtype=np.uint8)
    f = np.ascontiguousarray(freqs, dtype=np.uint32)
    assert f.size == 256
    cap = ctypes.c_uint64()
    _check(lib().ans_host_pack_bound(sym.size, chunk_symbols, lanes, layout, ctypes.byref(cap)),
           "ans_host_pack_bound")
    n_chunks = (sym.size + chunk_symbols - 1) // chunk_symbols
    n_sub = n_chunks * (lanes // 32)
    stream = np.empty(cap.value, dtype=np.uint8)
    offs = np.zeros(n_sub + 1, dtype=np.uint64)
    meta = np.zeros((n_sub, 0 if layout == ANS_LAYOUT_STRIPS else 32),
                    dtype=np.uint16 if layout == ANS_LAYOUT_INTERLEAVED else np.uint32)
    used = ctypes.c_uint64()
    _check(lib().ans_host_pack_layer(sym.ctypes.data, sym.size, f.ctypes.data, alphabet, table_log,
                                     chunk_symbols, lanes, layout, stream.ctypes.data, cap.value,
                                     ctypes.byref(used), offs.ctypes.data, meta.ctypes.data, n_threads),
           "ans_host_pack_layer")
    return stream[:used.value].copy(), offs, meta


def ans_histogram_device(d_symbols: int, n_symbols: int, d_counts: int, stream: int = 0) -> None:
    _check(lib().ans_histogram_device(d_symbols, n_symbols, d_counts, stream), "ans_histogram_device")


def ans_entropy_device(d_counts: int, alphabet: int, d_entropy_out: int, stream: int = 0) -> None:
    _check(lib().ans_entropy_device(d_counts, alphabet, d_entropy_out, stream), "ans_entropy_device")


def ans_normalize_freqs_device(d_counts: int, alphabet: int, table_log: int, d_freqs_out: int, d_status: int = 0,
                               stream: int = 0) -> None:
    _check(lib().ans_normalize_freqs_device(d_counts, alphabet, table_log, d_freqs_out, d_status, stream),
           "ans_normalize_freqs_device")


def ans_encode_scratch_bytes(n_symbols: int, chunk_symbols: int, lanes: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().ans_encode_scratch_bytes(n_symbols, chunk_symbols, lanes, ctypes.byref(out)), "ans_encode_scratch_bytes")
    return out.value


def ans_host_pack_bound(n_symbols: int, chunk_symbols: int, lanes: int, layout: int) -> int:
    cap = ctypes.c_uint64()
    _check(lib().ans_host_pack_bound(n_symbols, chunk_symbols, lanes, layout, ctypes.byref(cap)), "ans_host_pack_bound")
    return cap.value


def ans_encode_layer_device(d_symbols: int, n_symbols: int, d_table: int, table_log: int, chunk_symbols: int,
                            lanes: int, layout: int, d_stream_out: int, stream_cap: int, d_sub_offsets_out: int,
                            d_scratch: int, d_scratch_bytes: int, d_status: int, stream: int = 0) -> None:
    _check(lib().ans_encode_layer_device(d_symbols, n_symbols, d_table, table_log, chunk_symbols, lanes, layout,
                                         d_stream_out, stream_cap, d_sub_offsets_out, d_scratch, d_scratch_bytes,
                                         d_status, stream), "ans_encode_layer_device")


def ans_encode_channels_device(d_symbols: int, n_symbols: int, d_table: int, table_log: int, chunk_symbols: int,
                               lanes: int, piece_symbols: int, d_stream_out: int, stream_cap: int,
                               d_sub_offsets_out: int, d_scratch: int, d_scratch_bytes: int, d_status: int,
                               stream: int = 0) -> None:
    _check(lib().ans_encode_channels_device(d_symbols, n_symbols, d_table, table_log, chunk_symbols, lanes,
                                            piece_symbols, d_stream_out, stream_cap, d_sub_offsets_out, d_scratch,
                                            d_scratch_bytes, d_status, stream), "ans_encode_channels_device")


def ans_encode_quads_device(d_symbols: int, n_symbols: int, d_table: int, table_log: int, chunk_symbols: int,
                            lanes: int, d_stream_out: int, stream_cap: int, d_sub_offsets_out: int,
                            d_lane_meta_out: int, d_scratch: int, d_scratch_bytes: int, d_status: int,
                            stream: int = 0) -> None:
    _check(lib().ans_encode_quads_device(d_symbols, n_symbols, d_table, table_log, chunk_symbols, lanes, d_stream_out,
                                         stream_cap, d_sub_offsets_out, d_lane_meta_out, d_scratch, d_scratch_bytes,
                                         d_status, stream), "ans_encode_quads_device")


def ans_host_pack_channels(symbols: np.ndarray, freqs: np.ndarray, alphabet: int, table_log: int,
                           chunk_symbols: int, lanes: int, piece_symbols: int, n_threads: int = 0):
    """ANS_LAYOUT_CHANNELS: returns (stream uint8[], sub_offsets uint64[n_sub+1], empty lane_meta)."""
    sym = np.ascontiguousarray(symbols, dtype=np.uint8)
    f = np.ascontiguousarray(freqs, dtype=np.uint32)
    assert f.size == 256
    cap = ans_host_pack_bound(sym.size, chunk_symbols, lanes, ANS_LAYOUT_CHANNELS)
    n_sub = -(-sym.size // chunk_symbols) * (lanes // 32)
    stream = np.empty(cap, dtype=np.uint8)
    offs = np.zeros(n_sub + 1, dtype=np.uint64)
    used = ctypes.c_uint64()
    _check(lib().ans_host_pack_channels(sym.ctypes.data, sym.size, f.ctypes.data, alphabet, table_log, chunk_symbols,
                                        lanes, piece_symbols, stream.ctypes.data, cap, ctypes.byref(used),
                                        offs.ctypes.data, n_threads), "ans_host_pack_channels")
    return stream[:used.value].copy(), offs, np.zeros((n_sub, 0), dtype=np.uint32)


def ans_decode_gemm_bf16(h_desc: ans_layer_desc, d_x: int, M: int, N: int, K: int, d_y: int, d_status: int,
                         stream: int = 0) -> None:
    _check(lib().ans_decode_gemm_bf16(ctypes.byref(h_desc), d_x, M, N, K, d_y, d_status, stream), "ans_decode_gemm_bf16")
