"""Python face of the CPU oracle (``ans_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the benchmark's CPU
baseline call this; the CUDA library never does, and this package imports
nothing from the CUDA library.  Argument marshalling only: every number comes
out of the C file, which follows the paper's decoder (Section II-A, Fig. 2),
its vector-of-states parallel form (Section III-B) and the zero-point uniform
quantiser (Section II-B).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

OK, ERR_ARG, ERR_FREQ, ERR_SPACE, ERR_CORRUPT = 0, -1, -2, -3, -4


class OracleError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"oracle: {what} failed with code {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile ans_oracle.c in-tree with gcc (no fast-math, no contraction)."""
    src = os.path.join(_HERE, "ans_oracle.c")
    out = os.path.join(_HERE, "libans_oracle.so")
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-ffp-contract=off", "-fno-fast-math",
                               "-shared", "-fPIC", "-o", out, src])
    return out


def _lib():
    global _LIB
    if _LIB is None:
        L = ctypes.CDLL(build())
        vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64
        L.anso_table_sizeof.restype = ctypes.c_size_t
        L.anso_build_table.argtypes = [vp, i32, i32, vp]
        L.anso_table_entry.argtypes = [vp, i32, vp, vp, vp]
        L.anso_encode_lane.argtypes = [vp, vp, i64, i64, vp, vp]
        L.anso_encode_plain.argtypes = [vp, vp, i64, vp, u64, vp]
        L.anso_decode_plain.argtypes = [vp, vp, u64, i32, i64, vp, vp, vp]
        L.anso_pack_interleaved.argtypes = [vp, vp, i64, i64, i32, vp, u64, vp, vp]
        L.anso_pack_interleaved.restype = i64
        L.anso_unpack_interleaved.argtypes = [vp, vp, vp, vp, i64, i64, i32, i64, i64, vp]
        L.anso_pack_private.argtypes = [vp, vp, i64, i64, i32, vp, u64, vp, vp]
        L.anso_pack_private.restype = i64
        L.anso_unpack_private.argtypes = [vp, vp, vp, vp, i64, i64, i32, i64, i64, vp]
        L.anso_pack_quads.argtypes = [vp, vp, i64, i64, i32, vp, u64, vp, vp]
        L.anso_pack_quads.restype = i64
        L.anso_unpack_quads.argtypes = [vp, vp, vp, vp, i64, i64, i32, i64, i64, vp]
        L.anso_pack_strips.argtypes = [vp, vp, i64, i64, i32, vp, u64, vp]
        L.anso_pack_strips.restype = i64
        L.anso_unpack_strips.argtypes = [vp, vp, vp, i64, i64, i32, i64, i64, vp]
        L.anso_pack_channels.argtypes = [vp, vp, i64, i64, i32, i32, vp, u64, vp]
        L.anso_pack_channels.restype = i64
        L.anso_unpack_channels.argtypes = [vp, vp, vp, i64, i64, i32, i32, i64, i64, vp]
        L.anso_dequant_f32.argtypes = [vp, i64, i32, ctypes.c_float, vp]
        L.anso_dequant_f32.restype = None
        L.anso_dequant_bf16.argtypes = [vp, i64, i32, ctypes.c_float, vp]
        L.anso_dequant_bf16.restype = None
        L.anso_normalize_freqs.argtypes = [vp, i32, i32, vp]
        L.anso_histogram.argtypes = [vp, i64, vp]
        L.anso_histogram.restype = None
        _LIB = L
    return _LIB


def _p(a: np.ndarray):
    return a.ctypes.data


INTERLEAVED, PRIVATE, QUADS, STRIPS, CHANNELS = 0, 1, 2, 3, 4


class Table:
    """Decode/encode table of one layer (Section II-A: symbol, nb_bits, newX per state)."""

    def __init__(self, freqs, table_log: int):
        lib = _lib()
        self.freqs = np.ascontiguousarray(freqs, dtype=np.uint32)
        self.A = int(self.freqs.size)
        self.R = int(table_log)
        self._buf = ctypes.create_string_buffer(lib.anso_table_sizeof())
        rc = lib.anso_build_table(_p(self.freqs), self.A, self.R, self._buf)
        if rc != OK:
            raise OracleError(rc, "build_table")

    @property
    def ptr(self):
        return ctypes.addressof(self._buf)

    def entries(self):
        """[(sym, nb, newX)] for state index 0 .. 2^R - 1."""
        lib = _lib()
        s, nb, nx = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        out = []
        for i in range(1 << self.R):
            lib.anso_table_entry(self.ptr, i, ctypes.byref(s), ctypes.byref(nb), ctypes.byref(nx))
            out.append((s.value, nb.value, nx.value))
        return out


def histogram(symbols: np.ndarray) -> np.ndarray:
    symbols = np.ascontiguousarray(symbols, dtype=np.uint8)
    c = np.zeros(256, dtype=np.uint64)
    _lib().anso_histogram(_p(symbols), symbols.size, _p(c))
    return c


def normalize_freqs(counts, alphabet: int, table_log: int) -> np.ndarray:
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    f = np.zeros(alphabet, dtype=np.uint32)
    rc = _lib().anso_normalize_freqs(_p(counts), alphabet, table_log, _p(f))
    if rc != OK:
        raise OracleError(rc, "normalize_freqs")
    return f


def encode_lane_fields(T: Table, msg):
    """Per-symbol transition labels (nb, value) in decode order and the initial state."""
    msg = np.ascontiguousarray(msg, dtype=np.uint8)
    nb = np.zeros(max(msg.size, 1), dtype=np.uint8)
    val = np.zeros(max(msg.size, 1), dtype=np.uint16)
    init = _lib().anso_encode_lane(T.ptr, _p(msg), msg.size, 1, _p(nb), _p(val))
    if init < 0:
        raise OracleError(init, "encode_lane")
    return init, nb[:msg.size], val[:msg.size]


def encode_plain(T: Table, msg):
    """One lane: (initial state, bit string as bytes, number of bits)."""
    msg = np.ascontiguousarray(msg, dtype=np.uint8)
    cap = (msg.size * T.R + 7) // 8 + 1
    out = np.zeros(cap, dtype=np.uint8)
    nbits = ctypes.c_uint64()
    init = _lib().anso_encode_plain(T.ptr, _p(msg), msg.size, _p(out), cap, ctypes.byref(nbits))
    if init < 0:
        raise OracleError(init, "encode_plain")
    return init, out[:(nbits.value + 7) // 8].copy(), nbits.value


def decode_plain(T: Table, data, init: int, n: int, want_trace: bool = False):
    data = np.ascontiguousarray(data, dtype=np.uint8)
    out = np.zeros(max(n, 1), dtype=np.uint8)
    trace = np.zeros(max(n, 1), dtype=np.int32)
    used = ctypes.c_uint64()
    rc = _lib().anso_decode_plain(T.ptr, _p(data), data.size, init, n, _p(out), _p(trace), ctypes.byref(used))
    res = (out[:n], rc, used.value)
    return res + (trace[:n],) if want_trace else res


class Packed:
    """One layer in a container: stream bytes, per-sub-stream offsets, per-lane metadata."""

    def __init__(self, layout, stream, sub_offsets, lane_meta, n, chunk, groups, piece=1):
        self.layout, self.stream, self.sub_offsets, self.lane_meta = layout, stream, sub_offsets, lane_meta
        self.n, self.chunk, self.groups, self.piece = n, chunk, groups, piece

    @property
    def n_chunks(self):
        return (self.n + self.chunk - 1) // self.chunk

    @property
    def n_sub(self):
        return self.n_chunks * self.groups

    def total_bytes(self):
        """Everything a decoder must read: stream, offsets and lane metadata."""
        return int(self.stream.nbytes + self.sub_offsets.nbytes + self.lane_meta.nbytes)


def pack(T: Table, symbols, chunk: int, groups: int = 1, layout: int = INTERLEAVED, piece: int = 1) -> Packed:
    symbols = np.ascontiguousarray(symbols, dtype=np.uint8)
    n = symbols.size
    n_chunks = (n + chunk - 1) // chunk
    n_sub = n_chunks * groups
    cap = n * 2 + n_sub * (32 * 8 + 32) + 64
    if layout == STRIPS:                   # per sub-stream: lengths, 32 states, worst-case fields, padding
        if chunk % (32 * groups):
            raise OracleError(ERR_ARG, "pack (strips: chunk must be a multiple of the lanes)")
        cap = n_sub * (64 + 4 * (chunk // (32 * groups) + 1) * T.R + 36) + 64
    stream = np.zeros(cap, dtype=np.uint8)
    offs = np.zeros(n_sub + 1, dtype=np.uint64)
    lib = _lib()
    if layout == CHANNELS:
        cap = n_sub * (64 + 4 * (chunk // (32 * groups) + 1) * T.R + 36) + 64
        stream = np.zeros(cap, dtype=np.uint8)
        meta = np.zeros((n_sub, 0), dtype=np.uint32)
        total = lib.anso_pack_channels(T.ptr, _p(symbols), n, chunk, groups, piece, _p(stream), cap, _p(offs))
    elif layout == STRIPS:
        meta = np.zeros((n_sub, 0), dtype=np.uint32)       # this container has no per-lane array
        total = lib.anso_pack_strips(T.ptr, _p(symbols), n, chunk, groups, _p(stream), cap, _p(offs))
    elif layout == INTERLEAVED:
        meta = np.zeros((n_sub, 32), dtype=np.uint16)
        total = lib.anso_pack_interleaved(T.ptr, _p(symbols), n, chunk, groups, _p(stream), cap, _p(offs), _p(meta))
    else:
        meta = np.zeros((n_sub, 32), dtype=np.uint32)
        fn = lib.anso_pack_private if layout == PRIVATE else lib.anso_pack_quads
        total = fn(T.ptr, _p(symbols), n, chunk, groups, _p(stream), cap, _p(offs), _p(meta))
    if total < 0:
        raise OracleError(total, "pack")
    return Packed(layout, stream[:total].copy(), offs, meta, n, chunk, groups, piece)


def unpack(T: Table, P: Packed, threads: int = 1, chunk_range=None):
    """Decode a packed layer to symbols.  Returns (symbols, rc)."""
    out = np.zeros(max(P.n, 1), dtype=np.uint8)
    lib = _lib()
    lo, hi = chunk_range if chunk_range is not None else (0, P.n_chunks)
    if P.layout == CHANNELS:
        def work(rng):
            return lib.anso_unpack_channels(T.ptr, _p(P.stream), _p(P.sub_offsets), P.n, P.chunk, P.groups, P.piece,
                                            rng[0], rng[1], _p(out))
    elif P.layout == STRIPS:
        def work(rng):
            return lib.anso_unpack_strips(T.ptr, _p(P.stream), _p(P.sub_offsets), P.n, P.chunk, P.groups,
                                            rng[0], rng[1], _p(out))
    else:
        fn = {INTERLEAVED: lib.anso_unpack_interleaved, PRIVATE: lib.anso_unpack_private,
              QUADS: lib.anso_unpack_quads}[P.layout]

        def work(rng):
            return fn(T.ptr, _p(P.stream), _p(P.sub_offsets), _p(P.lane_meta), P.n, P.chunk, P.groups,
                      rng[0], rng[1], _p(out))

    if threads <= 1 or hi - lo <= 1:
        rc = work((lo, hi))
    else:
        step = (hi - lo + threads - 1) // threads
        ranges = [(a, min(a + step, hi)) for a in range(lo, hi, step)]
        with ThreadPoolExecutor(threads) as ex:
            rcs = list(ex.map(work, ranges))
        rc = min(rcs)
    return out[:P.n], rc


def dequant(symbols, zero_point: int, scale: float, dtype: str, threads: int = 1):
    """w = (q - zero_point) * scale in fp32; 'bf16' returns the uint16 bit patterns."""
    symbols = np.ascontiguousarray(symbols, dtype=np.uint8)
    n = symbols.size
    lib = _lib()
    if dtype == "u8":
        return symbols.copy()
    if dtype == "f32":
        out = np.empty(n, dtype=np.float32)
        fn = lib.anso_dequant_f32
    elif dtype == "bf16":
        out = np.empty(n, dtype=np.uint16)
        fn = lib.anso_dequant_bf16
    else:
        raise ValueError(dtype)

    def work(rng):
        a, b = rng
        fn(_p(symbols) + a, b - a, zero_point, scale, _p(out) + a * out.itemsize)

    if threads <= 1 or n < (1 << 16):
        work((0, n))
    else:
        step = (n + threads - 1) // threads
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, [(a, min(a + step, n)) for a in range(0, n, step)]))
    return out
