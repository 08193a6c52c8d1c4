"""Device-side set-up for a list of packed layers: torch supplies memory and the stream,
the library does the rest (tables, decode, dequantisation).  No arithmetic here."""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np
import torch

from . import binding as B


@dataclass
class PackedLayer:
    """Host-side container of one layer, as ans_host_pack_layer (or any conforming
    encoder) makes it, with the parameters a decode call needs."""
    stream: np.ndarray          # uint8
    sub_offsets: np.ndarray     # uint64 [n_sub + 1]
    lane_meta: np.ndarray       # uint16 / uint32 [n_sub, 32]
    freqs: np.ndarray           # uint32 [256]
    alphabet: int
    n_symbols: int
    chunk_symbols: int
    lanes: int
    table_log: int
    bitwidth: int
    zero_point: int
    scale: float
    out_dtype: int
    layout: int
    piece_symbols: int = 1      # ANS_LAYOUT_CHANNELS: symbols of a piece (H * W)

    def compressed_bytes(self) -> int:
        return int(self.stream.nbytes + self.sub_offsets.nbytes + self.lane_meta.nbytes)


def pack_layer(symbols: np.ndarray, alphabet: int, table_log: int, chunk_symbols: int, lanes: int,
               layout: int, bitwidth: int, zero_point: int, scale: float, out_dtype: int,
               n_threads: int = 0, piece_symbols: int = 1) -> PackedLayer:
    """Histogram, normalise and encode one layer with the library's host packer."""
    counts = np.bincount(symbols, minlength=256).astype(np.uint64)
    freqs = B.ans_host_normalize_freqs(counts[:alphabet], alphabet, table_log)
    if layout == B.ANS_LAYOUT_CHANNELS:
        stream, offs, meta = B.ans_host_pack_channels(symbols, freqs, alphabet, table_log, chunk_symbols, lanes,
                                                      piece_symbols, n_threads)
    else:
        stream, offs, meta = B.ans_host_pack_layer(symbols, freqs, alphabet, table_log, chunk_symbols, lanes,
                                                   layout, n_threads)
    return PackedLayer(stream, offs, meta, freqs, alphabet, int(symbols.size), chunk_symbols, lanes,
                       table_log, bitwidth, zero_point, float(scale), out_dtype, layout, piece_symbols)


def gemm_block_order() -> np.ndarray:
    """Where element (r, c) of a 64 x 64 block of W lies among the block's 4096 symbols for
    ans_decode_gemm_bf16 (the order in which the tensor core reads a 128-byte-swizzled K-major
    tile): index [r, c] -> symbol number."""
    r, c = np.meshgrid(np.arange(64), np.arange(64), indexing="ij")
    return (r // 8) * 512 + (r % 8) * 64 + ((c // 8) ^ (r % 8)) * 8 + c % 8


def pack_gemm_layer(w_symbols: np.ndarray, alphabet: int, table_log: int, bitwidth: int, zero_point: int,
                    scale: float, n_threads: int = 0) -> PackedLayer:
    """Encode W (N x K symbols, row n = output feature; N and K multiples of 64) the way
    ans_decode_gemm_bf16 reads it: blocks of 64 x 64 ordered [N / 64][K / 64], each block in
    gemm_block_order(), one sub-stream of the strips container per block."""
    n, k = w_symbols.shape
    if n % 64 or k % 64:
        raise ValueError("N and K must be multiples of 64")
    blocks = w_symbols.reshape(n // 64, 64, k // 64, 64).transpose(0, 2, 1, 3).reshape(n // 64, k // 64, 4096)
    ordered = np.empty_like(blocks)
    ordered[:, :, gemm_block_order().ravel()] = blocks
    return pack_layer(np.ascontiguousarray(ordered).ravel(), alphabet, table_log, 4096, 32, B.ANS_LAYOUT_STRIPS,
                      bitwidth, zero_point, scale, B.ANS_BF16, n_threads)


_TORCH_DTYPE = {B.ANS_U8: torch.uint8, B.ANS_F32: torch.float32, B.ANS_BF16: torch.bfloat16}


def _pad16(n: int) -> int:
    return (n + 15) // 16 * 16


class DeviceBatch:
    """All layers of a model resident on the GPU in compressed form, ready to decode in
    one launch.  With `n_out_sets` > 1 everything a launch touches (compressed arena, tables,
    outputs) exists that many times, so that a timing loop which rotates over the sets reads
    and writes memory that the launches in between have pushed out of L2."""

    def __init__(self, layers: list[PackedLayer], device="cuda:0", n_out_sets: int = 1,
                 inputs_settled: bool = False, output_idle: bool = False):
        """inputs_settled: set ANS_DESC_INPUTS_SETTLED on every layer.  The tables and the compressed
        bytes are put on the device (and the device synchronised) in this constructor, so the
        statement holds for every decode call made through this object afterwards.
        output_idle: also set ANS_DESC_OUTPUT_IDLE; the caller must then see to it that the work
        queued before a decode call does not touch that call's output set."""
        self.layers = layers
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise RuntimeError("DeviceBatch needs a CUDA device: there is no CPU path")
        torch.cuda.set_device(self.device)
        n = len(layers)
        # one arena for everything compressed: streams, offsets, lane metadata
        sizes = []
        for L in layers:
            sizes += [_pad16(L.stream.nbytes), _pad16(L.sub_offsets.nbytes), _pad16(L.lane_meta.nbytes)]
        starts = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
        arena_h = torch.empty(int(starts[-1]) + 16, dtype=torch.uint8, pin_memory=True)
        ah = arena_h.numpy()
        for i, L in enumerate(layers):
            for j, a in enumerate((L.stream, L.sub_offsets, L.lane_meta)):
                s = int(starts[3 * i + j])
                ah[s:s + a.nbytes] = a.reshape(-1).view(np.uint8)
        n_sets = max(1, n_out_sets)
        self.arena = arena_h.to(self.device, non_blocking=True)
        self.arenas = [self.arena] + [self.arena.clone() for _ in range(n_sets - 1)]
        self.arena_host = arena_h
        # tables
        tbytes = sum(B.ans_table_bytes(L.table_log) for L in layers)
        self.tables = torch.empty(max(tbytes, 256), dtype=torch.uint8, device=self.device)
        stream = torch.cuda.current_stream().cuda_stream
        if n:
            freqs = np.stack([L.freqs for L in layers])
            self.table_offsets = B.ans_build_decode_tables(
                freqs, [L.alphabet for L in layers], [L.table_log for L in layers],
                self.tables.data_ptr(), self.tables.numel(), stream)
        self.table_sets = [self.tables] + [self.tables.clone() for _ in range(n_sets - 1)]
        # outputs
        self.out_sets = []
        for _ in range(n_sets):
            self.out_sets.append([torch.empty(max(L.n_symbols, 1), dtype=_TORCH_DTYPE[L.out_dtype],
                                              device=self.device) for L in layers])
        self.status = torch.zeros(64, dtype=torch.int32, device=self.device)
        # descriptors: one host array + device copy per output set
        self.h_descs = []
        self.d_descs = []
        torch.cuda.synchronize(self.device)                 # tables are built before they are cloned above
        for k in range(1, n_sets):
            self.table_sets[k].copy_(self.tables)
        for k, outs in enumerate(self.out_sets):
            base = self.arenas[k].data_ptr()
            arr = (B.ans_layer_desc * max(n, 1))()
            for i, L in enumerate(layers):
                d = arr[i]
                d.d_table = self.table_sets[k].data_ptr() + int(self.table_offsets[i])
                d.d_stream = base + int(starts[3 * i])
                d.d_sub_offsets = base + int(starts[3 * i + 1])
                d.d_lane_meta = base + int(starts[3 * i + 2])
                d.d_out = outs[i].data_ptr()
                d.stream_bytes = L.stream.nbytes
                d.n_symbols, d.chunk_symbols, d.lanes = L.n_symbols, L.chunk_symbols, L.lanes
                d.table_log, d.bitwidth, d.zero_point, d.scale = L.table_log, L.bitwidth, L.zero_point, L.scale
                d.out_dtype, d.layout, d.piece_symbols = L.out_dtype, L.layout, L.piece_symbols
                d.flags = (B.ANS_DESC_INPUTS_SETTLED | (B.ANS_DESC_OUTPUT_IDLE if output_idle else 0)) if inputs_settled else 0
            self.total_work = B.ans_plan_batch(arr) if n else 0
            raw = torch.frombuffer(bytearray(bytes(arr)), dtype=torch.uint8)
            self.h_descs.append(arr)
            self.d_descs.append(raw.to(self.device))
        torch.cuda.synchronize(self.device)

    def set_flags(self, flags: int) -> None:
        """Write `flags` (ANS_DESC_* bits) into every layer descriptor, host and device copies."""
        torch.cuda.synchronize(self.device)
        for k, arr in enumerate(self.h_descs):
            for i in range(len(self.layers)):
                arr[i].flags = flags
            self.d_descs[k].copy_(torch.frombuffer(bytearray(bytes(arr)), dtype=torch.uint8))
        torch.cuda.synchronize(self.device)

    # -- sizes for reporting -------------------------------------------------------------
    def compressed_bytes(self) -> int:
        return sum(L.compressed_bytes() for L in self.layers)

    def table_bytes(self) -> int:
        return sum(B.ans_table_bytes(L.table_log) for L in self.layers)

    def output_bytes(self) -> int:
        return sum(L.n_symbols * B.ELEM_SIZE[L.out_dtype] for L in self.layers)

    def n_symbols(self) -> int:
        return sum(L.n_symbols for L in self.layers)

    def launches_per_decode(self) -> int:
        """Kernel launches one decode() makes: one, except that the strips kernel takes the
        layers 64 at a time (a group in which every layer is empty is not launched)."""
        if not any(L.n_symbols for L in self.layers):
            return 0
        if self.layers[0].layout in (B.ANS_LAYOUT_STRIPS, B.ANS_LAYOUT_CHANNELS):
            return sum(1 for g in range(0, len(self.layers), 64) if any(L.n_symbols for L in self.layers[g:g + 64]))
        return 1

    # -- calls ---------------------------------------------------------------------------
    def decode(self, out_set: int = 0, stream: int | None = None) -> None:
        """ONE launch for all layers (asynchronous)."""
        if not self.layers:
            return
        st = torch.cuda.current_stream().cuda_stream if stream is None else stream
        B.ans_decode_dequant_batch(self.d_descs[out_set].data_ptr(), self.h_descs[out_set],
                                   self.status.data_ptr(), st)

    def decode_per_layer(self, out_set: int = 0) -> None:
        st = torch.cuda.current_stream().cuda_stream
        for i in range(len(self.layers)):
            B.ans_decode_dequant(self.h_descs[out_set][i], self.status.data_ptr(), st)

    def decode_symbols(self, i: int) -> torch.Tensor:
        """ans_decode_layer on layer i: raw symbols."""
        st = torch.cuda.current_stream().cuda_stream
        out = torch.empty(max(self.layers[i].n_symbols, 1), dtype=torch.uint8, device=self.device)
        B.ans_decode_layer(self.h_descs[0][i], out.data_ptr(), self.status.data_ptr(), st)
        return out[:self.layers[i].n_symbols]

    def read_status(self) -> int:
        return B.ans_read_status(self.status.data_ptr(), torch.cuda.current_stream().cuda_stream)

    def output(self, i: int, out_set: int = 0) -> torch.Tensor:
        return self.out_sets[out_set][i][:self.layers[i].n_symbols]
