// Small entry points: version, error text, status word, descriptor validation, and the
// end-to-end helper that takes HOST buffers.
#include <atomic>
#include <cmath>

#include "ans_common.cuh"

namespace ansb {

static std::atomic<int> g_last_cuda_error{0};
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error.store(static_cast<int>(e)); }

int validate_desc(const ans_layer_desc& d, bool need_out) {
  if (d.table_log < 1 || d.table_log > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
  if (d.lanes < 32 || d.lanes > ANS_MAX_LANES || d.lanes % 32) return ANS_ERR_UNSUPPORTED;
  if (!known_layout(d.layout)) return ANS_ERR_UNSUPPORTED;
  if (d.out_dtype != ANS_U8 && d.out_dtype != ANS_F32 && d.out_dtype != ANS_BF16) return ANS_ERR_UNSUPPORTED;
  if (d.chunk_symbols == 0) return ANS_ERR_INVALID_ARG;
  if (d.layout == ANS_LAYOUT_STRIPS &&
      (d.chunk_symbols % d.lanes || d.chunk_symbols / d.lanes > ANS_MAX_STRIP_LANE_SYMBOLS))
    return ANS_ERR_UNSUPPORTED;
  if (d.layout == ANS_LAYOUT_CHANNELS) {
    if (d.piece_symbols < 1 || d.piece_symbols > ANS_MAX_PIECE_SYMBOLS) return ANS_ERR_UNSUPPORTED;
    const uint64_t unit = uint64_t(d.lanes) * d.piece_symbols;
    if (d.chunk_symbols % unit || d.n_symbols % unit || d.chunk_symbols / d.lanes > ANS_MAX_CHANNEL_LANE_SYMBOLS)
      return ANS_ERR_UNSUPPORTED;
    if (d.piece_symbols * elem_size(d.out_dtype) > 128) return ANS_ERR_UNSUPPORTED;
  }
  if (d.bitwidth < 1 || d.bitwidth > 8) return ANS_ERR_INVALID_ARG;
  if (d.zero_point < 0 || d.zero_point >= (1 << d.bitwidth)) return ANS_ERR_INVALID_ARG;
  if (!std::isfinite(d.scale)) return ANS_ERR_INVALID_ARG;
  if (d.n_symbols == 0) return ANS_OK;
  if (!d.d_table || !d.d_stream || !d.d_sub_offsets) return ANS_ERR_INVALID_ARG;
  if (!d.d_lane_meta && lane_meta_size(d.layout)) return ANS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d.d_table) & 15) return ANS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d.d_stream) & 15) return ANS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d.d_sub_offsets) & 7) return ANS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d.d_lane_meta) & 3) return ANS_ERR_INVALID_ARG;
  if (need_out) {
    if (!d.d_out) return ANS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(d.d_out) & 15) return ANS_ERR_INVALID_ARG;
  }
  return ANS_OK;
}

}  // namespace ansb

using namespace ansb;

ANS_EXPORT int ans_version(void) { return 100; }

ANS_EXPORT int ans_last_cuda_error(void) { return g_last_cuda_error.load(); }

ANS_EXPORT const char* ans_strerror(int code) {
  switch (code) {
    case ANS_OK: return "ok";
    case ANS_ERR_INVALID_ARG: return "invalid argument";
    case ANS_ERR_BAD_FREQS: return "frequencies do not describe a table of 2^table_log states";
    case ANS_ERR_UNSUPPORTED: return "unsupported table_log, lanes, chunk size, layout or dtype";
    case ANS_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case ANS_ERR_CUDA: return "CUDA call failed (see ans_last_cuda_error)";
    case ANS_ERR_CORRUPT: return "a compressed stream did not decode soundly";
    default: return "unknown error code";
  }
}

ANS_EXPORT int ans_read_status(uint32_t* d_status, void* stream, uint32_t* h_status_out) {
  if (!d_status) return ANS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t h = 0;
  ANSB_CUDA(cudaMemcpyAsync(&h, d_status, sizeof(h), cudaMemcpyDeviceToHost, st));
  ANSB_CUDA(cudaMemsetAsync(d_status, 0, sizeof(h), st));
  ANSB_CUDA(cudaStreamSynchronize(st));
  if (h_status_out) *h_status_out = h;
  return h ? ANS_ERR_CORRUPT : ANS_OK;
}

// scratch layout: [status 256 B][stream][sub_offsets][lane_meta][out], each 256-byte aligned
static size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

ANS_EXPORT int ans_host_scratch_bytes(const ans_layer_desc* h_desc, uint64_t stream_bytes, size_t* h_bytes_out) {
  if (!h_desc || !h_bytes_out) return ANS_ERR_INVALID_ARG;
  if (h_desc->chunk_symbols == 0 || h_desc->lanes == 0 || h_desc->lanes % 32) return ANS_ERR_INVALID_ARG;
  // sizes that cannot be those of a real layer are refused before they can wrap a sum
  constexpr uint64_t kMaxBytes = uint64_t(1) << 46;
  if (h_desc->n_symbols > kMaxBytes / 4 || stream_bytes > kMaxBytes) return ANS_ERR_INVALID_ARG;
  const uint64_t n_sub = subs_of(*h_desc);
  if (n_sub > kMaxBytes / 128) return ANS_ERR_INVALID_ARG;
  const size_t meta = n_sub * 32 * lane_meta_size(h_desc->layout);
  *h_bytes_out = 256 + up256(stream_bytes) + up256((n_sub + 1) * 8) + up256(meta) +
                 up256(h_desc->n_symbols * elem_size(h_desc->out_dtype));
  return ANS_OK;
}

ANS_EXPORT int ans_decode_dequant_host(const ans_layer_desc* h_desc, const uint8_t* h_stream,
                                       uint64_t stream_bytes, const uint64_t* h_sub_offsets,
                                       const void* h_lane_meta, void* h_out, void* d_scratch,
                                       size_t d_scratch_bytes, void* stream) {
  if (!h_desc) return ANS_ERR_INVALID_ARG;
  size_t need = 0;
  int rc = ans_host_scratch_bytes(h_desc, stream_bytes, &need);
  if (rc != ANS_OK) return rc;
  if (h_desc->n_symbols == 0) return validate_desc(*h_desc, false);
  if (!h_stream || !h_sub_offsets || !h_out || !d_scratch) return ANS_ERR_INVALID_ARG;
  if (!h_lane_meta && lane_meta_size(h_desc->layout)) return ANS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_scratch) & 255) return ANS_ERR_INVALID_ARG;
  if (d_scratch_bytes < need) return ANS_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const uint64_t n_sub = subs_of(*h_desc);
  const size_t meta_bytes = n_sub * 32 * lane_meta_size(h_desc->layout);
  const size_t out_bytes = h_desc->n_symbols * elem_size(h_desc->out_dtype);
  uint8_t* p = static_cast<uint8_t*>(d_scratch);
  uint32_t* d_status = reinterpret_cast<uint32_t*>(p); p += 256;
  uint8_t* d_stream = p; p += up256(stream_bytes);
  uint64_t* d_offs = reinterpret_cast<uint64_t*>(p); p += up256((n_sub + 1) * 8);
  uint8_t* d_meta = p; p += up256(meta_bytes);
  uint8_t* d_out = p;

  ANSB_CUDA(cudaMemsetAsync(d_status, 0, 4, st));
  ANSB_CUDA(cudaMemcpyAsync(d_stream, h_stream, stream_bytes, cudaMemcpyHostToDevice, st));
  ANSB_CUDA(cudaMemcpyAsync(d_offs, h_sub_offsets, (n_sub + 1) * 8, cudaMemcpyHostToDevice, st));
  if (meta_bytes) ANSB_CUDA(cudaMemcpyAsync(d_meta, h_lane_meta, meta_bytes, cudaMemcpyHostToDevice, st));
  ans_layer_desc d = *h_desc;
  d.flags = 0;                                           // the inputs were copied in just now, on this stream
  d.stream_bytes = stream_bytes;
  d.d_stream = d_stream; d.d_sub_offsets = d_offs; d.d_lane_meta = d_meta; d.d_out = d_out;
  rc = ans_decode_dequant(&d, d_status, st);
  if (rc != ANS_OK) return rc;
  ANSB_CUDA(cudaMemcpyAsync(h_out, d_out, out_bytes, cudaMemcpyDeviceToHost, st));
  uint32_t h_status = 0;
  ANSB_CUDA(cudaMemcpyAsync(&h_status, d_status, 4, cudaMemcpyDeviceToHost, st));
  ANSB_CUDA(cudaStreamSynchronize(st));
  return h_status ? ANS_ERR_CORRUPT : ANS_OK;
}
