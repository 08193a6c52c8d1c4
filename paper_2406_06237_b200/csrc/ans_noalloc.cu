// ans_decode_dequant_host_noalloc: the host-buffer decode call for callers that cannot allocate
// device memory.  Everything the call needs on the device (status word, the layer's table, the
// compressed stream, offsets, lane metadata and the decoded output) lives in one fixed array that
// is part of the library image.
#include "ans_common.cuh"

namespace ansb {

// Fixed device-side working area.  Every GPU on which the library is loaded carries it until the
// process exits.  8 MiB holds any single layer of the ResNet workloads (the largest, 2 359 296
// bf16 weights, needs 4.7 MB of output plus well under 1 MB of compressed data and table).
constexpr size_t kNoAllocBytes = size_t(8) << 20;
static __device__ __align__(256) unsigned char g_noalloc_area[kNoAllocBytes];

// Device address of the area, per device ordinal.  In host code the name g_noalloc_area is only a
// handle for the runtime, never something a kernel may dereference; cudaGetSymbolAddress turns it
// into the real address, once per device, with that device current.
constexpr int kMaxDevices = 64;
static unsigned char* g_area_addr[kMaxDevices];

static int noalloc_area(unsigned char** out) {
  int dev = 0;
  ANSB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ANS_ERR_UNSUPPORTED;
  if (!g_area_addr[dev]) {
    void* p = nullptr;
    ANSB_CUDA(cudaGetSymbolAddress(&p, g_noalloc_area));
    g_area_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_area_addr[dev];
  return ANS_OK;
}

static size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace ansb

using namespace ansb;

ANS_EXPORT int ans_noalloc_max_bytes(size_t* h_bytes_out) {
  if (!h_bytes_out) return ANS_ERR_INVALID_ARG;
  *h_bytes_out = kNoAllocBytes;
  return ANS_OK;
}

ANS_EXPORT int ans_decode_dequant_host_noalloc(const ans_layer_desc* h_desc, const uint32_t* h_norm_freqs,
                                               int alphabet, const uint8_t* h_stream, uint64_t stream_bytes,
                                               const uint64_t* h_sub_offsets, const void* h_lane_meta,
                                               void* h_out, void* stream) {
  if (!h_desc || !h_norm_freqs) return ANS_ERR_INVALID_ARG;
  if (h_desc->chunk_symbols == 0 || h_desc->lanes == 0 || h_desc->lanes % 32) return ANS_ERR_INVALID_ARG;
  if (h_desc->n_symbols == 0) return validate_desc(*h_desc, false);   // nothing to decode, but still a sound layer?
  if (!h_stream || !h_sub_offsets || !h_out) return ANS_ERR_INVALID_ARG;
  if (!h_lane_meta && lane_meta_size(h_desc->layout)) return ANS_ERR_INVALID_ARG;

  // lay the call out in the fixed area and refuse what does not fit.  Every term is bounded by
  // the area before it enters a sum, so that no size, however absurd, can wrap around and pass.
  size_t table_bytes = 0;
  int rc = ans_table_bytes(h_desc->table_log, &table_bytes);
  if (rc != ANS_OK) return rc;
  if (h_desc->n_symbols > kNoAllocBytes || stream_bytes > kNoAllocBytes) return ANS_ERR_BUFFER_TOO_SMALL;
  const uint64_t n_sub = subs_of(*h_desc);               // <= n_symbols * 64 groups: no overflow
  if (n_sub > kNoAllocBytes / 128) return ANS_ERR_BUFFER_TOO_SMALL;
  const size_t offs_bytes = (n_sub + 1) * 8;
  const size_t meta_bytes = n_sub * 32 * lane_meta_size(h_desc->layout);
  const size_t out_bytes = h_desc->n_symbols * elem_size(h_desc->out_dtype);
  const size_t need = 256 + up256(table_bytes) + up256(stream_bytes) + up256(offs_bytes) + up256(meta_bytes) +
                      up256(out_bytes);
  if (need > kNoAllocBytes) return ANS_ERR_BUFFER_TOO_SMALL;

  unsigned char* area = nullptr;
  rc = noalloc_area(&area);
  if (rc != ANS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* p = area;
  uint32_t* d_status = reinterpret_cast<uint32_t*>(p); p += 256;
  unsigned char* d_table = p; p += up256(table_bytes);
  unsigned char* d_stream = p; p += up256(stream_bytes);
  uint64_t* d_offs = reinterpret_cast<uint64_t*>(p); p += up256(offs_bytes);
  unsigned char* d_meta = p; p += up256(meta_bytes);
  unsigned char* d_out = p;

  // the area keeps whatever the previous call left: the status word must start at zero, the rest
  // is overwritten before it is read
  ANSB_CUDA(cudaMemsetAsync(d_status, 0, 4, st));
  const int32_t a32 = alphabet, r32 = h_desc->table_log;
  uint64_t table_off = 0;
  rc = ans_build_decode_tables(h_norm_freqs, &a32, &r32, 1, d_table, up256(table_bytes), &table_off, st);
  if (rc != ANS_OK) return rc;
  ANSB_CUDA(cudaMemcpyAsync(d_stream, h_stream, stream_bytes, cudaMemcpyHostToDevice, st));
  ANSB_CUDA(cudaMemcpyAsync(d_offs, h_sub_offsets, offs_bytes, cudaMemcpyHostToDevice, st));
  if (meta_bytes) ANSB_CUDA(cudaMemcpyAsync(d_meta, h_lane_meta, meta_bytes, cudaMemcpyHostToDevice, st));
  ans_layer_desc d = *h_desc;
  d.flags = 0;                                           // the inputs were copied in just now, on this stream
  d.d_table = d_table + table_off;
  d.d_stream = d_stream;
  d.stream_bytes = stream_bytes;
  d.d_sub_offsets = d_offs;
  d.d_lane_meta = d_meta;
  d.d_out = d_out;
  rc = ans_decode_dequant(&d, d_status, st);
  if (rc != ANS_OK) return rc;
  ANSB_CUDA(cudaMemcpyAsync(h_out, d_out, out_bytes, cudaMemcpyDeviceToHost, st));
  uint32_t h_status = 0;
  ANSB_CUDA(cudaMemcpyAsync(&h_status, d_status, 4, cudaMemcpyDeviceToHost, st));
  ANSB_CUDA(cudaStreamSynchronize(st));
  return h_status ? ANS_ERR_CORRUPT : ANS_OK;
}
