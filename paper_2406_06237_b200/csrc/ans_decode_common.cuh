// Pieces the four walks of ans_decode.cu share: launch arguments, work-list walking, bounded
// waits, shared-memory accessors.
#pragma once

#include <cuda_bf16.h>

#include "ans_common.cuh"

namespace ansb {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr uint32_t kStatusTimeout = ANS_STATUS_COPY_TIMEOUT;   // a bounded wait on an asynchronous copy ran out

constexpr int kParamLayers = 96;
constexpr int kLockstepMaxLog = 9;        // private container: largest table walked one symbol per look-up

struct LaunchArgs {
  const ans_layer_desc* d_descs;   // device array, or nullptr when `one` is the only layer
  ans_layer_desc one;
  int n_layers;
  uint32_t total_work;
  uint32_t items_per_cta;
  uint32_t* d_status;
  uint8_t* d_symbols_override;     // ans_decode_layer: write symbols here instead of d_out
  uint32_t table_words;            // shared-memory words reserved for the table
  uint32_t stage_bytes;            // private layout: per-warp staging buffer for compressed bytes
  uint32_t rep_log;                // log2 of the copies of a largest table in shared memory (1 .. 16 copies)
  uint32_t max_log;                // largest table_log of the launch
  uint32_t succ_bytes;             // private layout: shared-memory bytes of the successor table
  uint32_t ring_bytes;             // private layout: per-warp output ring (kRingRows rows of the widest dtype)
  uint32_t unit;                   // the value 1 (a run-time operand keeps a multiply-add a multiply-add)
  uint32_t n_begin;                // entries of layer_begin in use (0: search the descriptors instead)
  uint32_t early;                  // 1: every layer's inputs (and the descriptor array) were settled before the
                                   // preceding work on the stream began; 2: and that work does not touch the outputs
  // Where each layer's work items start in the numbering the CTAs walk.  When the launch's layers
  // all fit here, every layer's count is rounded up to the items a CTA takes at a time, so that
  // a CTA's rounds line up with the start of every layer it meets (the padding items are empty);
  // otherwise the numbering is the plan's (work_begin) and the descriptors are searched.
  uint32_t layer_begin[kParamLayers];
};

__device__ __forceinline__ const ans_layer_desc& layer_at(const LaunchArgs& a, int l) {
  return a.d_descs ? a.d_descs[l] : a.one;
}

// dequantised value of symbol s in the output's bit pattern (low bits of a u32)
__device__ __forceinline__ uint32_t dequant_bits(int s, int zero_point, float scale, int dtype) {
  if (dtype == ANS_U8) return static_cast<uint32_t>(s);
  const float w = __fmul_rn(__int2float_rn(s - zero_point), scale);
  if (dtype == ANS_F32) return __float_as_uint(w);
  return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(w)));
}

template <int ES> struct ElemT;
template <> struct ElemT<1> { using type = uint8_t; };
template <> struct ElemT<2> { using type = uint16_t; };
template <> struct ElemT<4> { using type = uint32_t; };

__device__ __forceinline__ uint32_t lane_symbols(uint32_t nc, uint32_t W, uint32_t lambda) {
  return nc > lambda ? (nc - lambda + W - 1) / W : 0u;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- work list walking shared by both kernels ----------------------------------------------
struct Item {
  uint64_t sub;        // sub-stream index inside the layer
  uint64_t c0;         // first symbol of the chunk
  uint32_t nc;         // symbols in the chunk
  uint32_t g;          // sub-stream inside the chunk
  uint64_t off0;       // byte offset of the sub-stream
  uint64_t extent;     // its bytes (0 if the offsets are unusable)
  uint32_t bad;
};

// off0 / off1: d_sub_offsets[sub] and [sub + 1], loaded by the caller (so that it can request
// them together with whatever else it needs from memory)
__device__ __forceinline__ Item make_item(const ans_layer_desc& L, uint64_t sub, uint64_t off0, uint64_t off1) {
  Item it;
  const uint32_t G = L.lanes / 32u;
  it.sub = sub;
  const uint64_t chunk = sub / G;
  it.g = static_cast<uint32_t>(sub % G);
  it.c0 = chunk * L.chunk_symbols;
  it.nc = static_cast<uint32_t>(min(uint64_t(L.chunk_symbols), L.n_symbols - it.c0));
  it.off0 = off0;
  it.extent = off1 - it.off0;
  it.bad = 0;
  // never read outside the stream; both ends on 16-byte boundaries, as the bulk copy and the
  // zero fill after the staged bytes need
  if (off1 < it.off0 || off1 > L.stream_bytes || ((it.off0 | off1) & 15u)) {
    it.extent = 0;
    it.off0 = 0;
    it.bad = ANS_STATUS_BAD_LENGTH;
  }
  return it;
}

// layer that holds work item `cursor`: the last layer with work_begin <= cursor
__device__ __forceinline__ int find_layer(const LaunchArgs& a, uint64_t cursor) {
  int lo = 0, hi = a.n_layers;
  if (a.n_begin == static_cast<uint32_t>(a.n_layers)) {   // every layer's start is in the parameters
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (a.layer_begin[mid] <= cursor) lo = mid; else hi = mid;
    }
    return lo;
  }
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (layer_at(a, mid).work_begin <= cursor) lo = mid; else hi = mid;
  }
  return lo;
}

constexpr uint32_t kFlushRows = 16;            // rows a walk handles (decodes, or writes out) at a time
constexpr uint32_t kStagePad = 176;            // readable bytes after the staged sub-stream
constexpr uint32_t kWaitSpins = 1u << 22;      // tries before a wait on a bulk copy gives up

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t spin = 0; spin < kWaitSpins; ++spin) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

// ---- shared-memory accesses by absolute (shared-window) address --------------------------------
__device__ __forceinline__ uint32_t lds_u32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
template <int ES>
__device__ __forceinline__ void sts_elem(uint32_t a, uint32_t v) {
  if (ES == 1) asm volatile("st.shared.u8 [%0], %1;" :: "r"(a), "r"(v) : "memory");
  if (ES == 2) asm volatile("st.shared.u16 [%0], %1;" :: "r"(a), "r"(v) : "memory");
  if (ES == 4) asm volatile("st.shared.u32 [%0], %1;" :: "r"(a), "r"(v) : "memory");
}

template <int ES>
__device__ __forceinline__ void stg_elem(uint8_t* p, uint32_t v) {
  if (ES == 1) *p = static_cast<uint8_t>(v);
  if (ES == 2) *reinterpret_cast<uint16_t*>(p) = static_cast<uint16_t>(v);
  if (ES == 4) *reinterpret_cast<uint32_t*>(p) = v;
}

}  // namespace ansb
