// Shared definitions of the CUDA library: device table layout, entry packing, error plumbing.
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include "ans_b200.h"

#define ANS_EXPORT extern "C" __attribute__((visibility("default")))

namespace ansb {

// ---- device table blob of one layer ------------------------------------------------------
// [ TableHeader (16 B) | freqs[256] u32 | single[L] u32 | multi[L] u32 ], padded to 256 B.
// single[i]: the paper's per-state triple (Section II-A): symbol, nb_bits, newX.
// multi[i] : the same walk with the leading zero-bit transitions folded in: `run` states
//            that read no bits (each emits the layer's dominant symbol) are crossed first,
//            then the entry describes the state reached.  One look-up therefore stands for
//            run + 1 decode steps of the plain automaton.
struct TableHeader {
  uint32_t magic;
  uint32_t table_log;
  uint32_t alphabet;
  uint32_t dominant;   // the only symbol that can own zero-bit states (f > L/2); 0xFFFFFFFF if none
};
constexpr uint32_t kTableMagic = 0x534E4174u;  // "tANS"
constexpr int kMaxRun = 15;

constexpr size_t kHeaderBytes = sizeof(TableHeader);
constexpr size_t kFreqBytes = 256 * sizeof(uint32_t);
__host__ __device__ constexpr size_t single_offset() { return kHeaderBytes + kFreqBytes; }
__host__ __device__ constexpr size_t multi_offset(int R) { return single_offset() + (size_t(4) << R); }
__host__ __device__ constexpr size_t table_blob_bytes(int R) {
  return (multi_offset(R) + (size_t(4) << R) + 255) & ~size_t(255);
}

// entry = sym | nb << 8 | run << 12 | newX << 16
__host__ __device__ inline uint32_t pack_entry(uint32_t sym, uint32_t nb, uint32_t run, uint32_t newx) {
  return sym | (nb << 8) | (run << 12) | (newx << 16);
}
__device__ __forceinline__ uint32_t entry_sym(uint32_t e) { return e & 0xFFu; }
__device__ __forceinline__ uint32_t entry_nb(uint32_t e) { return (e >> 8) & 0xFu; }
__device__ __forceinline__ uint32_t entry_run(uint32_t e) { return (e >> 12) & 0xFu; }
__device__ __forceinline__ uint32_t entry_newx(uint32_t e) { return e >> 16; }

// ---- error plumbing ----------------------------------------------------------------------
void set_last_cuda_error(cudaError_t e);
inline int cuda_fail(cudaError_t e) {
  set_last_cuda_error(e);
  return ANS_ERR_CUDA;
}
#define ANSB_CUDA(call)                                   \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return ::ansb::cuda_fail(e__); \
  } while (0)

// NVTX range around an API call (visible in a profiler's timeline; costs nothing without one)
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
  ApiRange(const ApiRange&) = delete;
  ApiRange& operator=(const ApiRange&) = delete;
};

int validate_desc(const ans_layer_desc& d, bool need_out);
inline uint32_t groups_of(const ans_layer_desc& d) { return d.lanes / 32u; }
inline uint64_t chunks_of(const ans_layer_desc& d) {
  return d.n_symbols ? (d.n_symbols + d.chunk_symbols - 1) / d.chunk_symbols : 0;
}
inline uint64_t subs_of(const ans_layer_desc& d) { return chunks_of(d) * groups_of(d); }
constexpr uint32_t kGranule = 4;   // sub-streams per work item of the batch plan
inline uint64_t granules_of(const ans_layer_desc& d) { return (subs_of(d) + kGranule - 1) / kGranule; }
inline size_t elem_size(int dtype) { return dtype == ANS_U8 ? 1 : dtype == ANS_F32 ? 4 : 2; }
// bytes of d_lane_meta per lane (the strips layout has no such array)
inline size_t lane_meta_size(int layout) {
  return layout == ANS_LAYOUT_INTERLEAVED ? 2 : (layout == ANS_LAYOUT_STRIPS || layout == ANS_LAYOUT_CHANNELS) ? 0 : 4;
}
inline bool known_layout(int layout) { return layout >= ANS_LAYOUT_INTERLEAVED && layout <= ANS_LAYOUT_CHANNELS; }

}  // namespace ansb
