// Decode-table construction on the device (paper Section II-A: per state the decoded symbol,
// nb_bits and newX), plus the pre-walked table that folds chains of zero-bit transitions.
#include <vector>

#include "ans_common.cuh"

namespace ansb {

constexpr int kBuildThreads = 256;
constexpr int kLayersPerLaunch = 128;

struct BuildBatch {
  unsigned long long blob[kLayersPerLaunch];  // device address of each layer's blob
};

// One CTA per layer.  The blob already holds its header and the 256 frequencies (host copy).
// dynamic smem: single[L] u32 | slot[L] u8
__global__ void __launch_bounds__(kBuildThreads) build_tables_kernel(BuildBatch batch) {
  extern __shared__ __align__(16) uint32_t sm_single[];
  __shared__ uint32_t f[256];
  __shared__ uint32_t cum[257];
  __shared__ uint32_t dominant;

  uint8_t* blob = reinterpret_cast<uint8_t*>(batch.blob[blockIdx.x]);
  TableHeader* hdr = reinterpret_cast<TableHeader*>(blob);
  const int R = static_cast<int>(hdr->table_log);
  const uint32_t L = 1u << R;
  uint8_t* slot = reinterpret_cast<uint8_t*>(sm_single + L);
  const uint32_t* g_freq = reinterpret_cast<const uint32_t*>(blob + kHeaderBytes);
  uint32_t* g_single = reinterpret_cast<uint32_t*>(blob + single_offset());
  uint32_t* g_multi = reinterpret_cast<uint32_t*>(blob + multi_offset(R));
  const int tid = threadIdx.x;

  f[tid] = g_freq[tid];
  if (tid == 0) dominant = 0xFFFFFFFFu;
  __syncthreads();
  if (tid == 0) {
    uint32_t acc = 0;
    for (int s = 0; s < 256; ++s) { cum[s] = acc; acc += f[s]; }
    cum[256] = acc;
  }
  __syncthreads();

  // spread: the j-th state handed out (symbols ascending, f_s states each) sits at the
  // R-bit reversal of j
  for (uint32_t j = tid; j < L; j += kBuildThreads) {
    int lo = 0, hi = 256;            // largest s with cum[s] <= j
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cum[mid] <= j) lo = mid; else hi = mid;
    }
    slot[__brev(j) >> (32 - R)] = static_cast<uint8_t>(lo);
  }
  __syncthreads();

  // number each symbol's states upwards from f_s; thread s owns symbol s
  {
    const uint32_t s = tid;
    uint32_t x = f[s];
    if (x > 0) {
      if (2 * x > L) dominant = s;
      for (uint32_t i = 0; i < L; ++i) {
        if (slot[i] != s) continue;
        const uint32_t nb = static_cast<uint32_t>(R - (31 - __clz(x)));
        sm_single[i] = pack_entry(s, nb, 0, (x << nb) - L);
        ++x;
      }
    }
  }
  __syncthreads();

  for (uint32_t i = tid; i < L; i += kBuildThreads) {
    uint32_t cur = i, run = 0;
    uint32_t e = sm_single[cur];
    while (run < kMaxRun && entry_nb(e) == 0) {   // a zero-bit state has exactly one successor
      cur = entry_newx(e);
      e = sm_single[cur];
      ++run;
    }
    g_single[i] = sm_single[i];
    g_multi[i] = pack_entry(entry_sym(e), entry_nb(e), run, entry_newx(e));
  }
  if (tid == 0) hdr->dominant = dominant;
}

}  // namespace ansb

using namespace ansb;

ANS_EXPORT int ans_table_bytes(int table_log, size_t* h_bytes_out) {
  if (!h_bytes_out) return ANS_ERR_INVALID_ARG;
  if (table_log < 1 || table_log > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
  *h_bytes_out = table_blob_bytes(table_log);
  return ANS_OK;
}

ANS_EXPORT int ans_build_decode_tables(const uint32_t* h_norm_freqs, const int32_t* h_alphabet,
                                       const int32_t* h_table_log, int n_layers, void* d_tables,
                                       size_t d_tables_bytes, uint64_t* h_table_offsets_out,
                                       void* stream) {
  ApiRange range("ans_build_decode_tables");
  if (!h_norm_freqs || !h_alphabet || !h_table_log || !h_table_offsets_out || n_layers < 0)
    return ANS_ERR_INVALID_ARG;
  if (n_layers == 0) return ANS_OK;
  if (!d_tables || (reinterpret_cast<uintptr_t>(d_tables) & 255)) return ANS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  size_t off = 0;
  int max_log = 1;
  for (int l = 0; l < n_layers; ++l) {
    const int R = h_table_log[l], A = h_alphabet[l];
    if (R < 1 || R > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
    if (A < 1 || A > ANS_MAX_ALPHABET) return ANS_ERR_INVALID_ARG;
    uint64_t sum = 0;
    const uint32_t* f = h_norm_freqs + size_t(l) * 256;
    for (int s = 0; s < 256; ++s) {
      if (s >= A && f[s] != 0) return ANS_ERR_BAD_FREQS;
      sum += f[s];
    }
    if (sum != (1ull << R)) return ANS_ERR_BAD_FREQS;
    h_table_offsets_out[l] = off;
    off += table_blob_bytes(R);
    if (R > max_log) max_log = R;
  }
  if (off > d_tables_bytes) return ANS_ERR_BUFFER_TOO_SMALL;

  // header + frequencies of every layer go up first (pageable source: the runtime stages
  // it before the call returns), then one CTA per layer fills in the entries
  std::vector<uint32_t> head((kHeaderBytes + kFreqBytes) / 4);
  for (int l = 0; l < n_layers; ++l) {
    TableHeader h{kTableMagic, static_cast<uint32_t>(h_table_log[l]),
                  static_cast<uint32_t>(h_alphabet[l]), 0xFFFFFFFFu};
    memcpy(head.data(), &h, sizeof(h));
    memcpy(head.data() + kHeaderBytes / 4, h_norm_freqs + size_t(l) * 256, kFreqBytes);
    ANSB_CUDA(cudaMemcpyAsync(static_cast<uint8_t*>(d_tables) + h_table_offsets_out[l], head.data(),
                              kHeaderBytes + kFreqBytes, cudaMemcpyHostToDevice, st));
  }
  const size_t smem = (size_t(5) << max_log);
  ANSB_CUDA(cudaFuncSetAttribute(build_tables_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem)));
  for (int l0 = 0; l0 < n_layers; l0 += kLayersPerLaunch) {
    BuildBatch b;
    const int cnt = (n_layers - l0) < kLayersPerLaunch ? (n_layers - l0) : kLayersPerLaunch;
    for (int i = 0; i < cnt; ++i)
      b.blob[i] = reinterpret_cast<unsigned long long>(static_cast<uint8_t*>(d_tables) +
                                                       h_table_offsets_out[l0 + i]);
    build_tables_kernel<<<cnt, kBuildThreads, smem, st>>>(b);
    ANSB_CUDA(cudaGetLastError());
  }
  return ANS_OK;
}
