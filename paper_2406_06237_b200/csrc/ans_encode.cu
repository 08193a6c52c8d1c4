// The compress side on the device: histogram of a layer's symbols, the entropy of that histogram
// (the quantity the paper's training loss regularises, Section II-C, Eq. 3: the entropy H_W of
// the quantised weights), its normalisation to 2^R states, and the tANS encoder for the strips
// container (Section II-A: encoding follows a state transition of the automaton and appends the
// bits that label it).  Off the inference path; written so that its output is byte-identical
// with the host packer's.
#include "ans_common.cuh"

namespace ansb {

constexpr int kEncWarps = 8;                 // sub-streams (warps) per CTA of the encoder kernels
constexpr uint32_t kEncHeader = 64;          // bytes: 32 lanes x 16-bit length

// ---- histogram --------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) histogram_kernel(const uint8_t* __restrict__ sym, uint64_t n,
                                                       unsigned long long* __restrict__ counts) {
  __shared__ unsigned int h[256];
  h[threadIdx.x] = 0;
  __syncthreads();
  // 16 bytes per thread per trip where the address allows, single bytes at the ragged ends
  const uint64_t tid = uint64_t(blockIdx.x) * blockDim.x + threadIdx.x, nthreads = uint64_t(gridDim.x) * blockDim.x;
  const uint64_t head = min(n, (16 - (reinterpret_cast<uintptr_t>(sym) & 15)) & 15);
  const uint64_t vecs = (n - head) / 16;
  const uint4* v = reinterpret_cast<const uint4*>(sym + head);
  for (uint64_t i = tid; i < vecs; i += nthreads) {
    const uint4 q = __ldg(v + i);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      atomicAdd(&h[w[k] & 0xFF], 1u);
      atomicAdd(&h[(w[k] >> 8) & 0xFF], 1u);
      atomicAdd(&h[(w[k] >> 16) & 0xFF], 1u);
      atomicAdd(&h[w[k] >> 24], 1u);
    }
  }
  for (uint64_t i = tid; i < head; i += nthreads) atomicAdd(&h[sym[i]], 1u);
  for (uint64_t i = head + vecs * 16 + tid; i < n; i += nthreads) atomicAdd(&h[sym[i]], 1u);
  __syncthreads();
  if (h[threadIdx.x]) atomicAdd(&counts[threadIdx.x], static_cast<unsigned long long>(h[threadIdx.x]));
}

// ---- entropy of a histogram: -sum p log2 p, in bits per symbol, fp64 ------------------------------
__global__ void __launch_bounds__(256) entropy_kernel(const unsigned long long* __restrict__ counts, int alphabet,
                                                     double* __restrict__ out) {
  __shared__ double part[256];
  __shared__ unsigned long long total;
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int s = 0; s < alphabet; ++s) t += counts[s];
    total = t;
  }
  __syncthreads();
  double e = 0.0;
  const int s = threadIdx.x;
  if (s < alphabet && counts[s] && total) {
    const double p = static_cast<double>(counts[s]) / static_cast<double>(total);
    e = -p * log2(p);
  }
  part[s] = e;
  __syncthreads();
  if (threadIdx.x == 0) {                     // summed in symbol order, so that the result does not depend on timing
    double acc = 0.0;
    for (int k = 0; k < 256; ++k) acc += part[k];
    out[0] = acc;
    out[1] = acc * static_cast<double>(total);
  }
}

// ---- histogram -> 2^R states ------------------------------------------------------------------------
// Floor share, at least one state per symbol that occurs; a shortfall goes one state each to the
// largest remainders (ties to the lower symbol), an excess is taken one state at a time from the
// largest share (ties to the lower symbol).  Integers only.  status: 1 = cannot be normalised.
__global__ void __launch_bounds__(256) normalize_kernel(const unsigned long long* __restrict__ counts, int alphabet,
                                                       int R, uint32_t* __restrict__ freqs, uint32_t* __restrict__ status) {
  __shared__ unsigned long long rem[256];
  __shared__ uint32_t f[256];
  __shared__ unsigned long long total;
  __shared__ long long given;
  __shared__ int present;
  const int s = threadIdx.x;
  const unsigned long long L = 1ull << R;
  if (s == 0) {
    unsigned long long t = 0;
    int p = 0;
    for (int k = 0; k < alphabet; ++k) { t += counts[k]; p += counts[k] != 0; }
    total = t;
    present = p;
  }
  __syncthreads();
  const unsigned long long c = s < alphabet ? counts[s] : 0ull;
  if (total == 0 || static_cast<unsigned long long>(present) > L || total >= (1ull << 50)) {
    freqs[s] = 0;
    if (s == 0 && status) atomicOr(status, 1u);
    return;
  }
  uint32_t mine = 0;
  unsigned long long r = 0;
  if (c) {
    const unsigned long long scaled = c * L;        // < 2^64: counts below 2^50, L at most 2^14
    const unsigned long long q = scaled / total;
    r = scaled % total;
    mine = static_cast<uint32_t>(q ? q : 1ull);
  }
  f[s] = mine;
  rem[s] = r;
  __syncthreads();
  if (s == 0) {
    long long g = 0;
    for (int k = 0; k < 256; ++k) g += f[k];
    given = g;
  }
  __syncthreads();
  long long diff = static_cast<long long>(L) - given;
  if (diff > 0) {
    // rank among the symbols that occur, by remainder downwards, the lower symbol first on a tie
    int rank = 0;
    if (c)
      for (int t = 0; t < alphabet; ++t)
        if (counts[t] && (rem[t] > r || (rem[t] == r && t < s))) ++rank;
    if (c && rank < diff) mine += 1;
    f[s] = mine;
  }
  __syncthreads();
  if (diff < 0 && s == 0) {
    for (; diff < 0; ++diff) {
      int best = -1;
      for (int k = 0; k < alphabet; ++k)
        if (f[k] > 1 && (best < 0 || f[k] > f[best])) best = k;
      if (best < 0) { if (status) atomicOr(status, 1u); break; }
      f[best] -= 1;
    }
  }
  __syncthreads();
  freqs[s] = f[s];
}

// ---- encoder ----------------------------------------------------------------------------------------
struct EncArgs {
  const uint8_t* sym;
  uint64_t n;
  const uint8_t* blob;         // the layer's decode table, from ans_build_decode_tables
  int R;
  uint32_t chunk;
  uint32_t G;                  // lanes / 32
  uint32_t piece;              // channels container: symbols of a piece; 0: strips
  uint32_t* meta;              // quads container (not null): [n_sub][32] initial state | first word << 16
  uint64_t n_sub;
  uint32_t* lens;              // [n_sub][32] bit length of every lane's string
  unsigned long long* sizes;   // [n_sub] bytes of every sub-stream
  const unsigned long long* offsets;   // [n_sub + 1], for the writing pass
  uint8_t* out;
  uint64_t cap;
  uint32_t* status;
};

// per-CTA encoding tables in shared memory, rebuilt from the decode table: for symbol s and
// reduced state x_s in [f_s, 2 f_s) the state index whose decoding yields (s, x_s)
struct EncTables {
  uint32_t* f;        // [256]
  uint32_t* first;    // [256] states handed out before symbol s
  uint16_t* index;    // [2^R]
};

__device__ __forceinline__ void build_enc_tables(const uint8_t* blob, int R, EncTables T) {
  const uint32_t L = 1u << R;
  const uint32_t* g_freq = reinterpret_cast<const uint32_t*>(blob + kHeaderBytes);
  const uint32_t* g_single = reinterpret_cast<const uint32_t*>(blob + single_offset());
  for (uint32_t s = threadIdx.x; s < 256; s += blockDim.x) T.f[s] = g_freq[s];
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t acc = 0;
    for (int s = 0; s < 256; ++s) { T.first[s] = acc; acc += T.f[s]; }
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < L; i += blockDim.x) {
    const uint32_t e = g_single[i];
    const uint32_t s = entry_sym(e), nb = entry_nb(e);
    const uint32_t xs = (entry_newx(e) + L) >> nb;      // newX = (x_s << nb) - L
    T.index[T.first[s] + xs - T.f[s]] = static_cast<uint16_t>(i);
  }
  __syncthreads();
}

// One lane's encoding, backwards from state index 0 (so that its decoder ends there).  With WRITE
// the fields go to their places: the string ends at bit `end` of the sub-stream's body and is
// filled from the back; bit p of the body is bit 31 - p % 32 of its 32-bit little-endian word p / 32.
// strip: the lane's symbol t is strip[t * 32 + lane] (strips: `strip` is the sub-stream's first
// symbol), or, with piece = E > 0 (channels), strip[((t / E) * row + lane) * E + t % E], `strip`
// being the first symbol of the sub-stream's first lane and row = lanes per chunk.
template <bool WRITE>
__device__ __forceinline__ uint32_t encode_lane(const EncTables& T, int R, const uint8_t* strip, uint32_t count,
                                                uint32_t lane, uint32_t* body, uint64_t body_words, uint32_t end,
                                                uint32_t& state_out, bool& bad_symbol, uint32_t piece = 0,
                                                uint32_t row = 0, bool state_in_stream = true) {
  const uint32_t L = 1u << R;
  uint32_t x = L, bits = 0;
  uint32_t word = 0, acc = 0;            // WRITE: the word being filled and the bits collected for it
  bool have = false;
  auto put = [&](uint32_t val, uint32_t nb) {   // nb bits of val, most significant first, ending at bit `end`
    while (nb) {
      const uint32_t p = end - 1u, w = p >> 5, room = (p & 31u) + 1u;   // bits of word w at or before p
      const uint32_t take = nb < room ? nb : room;
      if (have && w != word) { if (word < body_words) atomicOr(body + word, acc); acc = 0; }
      word = w; have = true;
      acc |= (val & ((1u << take) - 1u)) << (31u - (p & 31u));
      val >>= take; nb -= take; end -= take;
    }
  };
  for (uint32_t t = count; t-- > 0;) {
    const uint32_t s = piece ? strip[(size_t(t / piece) * row + lane) * piece + t % piece] : strip[size_t(t) * 32u + lane];
    const uint32_t f = T.f[s];
    if (!f) { bad_symbol = true; break; }
    const uint32_t maxb = static_cast<uint32_t>(R) - (31u - static_cast<uint32_t>(__clz(f)));
    const uint32_t k = maxb - (x < (f << maxb) ? 1u : 0u);
    if (WRITE) put(x & ((1u << k) - 1u), k);
    bits += k;
    x = L + T.index[T.first[s] + (x >> k) - f];
  }
  state_out = x - L;
  if (WRITE && count) {
    if (state_in_stream) put(x - L, static_cast<uint32_t>(R));
    if (have && word < body_words) atomicOr(body + word, acc);
  }
  return count ? bits + (state_in_stream ? static_cast<uint32_t>(R) : 0u) : 0u;
}

template <bool WRITE>
__global__ void __launch_bounds__(kEncWarps * 32) encode_strips_kernel(const EncArgs a) {
  extern __shared__ __align__(16) uint8_t sm[];
  EncTables T;
  T.f = reinterpret_cast<uint32_t*>(sm);
  T.first = T.f + 256;
  T.index = reinterpret_cast<uint16_t*>(T.first + 256);
  build_enc_tables(a.blob, a.R, T);
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint64_t sub = uint64_t(blockIdx.x) * kEncWarps + warp;
  if (sub >= a.n_sub) return;
  const uint32_t S = a.chunk / (32u * a.G);
  const uint64_t chunk = sub / a.G;
  const uint32_t g = static_cast<uint32_t>(sub - chunk * a.G);
  const uint64_t c0 = chunk * a.chunk;
  const uint64_t nc = min(uint64_t(a.chunk), a.n - c0);
  const uint64_t sfirst = uint64_t(g) * 32u * S;
  const uint32_t ns = nc > sfirst ? static_cast<uint32_t>(min(nc - sfirst, uint64_t(32u) * S)) : 0u;
  uint32_t count = ns > lane ? (ns - lane + 31u) / 32u : 0u;
  const uint8_t* strip = a.sym + c0 + sfirst;
  const uint32_t row = 32u * a.G;
  if (a.piece) {               // channels: lanes 32 g .. 32 g + 31 of the chunk, every lane nc / W symbols in pieces
    count = static_cast<uint32_t>(nc / row);
    strip = a.sym + c0 + size_t(32u * g) * a.piece;
  }
  uint32_t state = 0;
  bool bad = false;
  if (a.meta) {
    // quads: the chunk is dealt in pieces of four to its lanes, the last piece may be short and the
    // lanes own different numbers of pieces; a lane's string is its fields alone, padded to a whole
    // 32-bit word, the strings one after the other, the state in the lane metadata
    const uint32_t lambda = 32u * g + lane;
    const uint64_t full = nc / 4u, rem = nc % 4u;
    count = 4u * static_cast<uint32_t>(full > lambda ? (full - lambda + row - 1u) / row : 0u) +
            ((rem && full % row == lambda) ? static_cast<uint32_t>(rem) : 0u);
    strip = a.sym + c0 + size_t(32u * g) * 4u;
    uint32_t len = WRITE ? a.lens[sub * 32 + lane] : 0u;
    if (!WRITE) {
      len = encode_lane<false>(T, a.R, strip, count, lane, nullptr, 0, 0, state, bad, 4u, row, false);
      a.lens[sub * 32 + lane] = len;
    }
    const uint32_t words = (len + 31u) >> 5;
    uint32_t incl = words;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= static_cast<uint32_t>(d)) incl += up;
    }
    const uint32_t word0 = incl - words, total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    if (!WRITE) {
      if (lane == 0) a.sizes[sub] = (uint64_t(total) * 4u + 15u) & ~15ull;
      if (word0 > 0xFFFFu) bad = true;
    } else {
      const unsigned long long off0 = a.offsets[sub], off1 = a.offsets[sub + 1];
      if (off1 <= a.cap) {
        uint32_t* body = reinterpret_cast<uint32_t*>(a.out + off0);
        encode_lane<true>(T, a.R, strip, count, lane, body, (off1 - off0) / 4, word0 * 32u + len, state, bad, 4u, row, false);
        a.meta[sub * 32 + lane] = state | (word0 << 16);
      } else if (lane == 0 && a.status) {
        atomicOr(a.status, 2u);
      }
    }
    if (bad && a.status) atomicOr(a.status, 4u);
    return;
  }
  if (!WRITE) {
    const uint32_t len = encode_lane<false>(T, a.R, strip, count, lane, nullptr, 0, 0, state, bad, a.piece, row);
    a.lens[sub * 32 + lane] = len;
    uint32_t total = len;
#pragma unroll
    for (int d = 16; d; d >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, d);
    if (lane == 0) a.sizes[sub] = (kEncHeader + ((total + 31u) / 32u) * 4u + 15u) & ~15ull;
    if (len > 0xFFFFu) bad = true;
  } else {
    const uint32_t len = a.lens[sub * 32 + lane];
    uint32_t incl = len;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= static_cast<uint32_t>(d)) incl += up;
    }
    const unsigned long long off0 = a.offsets[sub], off1 = a.offsets[sub + 1];
    if (off1 <= a.cap) {                        // (a stream that does not fit is flagged and left unwritten)
      uint8_t* dst = a.out + off0;
      reinterpret_cast<uint16_t*>(dst)[lane] = static_cast<uint16_t>(len);
      uint32_t* body = reinterpret_cast<uint32_t*>(dst + kEncHeader);
      const uint64_t body_words = (off1 - off0 - kEncHeader) / 4;
      encode_lane<true>(T, a.R, strip, count, lane, body, body_words, incl, state, bad, a.piece, row);
    } else if (lane == 0 && a.status) {
      atomicOr(a.status, 2u);
    }
  }
  if (bad && a.status) atomicOr(a.status, 4u);
}

// exclusive running sum of the sub-streams' sizes: offsets[0 .. n], one CTA
__global__ void __launch_bounds__(1024) offsets_kernel(const unsigned long long* __restrict__ sizes, uint64_t n,
                                                       unsigned long long* __restrict__ offsets) {
  __shared__ unsigned long long part[1024];
  __shared__ unsigned long long carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (uint64_t base = 0; base < n; base += 1024) {
    const uint64_t i = base + threadIdx.x;
    const unsigned long long v = i < n ? sizes[i] : 0ull;
    part[threadIdx.x] = v;
    __syncthreads();
    for (int d = 1; d < 1024; d <<= 1) {
      const unsigned long long add = threadIdx.x >= static_cast<unsigned>(d) ? part[threadIdx.x - d] : 0ull;
      __syncthreads();
      part[threadIdx.x] += add;
      __syncthreads();
    }
    if (i < n) offsets[i] = carry + part[threadIdx.x] - v;
    __syncthreads();
    if (threadIdx.x == 1023) carry += part[1023];
    __syncthreads();
  }
  if (threadIdx.x == 0) offsets[n] = carry;
}

static size_t up256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace ansb

using namespace ansb;

ANS_EXPORT int ans_histogram_device(const uint8_t* d_symbols, uint64_t n_symbols, uint64_t* d_counts, void* stream) {
  if (!d_counts || (n_symbols && !d_symbols)) return ANS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ANSB_CUDA(cudaMemsetAsync(d_counts, 0, 256 * sizeof(uint64_t), st));
  if (n_symbols == 0) return ANS_OK;
  const uint64_t want = (n_symbols / 16 + 255) / 256 / 8 + 1;
  const unsigned blocks = static_cast<unsigned>(want < 148 * 8 ? want : 148 * 8);
  histogram_kernel<<<blocks, 256, 0, st>>>(d_symbols, n_symbols, reinterpret_cast<unsigned long long*>(d_counts));
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}

ANS_EXPORT int ans_entropy_device(const uint64_t* d_counts, int alphabet, double* d_entropy_out, void* stream) {
  if (!d_counts || !d_entropy_out || alphabet < 1 || alphabet > ANS_MAX_ALPHABET) return ANS_ERR_INVALID_ARG;
  entropy_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const unsigned long long*>(d_counts), alphabet, d_entropy_out);
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}

ANS_EXPORT int ans_normalize_freqs_device(const uint64_t* d_counts, int alphabet, int table_log, uint32_t* d_freqs_out,
                                          uint32_t* d_status, void* stream) {
  if (!d_counts || !d_freqs_out || alphabet < 1 || alphabet > ANS_MAX_ALPHABET) return ANS_ERR_INVALID_ARG;
  if (table_log < 1 || table_log > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
  normalize_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const unsigned long long*>(d_counts), alphabet, table_log, d_freqs_out, d_status);
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}

ANS_EXPORT int ans_encode_scratch_bytes(uint64_t n_symbols, uint32_t chunk_symbols, uint32_t lanes, size_t* h_bytes_out) {
  if (!h_bytes_out || chunk_symbols == 0 || lanes == 0 || lanes % 32) return ANS_ERR_INVALID_ARG;
  if (n_symbols > (uint64_t(1) << 46)) return ANS_ERR_INVALID_ARG;
  const uint64_t chunks = n_symbols ? (n_symbols + chunk_symbols - 1) / chunk_symbols : 0;
  const uint64_t n_sub = chunks * (lanes / 32);
  *h_bytes_out = up256(n_sub * 128) + up256(n_sub * 8) + 256;
  return ANS_OK;
}

static int encode_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                         uint32_t chunk_symbols, uint32_t lanes, uint32_t piece, uint32_t* d_lane_meta_out, uint8_t* d_stream_out,
                         uint64_t stream_cap, uint64_t* d_sub_offsets_out, void* d_scratch,
                         size_t d_scratch_bytes, uint32_t* d_status, void* stream) {
  if (!d_sub_offsets_out || !d_status) return ANS_ERR_INVALID_ARG;
  if (table_log < 1 || table_log > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
  if (lanes < 32 || lanes > ANS_MAX_LANES || lanes % 32 || chunk_symbols == 0) return ANS_ERR_UNSUPPORTED;
  if (piece) {                                             // channels container
    if (piece > ANS_MAX_PIECE_SYMBOLS) return ANS_ERR_UNSUPPORTED;
    const uint64_t unit = uint64_t(lanes) * piece;
    if (chunk_symbols % unit || n_symbols % unit || chunk_symbols / lanes > ANS_MAX_CHANNEL_LANE_SYMBOLS)
      return ANS_ERR_UNSUPPORTED;
  } else if (!d_lane_meta_out && (chunk_symbols % lanes || chunk_symbols / lanes > ANS_MAX_STRIP_LANE_SYMBOLS)) {
    return ANS_ERR_UNSUPPORTED;
  }
  size_t need = 0;
  int rc = ans_encode_scratch_bytes(n_symbols, chunk_symbols, lanes, &need);
  if (rc != ANS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n_symbols == 0) {
    ANSB_CUDA(cudaMemsetAsync(d_sub_offsets_out, 0, sizeof(uint64_t), st));
    return ANS_OK;
  }
  if (!d_symbols || !d_table || !d_stream_out || !d_scratch) return ANS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_scratch) & 255) || (reinterpret_cast<uintptr_t>(d_stream_out) & 15) ||
      (reinterpret_cast<uintptr_t>(d_table) & 15))
    return ANS_ERR_INVALID_ARG;
  if (d_scratch_bytes < need) return ANS_ERR_BUFFER_TOO_SMALL;

  EncArgs a{};
  a.sym = d_symbols;
  a.n = n_symbols;
  a.blob = static_cast<const uint8_t*>(d_table);
  a.R = table_log;
  a.chunk = chunk_symbols;
  a.G = lanes / 32;
  a.piece = piece;
  a.meta = d_lane_meta_out;
  a.n_sub = ((n_symbols + chunk_symbols - 1) / chunk_symbols) * a.G;
  if (a.n_sub > 0x7FFFFFFFull * kEncWarps) return ANS_ERR_UNSUPPORTED;
  uint8_t* p = static_cast<uint8_t*>(d_scratch);
  a.lens = reinterpret_cast<uint32_t*>(p); p += up256(a.n_sub * 128);
  a.sizes = reinterpret_cast<unsigned long long*>(p);
  a.offsets = reinterpret_cast<const unsigned long long*>(d_sub_offsets_out);
  a.out = d_stream_out;
  a.cap = stream_cap;
  a.status = d_status;
  const size_t smem = 2048 + (size_t(2) << table_log);
  const unsigned blocks = static_cast<unsigned>((a.n_sub + kEncWarps - 1) / kEncWarps);
  // the strings are written by OR into zeroed words
  ANSB_CUDA(cudaMemsetAsync(d_stream_out, 0, stream_cap, st));
  encode_strips_kernel<false><<<blocks, kEncWarps * 32, smem, st>>>(a);
  ANSB_CUDA(cudaGetLastError());
  offsets_kernel<<<1, 1024, 0, st>>>(a.sizes, a.n_sub, reinterpret_cast<unsigned long long*>(d_sub_offsets_out));
  ANSB_CUDA(cudaGetLastError());
  encode_strips_kernel<true><<<blocks, kEncWarps * 32, smem, st>>>(a);
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}

ANS_EXPORT int ans_encode_layer_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                                       uint32_t chunk_symbols, uint32_t lanes, int layout, uint8_t* d_stream_out,
                                       uint64_t stream_cap, uint64_t* d_sub_offsets_out, void* d_scratch,
                                       size_t d_scratch_bytes, uint32_t* d_status, void* stream) {
  if (layout != ANS_LAYOUT_STRIPS) return ANS_ERR_UNSUPPORTED;
  return encode_device(d_symbols, n_symbols, d_table, table_log, chunk_symbols, lanes, 0, nullptr, d_stream_out, stream_cap,
                       d_sub_offsets_out, d_scratch, d_scratch_bytes, d_status, stream);
}

ANS_EXPORT int ans_encode_channels_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                                          uint32_t chunk_symbols, uint32_t lanes, uint32_t piece_symbols,
                                          uint8_t* d_stream_out, uint64_t stream_cap, uint64_t* d_sub_offsets_out,
                                          void* d_scratch, size_t d_scratch_bytes, uint32_t* d_status, void* stream) {
  if (piece_symbols < 1) return ANS_ERR_UNSUPPORTED;
  return encode_device(d_symbols, n_symbols, d_table, table_log, chunk_symbols, lanes, piece_symbols, nullptr, d_stream_out,
                       stream_cap, d_sub_offsets_out, d_scratch, d_scratch_bytes, d_status, stream);
}

ANS_EXPORT int ans_encode_quads_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                                       uint32_t chunk_symbols, uint32_t lanes, uint8_t* d_stream_out, uint64_t stream_cap,
                                       uint64_t* d_sub_offsets_out, uint32_t* d_lane_meta_out, void* d_scratch,
                                       size_t d_scratch_bytes, uint32_t* d_status, void* stream) {
  if (n_symbols && (!d_lane_meta_out || (reinterpret_cast<uintptr_t>(d_lane_meta_out) & 3))) return ANS_ERR_INVALID_ARG;
  static uint32_t dummy = 0;                               // (an empty layer writes no metadata)
  return encode_device(d_symbols, n_symbols, d_table, table_log, chunk_symbols, lanes, 0,
                       d_lane_meta_out ? d_lane_meta_out : &dummy, d_stream_out, stream_cap, d_sub_offsets_out, d_scratch,
                       d_scratch_bytes, d_status, stream);
}
