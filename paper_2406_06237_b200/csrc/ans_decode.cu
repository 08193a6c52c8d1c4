// tANS decode (+ fused zero-point dequantisation) kernels for sm_100a and their C entry points.
//
// Paper Section II-A / Fig. 2: state -> (symbol, nb_bits, newX); take nb_bits from the stream;
// next state = newX + bits.  Section III-B: one table per layer, a vector of states, one state per
// stream.  Here a warp holds 32 of those states (one per thread) and walks them together; the
// layer's table sits in shared memory; the decoded symbol goes through a 256-entry table of
// already dequantised values (Section II-B: w = scale * (q - zero_point)) on its way out.
//
// Work item = one sub-stream (32 lanes) = one warp.  A CTA owns a contiguous range of the work
// list, walks it kWarps items at a time and restages the table only when the layer changes.
#include <cuda_bf16.h>

#include "ans_common.cuh"

namespace ansb {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kTileRows = 64;          // private layout: rows of 32 symbols staged per warp
constexpr unsigned kFull = 0xFFFFFFFFu;

struct LaunchArgs {
  const ans_layer_desc* d_descs;   // device array, or nullptr when `one` is the only layer
  ans_layer_desc one;
  int n_layers;
  uint32_t total_work;
  uint32_t items_per_cta;
  uint32_t* d_status;
  uint8_t* d_symbols_override;     // ans_decode_layer: write symbols here instead of d_out
  uint32_t table_words;            // shared-memory words reserved for the table
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

// ---------------------------------------------------------------------------------------------
// Interleaved container: the warp's 32 lanes share one sequence of 16-bit units; a lane whose
// buffer holds fewer than 16 bits takes the next unit, its place found by ballot + popcount.
// ---------------------------------------------------------------------------------------------
template <int ES>
__device__ __forceinline__ uint32_t decode_interleaved(
    const uint32_t* __restrict__ tab, const uint32_t* __restrict__ vals,
    const uint16_t* __restrict__ units, uint32_t unit_cap, uint32_t state, uint32_t my_count,
    uint32_t rounds, typename ElemT<ES>::type* __restrict__ out, size_t row_stride, uint32_t lane) {
  using E = typename ElemT<ES>::type;
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t buf = 0, pos = 0;
  int cnt = 0;
  for (uint32_t r = 0; r < rounds; ++r) {
    const bool active = r < my_count;               // only the last round can have idle lanes
    const bool need = active && cnt < 16;
    const uint32_t b = __ballot_sync(kFull, need);
    if (need) {
      const uint32_t idx = pos + __popc(b & lt);
      const uint32_t u = idx < unit_cap ? static_cast<uint32_t>(__ldg(units + idx)) : 0u;
      buf |= u << cnt;
      cnt += 16;
    }
    pos += __popc(b);
    if (active) {
      const uint32_t e = tab[state];
      const uint32_t nb = entry_nb(e);
      const uint32_t v = buf & ((1u << nb) - 1u);
      buf >>= nb;
      cnt -= static_cast<int>(nb);
      state = entry_newx(e) + v;
      out[size_t(r) * row_stride] = static_cast<E>(vals[entry_sym(e)]);
    }
  }
  uint32_t bad = 0;
  if (state != 0) bad |= ANS_STATUS_BAD_FINAL_STATE;
  // the units taken, padded to 16 bytes, must be exactly the sub-stream's extent
  if (((pos * 2u + 15u) & ~15u) != unit_cap * 2u) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

// ---------------------------------------------------------------------------------------------
// Private container: every lane reads its own run of 32-bit words.  Look-ups go through the
// pre-walked table, so one look-up may stand for several symbols: `run` copies of the layer's
// dominant symbol followed by one more.  The warp stages kTileRows rows of output in shared
// memory, pre-filled with the dominant value, drops the other symbols into place and writes
// the rows out with 16-byte stores.
// ---------------------------------------------------------------------------------------------
template <int ES>
__device__ __forceinline__ void flush_rows(const uint8_t* tile, uint8_t* out_row0, size_t row_stride_bytes,
                                           uint32_t full_rows, uint32_t part_row_lanes, uint32_t lane) {
  constexpr uint32_t RB = 32u * ES;                 // bytes per row
  constexpr uint32_t PPR = RB / 16u;                // 16-byte pieces per row
  if ((reinterpret_cast<uintptr_t>(out_row0) & 15u) == 0 && (row_stride_bytes & 15u) == 0) {
    for (uint32_t idx = lane; idx < full_rows * PPR; idx += 32u) {
      const uint32_t row = idx / PPR, piece = idx % PPR;
      const uint4 v = *reinterpret_cast<const uint4*>(tile + size_t(idx) * 16u);
      *reinterpret_cast<uint4*>(out_row0 + size_t(row) * row_stride_bytes + piece * 16u) = v;
    }
  } else {
    using E = typename ElemT<ES>::type;
    for (uint32_t row = 0; row < full_rows; ++row)
      reinterpret_cast<E*>(out_row0 + size_t(row) * row_stride_bytes)[lane] =
          reinterpret_cast<const E*>(tile)[row * 32u + lane];
  }
  if (lane < part_row_lanes) {
    using E = typename ElemT<ES>::type;
    reinterpret_cast<E*>(out_row0 + size_t(full_rows) * row_stride_bytes)[lane] =
        reinterpret_cast<const E*>(tile)[full_rows * 32u + lane];
  }
}

template <int ES>
__device__ __forceinline__ uint32_t decode_private(
    const uint32_t* __restrict__ mtab, const uint32_t* __restrict__ g_single,
    const uint32_t* __restrict__ vals, uint32_t dom_val, const uint32_t* __restrict__ words,
    uint32_t wbeg, uint32_t wend, bool last_lane, uint32_t state, uint32_t my_count, uint32_t rows,
    uint32_t min_count, uint8_t* __restrict__ tile, uint8_t* __restrict__ out, size_t row_stride_bytes,
    uint32_t lane) {
  using E = typename ElemT<ES>::type;
  E* trow = reinterpret_cast<E*>(tile);
  auto load_word = [&](uint32_t i) -> uint32_t { return i < wend ? __ldg(words + i) : 0u; };
  uint32_t idx = wbeg;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1), w2 = load_word(idx + 2);
  idx += 3;
  uint32_t bitpos = 0;
  uint32_t t = 0;                 // next row this lane decodes
  bool pending = false;           // a decoded symbol waiting for the next window
  uint32_t pend_val = 0;

  uint32_t fill = dom_val;
  if (ES == 1) fill *= 0x01010101u;
  if (ES == 2) fill *= 0x00010001u;
  const uint4 fill4 = make_uint4(fill, fill, fill, fill);

  for (uint32_t r0 = 0; r0 < rows; r0 += kTileRows) {
    const uint32_t rend = min(r0 + kTileRows, rows);
    for (uint32_t i = lane; i < (kTileRows * 32u * ES) / 16u; i += 32u)
      reinterpret_cast<uint4*>(tile)[i] = fill4;
    __syncwarp();
    if (pending) {                                   // t - 1 is the row it belongs to
      trow[(t - 1 - r0) * 32u + lane] = static_cast<E>(pend_val);
      pending = false;
    }
    const uint32_t my_end = min(rend, my_count);
    while (t < my_end) {
      uint32_t e;
      if (my_count - t > kMaxRun) e = mtab[state];   // run + 1 <= 16 symbols are still owed
      else e = __ldg(g_single + state);              // tail: one symbol per look-up
      t += entry_run(e);
      const uint32_t val = vals[entry_sym(e)];
      if (t < rend) trow[(t - r0) * 32u + lane] = static_cast<E>(val);
      else { pending = true; pend_val = val; }
      t += 1;
      const uint32_t nb = entry_nb(e);
      const uint32_t x = __funnelshift_r(w0, w1, bitpos);
      state = entry_newx(e) + (x & ((1u << nb) - 1u));
      bitpos += nb;
      if (bitpos >= 32u) {
        w0 = w1; w1 = w2; w2 = load_word(idx); ++idx;
        bitpos -= 32u;
      }
    }
    __syncwarp();
    const uint32_t nrows = rend - r0;
    const bool has_part = (rend == rows) && (min_count < rows);   // last row is ragged
    const uint32_t full_rows = has_part ? nrows - 1 : nrows;
    uint32_t part_lanes = 0;
    if (has_part) part_lanes = __popc(__ballot_sync(kFull, my_count == rows));
    flush_rows<ES>(tile, out + size_t(r0) * row_stride_bytes, row_stride_bytes, full_rows, part_lanes, lane);
    __syncwarp();
  }
  uint32_t bad = 0;
  if (state != 0) bad |= ANS_STATUS_BAD_FINAL_STATE;
  // words used must be exactly the lane's run (the last lane's run is followed by < 16 pad bytes)
  const uint32_t bits = (idx - 3u - wbeg) * 32u + bitpos;
  const uint32_t need = (bits + 31u) / 32u;
  const uint32_t have = wend - wbeg;
  if (last_lane ? (need > have || have - need >= 4u) : (need != have)) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

// ---------------------------------------------------------------------------------------------
template <int LAYOUT>
__global__ void __launch_bounds__(kThreads) ans_decode_kernel(const LaunchArgs args) {
  extern __shared__ __align__(16) uint32_t smem[];
  uint32_t* tab = smem;                                   // [table_words]
  uint32_t* vals = smem + args.table_words;               // [256]
  uint8_t* tiles = reinterpret_cast<uint8_t*>(vals + 256);  // private: kWarps * kTileRows * 128 B
  __shared__ uint32_t s_dom;

  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  uint64_t cursor = uint64_t(blockIdx.x) * args.items_per_cta;
  const uint64_t cta_end = min(cursor + uint64_t(args.items_per_cta), uint64_t(args.total_work));
  if (cursor >= cta_end) return;

  // layer that holds `cursor`: last layer with work_begin <= cursor
  int l = 0;
  {
    int lo = 0, hi = args.n_layers;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (layer_at(args, mid).work_begin <= cursor) lo = mid; else hi = mid;
    }
    l = lo;
  }
  uint32_t bad = 0;
  for (; cursor < cta_end; ++l) {
    const ans_layer_desc& L = layer_at(args, l);
    const uint64_t lbeg = L.work_begin, lend = lbeg + L.work_count;
    if (lend <= cursor) continue;                         // empty layer
    const uint64_t stop = min(lend, cta_end);
    const int R = L.table_log;
    const uint8_t* blob = static_cast<const uint8_t*>(L.d_table);
    const TableHeader* hdr = reinterpret_cast<const TableHeader*>(blob);
    const uint32_t* g_single = reinterpret_cast<const uint32_t*>(blob + single_offset());
    const uint32_t* g_tab = LAYOUT == ANS_LAYOUT_PRIVATE
                                ? reinterpret_cast<const uint32_t*>(blob + multi_offset(R)) : g_single;
    const int dtype = args.d_symbols_override ? ANS_U8 : L.out_dtype;

    __syncthreads();                                      // previous layer's readers are done
    {
      const uint4* src = reinterpret_cast<const uint4*>(g_tab);
      uint4* dst = reinterpret_cast<uint4*>(tab);
      const uint32_t n16 = (1u << R) / 4u;
      for (uint32_t i = threadIdx.x; i < n16; i += kThreads) dst[i] = __ldg(src + i);
      if (R < 2 && threadIdx.x < (1u << R)) tab[threadIdx.x] = __ldg(g_tab + threadIdx.x);
      vals[threadIdx.x] = dequant_bits(static_cast<int>(threadIdx.x), L.zero_point, L.scale, dtype);
      if (threadIdx.x == 0) {
        s_dom = hdr->dominant;
        if (hdr->magic != kTableMagic || hdr->table_log != uint32_t(R) ||
            hdr->alphabet > (1u << L.bitwidth))
          bad |= ANS_STATUS_BAD_SYMBOL;
      }
    }
    __syncthreads();

    const uint32_t G = L.lanes / 32u, W = L.lanes, C = L.chunk_symbols;
    const size_t es = dtype == ANS_U8 ? 1 : dtype == ANS_F32 ? 4 : 2;
    uint8_t* out_base = args.d_symbols_override ? args.d_symbols_override : static_cast<uint8_t*>(L.d_out);
    for (uint64_t base = cursor; base < stop; base += kWarps) {
      const uint64_t item = base + warp;
      if (item >= stop) continue;
      const uint64_t sub = item - lbeg;
      const uint64_t chunk = sub / G;
      const uint32_t g = static_cast<uint32_t>(sub % G);
      const uint64_t c0 = chunk * C;
      const uint32_t nc = static_cast<uint32_t>(min(uint64_t(C), L.n_symbols - c0));
      const uint32_t lambda = 32u * g + lane;
      const uint32_t my_count = lane_symbols(nc, W, lambda);
      const uint32_t rows = lane_symbols(nc, W, 32u * g);          // lane 0 owns the most
      const uint32_t min_count = lane_symbols(nc, W, 32u * g + 31u);
      const uint64_t off0 = __ldg(L.d_sub_offsets + sub), off1 = __ldg(L.d_sub_offsets + sub + 1);
      uint32_t wbad = 0;
      uint64_t extent = off1 - off0;
      if (off1 < off0 || off1 > L.stream_bytes || (off0 & 15u)) {   // never read outside the stream
        extent = 0;
        wbad |= ANS_STATUS_BAD_LENGTH;
      }
      uint8_t* out = out_base + (c0 + lambda) * es;
      const size_t row_stride = W;
      if (LAYOUT == ANS_LAYOUT_INTERLEAVED) {
        const uint32_t state = __ldg(static_cast<const uint16_t*>(L.d_lane_meta) + sub * 32 + lane) &
                               ((1u << R) - 1u);
        const uint16_t* units = reinterpret_cast<const uint16_t*>(L.d_stream + (extent ? off0 : 0));
        const uint32_t cap = static_cast<uint32_t>(min(extent / 2, uint64_t(0xFFFFFFFFu)));
        if (es == 1)
          wbad |= decode_interleaved<1>(tab, vals, units, cap, state, my_count, rows, out, row_stride, lane);
        else if (es == 2)
          wbad |= decode_interleaved<2>(tab, vals, units, cap, state, my_count, rows,
                                       reinterpret_cast<uint16_t*>(out), row_stride, lane);
        else
          wbad |= decode_interleaved<4>(tab, vals, units, cap, state, my_count, rows,
                                       reinterpret_cast<uint32_t*>(out), row_stride, lane);
      } else {
        const uint32_t meta = __ldg(static_cast<const uint32_t*>(L.d_lane_meta) + sub * 32 + lane);
        const uint32_t state = meta & ((1u << R) - 1u);
        const uint32_t ext_words = static_cast<uint32_t>(min(extent / 4, uint64_t(0x7FFFFFFFu)));
        uint32_t wbeg = meta >> 16;
        uint32_t wend = __shfl_down_sync(kFull, wbeg, 1);
        if (lane == 31) wend = ext_words;
        if (wend > ext_words) { wend = ext_words; wbad |= ANS_STATUS_BAD_LENGTH; }
        if (wbeg > wend) { wbeg = wend; wbad |= ANS_STATUS_BAD_LENGTH; }
        const uint32_t* words = reinterpret_cast<const uint32_t*>(L.d_stream + (extent ? off0 : 0));
        uint8_t* tile = tiles + size_t(warp) * (kTileRows * 32u * es);
        uint8_t* out_row0 = out_base + (c0 + 32u * g) * es;     // row 0 of this sub-stream
        const uint32_t dom = s_dom < 256u ? vals[s_dom] : 0u;
        if (es == 1)
          wbad |= decode_private<1>(tab, g_single, vals, dom, words, wbeg, wend, lane == 31, state, my_count,
                                    rows, min_count, tile, out_row0, row_stride * es, lane);
        else if (es == 2)
          wbad |= decode_private<2>(tab, g_single, vals, dom, words, wbeg, wend, lane == 31, state, my_count,
                                    rows, min_count, tile, out_row0, row_stride * es, lane);
        else
          wbad |= decode_private<4>(tab, g_single, vals, dom, words, wbeg, wend, lane == 31, state, my_count,
                                    rows, min_count, tile, out_row0, row_stride * es, lane);
      }
      bad |= wbad;
    }
    cursor = stop;
  }
  bad = __reduce_or_sync(kFull, bad);
  if (lane == 0 && bad && args.d_status) atomicOr(args.d_status, bad);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static int launch(const ans_layer_desc* d_descs, const ans_layer_desc* h_descs, int n_layers,
                  uint8_t* d_symbols_override, uint32_t* d_status, cudaStream_t st) {
  int max_log = 1;
  uint64_t total = 0;
  const int layout = h_descs[0].layout;
  for (int l = 0; l < n_layers; ++l) {
    const int rc = validate_desc(h_descs[l], d_symbols_override == nullptr);
    if (rc != ANS_OK) return rc;
    if (h_descs[l].layout != layout) return ANS_ERR_UNSUPPORTED;
    if (h_descs[l].work_begin != total || h_descs[l].work_count != subs_of(h_descs[l]))
      return ANS_ERR_INVALID_ARG;                         // ans_plan_batch was not run on this array
    total += h_descs[l].work_count;
    if (h_descs[l].table_log > max_log) max_log = h_descs[l].table_log;
  }
  if (total == 0) return ANS_OK;
  if (total > 0xFFFFFFFFull) return ANS_ERR_UNSUPPORTED;

  LaunchArgs a{};
  a.d_descs = d_descs;
  if (!d_descs) a.one = h_descs[0];
  a.n_layers = n_layers;
  a.total_work = static_cast<uint32_t>(total);
  a.d_status = d_status;
  a.d_symbols_override = d_symbols_override;
  a.table_words = max_log < 2 ? 4u : (1u << max_log);
  size_t smem = (size_t(a.table_words) + 256) * 4;
  if (layout == ANS_LAYOUT_PRIVATE) smem += size_t(kWarps) * kTileRows * 32 * 4;

  const void* fn = layout == ANS_LAYOUT_PRIVATE
                       ? reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE>)
                       : reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_INTERLEAVED>);
  int dev = 0, sms = 0, per_sm = 0;
  ANSB_CUDA(cudaGetDevice(&dev));
  ANSB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ANSB_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  ANSB_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, smem));
  if (per_sm < 1) return ANS_ERR_UNSUPPORTED;
  const uint64_t want = (total + kWarps - 1) / kWarps;
  const uint64_t grid = want < uint64_t(sms) * per_sm ? want : uint64_t(sms) * per_sm;
  uint64_t ipc = (total + grid - 1) / grid;
  ipc = (ipc + kWarps - 1) / kWarps * kWarps;             // whole warps-per-CTA steps
  a.items_per_cta = static_cast<uint32_t>(ipc);
  const unsigned blocks = static_cast<unsigned>((total + ipc - 1) / ipc);
  if (layout == ANS_LAYOUT_PRIVATE)
    ans_decode_kernel<ANS_LAYOUT_PRIVATE><<<blocks, kThreads, smem, st>>>(a);
  else
    ans_decode_kernel<ANS_LAYOUT_INTERLEAVED><<<blocks, kThreads, smem, st>>>(a);
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}

}  // namespace ansb

using namespace ansb;

ANS_EXPORT int ans_plan_batch(ans_layer_desc* h_descs, int n_layers, uint64_t* h_total_work_out) {
  if (!h_descs || n_layers < 0) return ANS_ERR_INVALID_ARG;
  uint64_t total = 0;
  for (int l = 0; l < n_layers; ++l) {
    ans_layer_desc& d = h_descs[l];
    if (d.chunk_symbols == 0 || d.lanes == 0 || d.lanes % 32) return ANS_ERR_INVALID_ARG;
    const uint64_t n = subs_of(d);
    if (total + n > 0xFFFFFFFFull) return ANS_ERR_UNSUPPORTED;
    d.work_begin = static_cast<uint32_t>(total);
    d.work_count = static_cast<uint32_t>(n);
    total += n;
  }
  if (h_total_work_out) *h_total_work_out = total;
  return ANS_OK;
}

ANS_EXPORT int ans_decode_layer(const ans_layer_desc* h_desc, uint8_t* d_symbols_out, uint32_t* d_status,
                                void* stream) {
  if (!h_desc || !d_status) return ANS_ERR_INVALID_ARG;
  if (!d_symbols_out && h_desc->n_symbols) return ANS_ERR_INVALID_ARG;
  ans_layer_desc d = *h_desc;
  const int rc = ans_plan_batch(&d, 1, nullptr);
  if (rc != ANS_OK) return rc;
  if (d.n_symbols == 0) return validate_desc(d, false);
  return launch(nullptr, &d, 1, d_symbols_out, d_status, static_cast<cudaStream_t>(stream));
}

ANS_EXPORT int ans_decode_dequant(const ans_layer_desc* h_desc, uint32_t* d_status, void* stream) {
  if (!h_desc || !d_status) return ANS_ERR_INVALID_ARG;
  ans_layer_desc d = *h_desc;
  const int rc = ans_plan_batch(&d, 1, nullptr);
  if (rc != ANS_OK) return rc;
  return launch(nullptr, &d, 1, nullptr, d_status, static_cast<cudaStream_t>(stream));
}

ANS_EXPORT int ans_decode_dequant_batch(const ans_layer_desc* d_descs, const ans_layer_desc* h_descs,
                                        int n_layers, uint32_t* d_status, void* stream) {
  if (n_layers < 0 || !d_status) return ANS_ERR_INVALID_ARG;
  if (n_layers == 0) return ANS_OK;
  if (!d_descs || !h_descs) return ANS_ERR_INVALID_ARG;
  return launch(d_descs, h_descs, n_layers, nullptr, d_status, static_cast<cudaStream_t>(stream));
}
