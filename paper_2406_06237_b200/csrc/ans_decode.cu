// tANS decode (+ fused zero-point dequantisation) kernels for sm_100a and their C entry points.
//
// Paper Section II-A / Fig. 2: state -> (symbol, nb_bits, newX); take nb_bits from the stream;
// next state = newX + bits.  Section III-B: one table per layer, a vector of states, one state per
// stream.  Here a warp holds 32 of those states (one per thread) and walks them together; the
// layer's table sits in shared memory, its entries already carrying the dequantised value
// (Section II-B: w = scale * (q - zero_point)) in the output's bit pattern.
//
// One sub-stream (32 lanes) is decoded by one warp.  The work list counts granules of up to
// kGranule consecutive sub-streams of a layer; a CTA owns a contiguous range of granules, walks
// it one sub-stream per warp at a time and restages the table only when the layer changes.
// Four walks share that skeleton: the interleaved container; the private container through its
// pre-walked entries (a look-up may emit a run of the dominant symbol plus one symbol) or one
// symbol per look-up with the lanes in lockstep; the quads container (always lockstep).
#include <cuda_bf16.h>

#include "ans_common.cuh"

namespace ansb {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr uint32_t kStatusTimeout = 8u;   // a bounded wait on an asynchronous copy ran out

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
  if (off1 < it.off0 || off1 > L.stream_bytes || (it.off0 & 15u)) {   // never read outside the stream
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

// =============================================================================================
// Private container: every lane reads its own run of 32-bit words.
//
// Look-ups go through the pre-walked table, so one look-up can stand for several symbols: `run`
// copies of the layer's dominant symbol (its zero-bit states, Section II-A's unlabeled
// transitions) followed by one more symbol.  Lanes therefore drift apart; each warp keeps a ring
// of output rows in shared memory, pre-filled with the dominant value, into which lanes drop
// the other symbols.  A quarter of the ring is written out (16-byte stores) as soon as the
// slowest lane has left it.  The sub-stream's compressed bytes are brought into shared memory by
// one bulk asynchronous copy per warp, so a lane's refill is a shared-memory load.
// =============================================================================================
constexpr uint32_t kRingRows = 64;             // rows (of 32 symbols) in a warp's output ring
constexpr uint32_t kFlushRows = 16;            // rows written out at a time
constexpr uint32_t kStagePad = 176;            // readable bytes after the staged sub-stream
constexpr uint32_t kWaitSpins = 1u << 22;
constexpr uint32_t kPair = 2 * (kMaxRun + 1);  // symbols two look-ups can emit

// shared-memory form of a pre-walked entry, two words:
//   a: nb [3:0] (bits 4-5 stay 0) | symbols emitted = run + 1 [10:6] | newX [31:17]
//   b: 1- and 2-byte outputs: dequantised value [15:0] | row bytes * (run + 1) [31:16]
//      4-byte outputs:        dequantised value
// One extra entry after the table (index 2^R, which the 15-bit newX field can hold) emits nothing, reads
// nothing and leads to itself: a lane that must wait is parked on it.
__device__ __forceinline__ uint2 to_smem_entry(uint32_t g, uint32_t val, uint32_t row_bytes) {
  const uint32_t adv = entry_run(g) + 1u;
  uint2 e;
  e.x = entry_nb(g) | (adv << 6) | (entry_newx(g) << 17);
  e.y = row_bytes == 128u ? val : ((val & 0xFFFFu) | ((adv * row_bytes) << 16));
  return e;
}
constexpr int kMaxParkLog = 14;

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

template <int ES>
__device__ __forceinline__ void flush_rows(const uint8_t* tile, uint8_t* out_row0, size_t row_stride_bytes,
                                           uint32_t full_rows, uint32_t part_row_lanes, uint32_t lane) {
  constexpr uint32_t RB = 32u * ES;                 // bytes per row
  constexpr uint32_t PPR = RB / 16u;                // 16-byte pieces per row
  using E = typename ElemT<ES>::type;
  if ((reinterpret_cast<uintptr_t>(out_row0) & 15u) == 0 && (row_stride_bytes & 15u) == 0) {
    for (uint32_t idx = lane; idx < full_rows * PPR; idx += 32u) {
      const uint32_t row = idx / PPR, piece = idx % PPR;
      const uint4 v = *reinterpret_cast<const uint4*>(tile + size_t(idx) * 16u);
      *reinterpret_cast<uint4*>(out_row0 + size_t(row) * row_stride_bytes + piece * 16u) = v;
    }
  } else {
    for (uint32_t row = 0; row < full_rows; ++row)
      reinterpret_cast<E*>(out_row0 + size_t(row) * row_stride_bytes)[lane] =
          reinterpret_cast<const E*>(tile)[row * 32u + lane];
  }
  if (lane < part_row_lanes)
    reinterpret_cast<E*>(out_row0 + size_t(full_rows) * row_stride_bytes)[lane] =
        reinterpret_cast<const E*>(tile)[full_rows * 32u + lane];
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

// The hot loop, for a staged sub-stream: kPairsPerCall times, every lane makes two pre-walked
// look-ups that share one 32-bit extract of its bit window and one refill check (the loop ends
// early once no lane has work).  A lane whose
// next row is at or beyond its limit does the same work on the parking entry, which changes
// nothing, so the loop has no divergent branch.  Written as one PTX block so that the
// loop-carried values stay in registers across iterations.
//   st  : shared address of the state's table entry   tbm : RB * (last row the lane wrote), signed
//   bitpos : bits of w0 already used; only its low 5 bits are kept clean
//   w0,w1,w2 : bit window and the word after it        sp : shared address of the next word
// ring_lane_abs is the ring's address (a multiple of its size) + lane * ES, so OR forms the row address.
constexpr int kPairsPerCall = 32;

// ADV_: how tbm advances (from word b for narrow outputs, from word a's field for 4-byte ones)
#define ANSB_STEP(ADV_, STOP_)                                    \
  "ld.shared.v2.u32 {ea, eb}, [stx];\n\t"                         \
  "shf.l.wrap.b32 m, 0, -1, ea;\n\t"                              \
  "shr.u32 nx, ea, 17;\n\t"                                       \
  "lop3.b32 t, nx, x, m, 0xF4;\n\t"                               \
  "mad.lo.u32 stx, t, %13, %8;\n\t"                               \
  ADV_                                                            \
  "lop3.b32 a, %1, %11, %9, 0xEA;\n\t"                            \
  "@p " STOP_ " [a], eb;\n\t"                                     \
  "add.u32 %2, %2, ea;\n\t"

#define ANSB_ADV_NARROW "shr.u32 r, eb, 16;\n\tadd.u32 %1, %1, r;\n\t"
#define ANSB_ADV_WIDE "bfe.u32 r, ea, 6, 5;\n\tmad.lo.u32 %1, r, 128, %1;\n\t"

template <int ES>
__device__ __forceinline__ void pair_steps(uint32_t& st, uint32_t& tbm, uint32_t& bitpos, uint32_t& w0,
                                           uint32_t& w1, uint32_t& w2, uint32_t& sp, int32_t limm,
                                           uint32_t tab_abs, uint32_t ring_lane_abs, uint32_t park_abs,
                                           uint32_t stride) {
  constexpr uint32_t MASK = kRingRows * 32u * ES - 1u;
#define ANSB_ONE_PAIR(ADV_, STOP_)                                                         \
      "setp.lt.s32 p, %1, %7;\n\t"                                                         \
      "selp.b32 stx, %0, %10, p;\n\t"                                                      \
      "shf.r.wrap.b32 x, %3, %4, %2;\n\t"                                                  \
      "and.b32 %2, %2, 31;\n\t"                                                            \
      ANSB_STEP(ADV_, STOP_)                                                               \
      "shf.r.wrap.b32 x, x, 0, ea;\n\t"                                                    \
      ANSB_STEP(ADV_, STOP_)                                                               \
      "selp.b32 %0, stx, %0, p;\n\t"                                                       \
      "and.b32 t, %2, 32;\n\t"                                                             \
      "setp.ne.u32 q, t, 0;\n\t"                                                           \
      "@q mov.u32 %3, %4;\n\t"                                                             \
      "@q mov.u32 %4, %5;\n\t"                                                             \
      "@q ld.shared.u32 nw, [%6];\n\t"                                                     \
      "@q mov.u32 %5, nw;\n\t"                                                             \
      "@q add.u32 %6, %6, 4;\n\t"
#define ANSB_PAIRS(ADV_, STOP_)                                                            \
  asm volatile(                                                                            \
      "{\n\t"                                                                              \
      ".reg .pred p, q;\n\t"                                                               \
      ".reg .u32 x, ea, eb, m, t, nx, r, a, cnt, stx, nw;\n\t"                             \
      "mov.u32 cnt, %12;\n"                                                                \
      "ANSB_LOOP:\n\t"                                                                     \
      "setp.lt.s32 p, %1, %7;\n\t"                                                         \
      "vote.sync.any.pred q, p, 0xffffffff;\n\t"                                           \
      "@!q bra ANSB_DONE;\n\t"                                                             \
      ANSB_ONE_PAIR(ADV_, STOP_)                                                           \
      ANSB_ONE_PAIR(ADV_, STOP_)                                                           \
      "add.u32 cnt, cnt, -1;\n\t"                                                          \
      "setp.ne.u32 q, cnt, 0;\n\t"                                                         \
      "@q bra ANSB_LOOP;\n"                                                                \
      "ANSB_DONE:\n\t"                                                                     \
      "and.b32 %2, %2, 31;\n\t"                                                            \
      "}"                                                                                  \
      : "+r"(st), "+r"(tbm), "+r"(bitpos), "+r"(w0), "+r"(w1), "+r"(w2), "+r"(sp)          \
      : "r"(limm), "r"(tab_abs), "r"(ring_lane_abs), "r"(park_abs), "n"(MASK),             \
        "n"(kPairsPerCall / 2), "r"(stride)                                                \
      : "memory")
  if (ES == 1) ANSB_PAIRS(ANSB_ADV_NARROW, "st.shared.u8");
  if (ES == 2) ANSB_PAIRS(ANSB_ADV_NARROW, "st.shared.u16");
  if (ES == 4) ANSB_PAIRS(ANSB_ADV_WIDE, "st.shared.u32");
#undef ANSB_PAIRS
#undef ANSB_ONE_PAIR
}

// Decode one sub-stream.  Shared memory is addressed by absolute shared-window addresses:
// tab_abs (this lane's copy of the table; entries are 1 << stride_log bytes apart), succ_abs (u16
// successor of every zero-bit state), ring_abs (this warp's ring,
// aligned to its size), stage_abs (staged sub-stream when STAGED, with kStagePad readable bytes
// after it).  `ring` is the generic pointer to the same ring; `words` the sub-stream in
// global memory, used when it was not staged.
template <int ES, bool STAGED>
__device__ __noinline__ uint32_t decode_private(
    uint32_t tab_abs, uint32_t stride_log, uint32_t succ_abs, uint32_t ring_abs, uint32_t stage_abs,
    uint32_t park_abs, uint8_t* __restrict__ ring, uint32_t dom_val,
    const uint32_t* __restrict__ words, uint32_t ext_words, uint32_t wbeg, uint32_t wend, bool last_lane,
    uint32_t state, uint32_t my_count, uint32_t rows, uint32_t min_count, uint8_t* __restrict__ out_row0,
    size_t row_stride_bytes, uint32_t lane, uint32_t max_adv) {
  constexpr int RB = 32 * ES;
  constexpr uint32_t RING = kRingRows;              // rows in the ring
  constexpr uint32_t FL = kFlushRows;               // rows written out at a time
  constexpr uint32_t kRingBytes = RING * RB;
  constexpr uint32_t MASK = kRingBytes - 1u;
  static_assert(RING - FL >= kPair + FL, "a lane must be able to run ahead of the write-out");
  const uint32_t ring_lane_abs = ring_abs + lane * ES;

  // bit window: w0/w1 hold the 64 bits being read, w2 is one word ahead.  A staged lane may look
  // up to word_limit + kPairsPerCall + 3 words into its buffer, which holds ext_words + kStagePad / 4.
  static_assert(kStagePad / 4u >= 4u + kPairsPerCall + 4u, "staging pad too small for the look-ahead");
  const uint32_t word_limit = STAGED ? ext_words + 4u : ext_words;
  auto load_word = [&](uint32_t i) -> uint32_t {
    if (STAGED) return lds_u32(stage_abs + i * 4u);
    return i < word_limit ? __ldg(words + i) : 0u;
  };
  uint32_t idx = wbeg;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1), w2 = load_word(idx + 2);
  idx += 3;
  uint32_t bitpos = 0;
  bool overran = false;

  uint32_t fill = dom_val;
  if (ES == 1) fill *= 0x01010101u;
  if (ES == 2) fill *= 0x00010001u;
  const uint4 fill4 = make_uint4(fill, fill, fill, fill);
  for (uint32_t i = lane; i < kRingBytes / 16u; i += 32u) reinterpret_cast<uint4*>(ring)[i] = fill4;
  __syncwarp();

  // rows [first_row, first_row + n_rows), then `part_lanes` elements of the row after them;
  // the range may wrap around the ring's end
  auto write_out = [&](uint32_t first_row, uint32_t n_rows, uint32_t part_lanes) {
    uint32_t done = 0;
    while (done < n_rows) {
      const uint32_t r = first_row + done;
      const uint32_t ring_row = r % RING;
      const uint32_t piece = min(n_rows - done, RING - ring_row);
      flush_rows<ES>(ring + size_t(ring_row) * RB, out_row0 + size_t(r) * row_stride_bytes, row_stride_bytes,
                     piece, 0u, lane);
      done += piece;
    }
    if (part_lanes) {
      const uint32_t r = first_row + n_rows;
      flush_rows<ES>(ring + size_t(r % RING) * RB, out_row0 + size_t(r) * row_stride_bytes, row_stride_bytes,
                     0u, part_lanes, lane);
    }
  };
  // FL full rows starting at a multiple of FL leave the ring and are filled again: each 16-byte
  // piece is read, written out and re-filled by the same lane, so one warp barrier on each side
  // is all the ordering needed.  (Bulk asynchronous stores were measured here too: the wait for
  // the copy engine before the rows can be re-filled costs more than these few instructions.)
  auto write_block = [&](uint32_t first_row) {
    __syncwarp();
    uint8_t* part = ring + size_t(first_row % RING) * RB;
    uint8_t* dst = out_row0 + size_t(first_row) * row_stride_bytes;
    constexpr uint32_t PPR = RB / 16u;
    if (((reinterpret_cast<uintptr_t>(dst) | row_stride_bytes) & 15u) == 0) {
#pragma unroll
      for (uint32_t i = lane; i < FL * PPR; i += 32u) {
        const uint4 v = reinterpret_cast<const uint4*>(part)[i];
        *reinterpret_cast<uint4*>(dst + size_t(i / PPR) * row_stride_bytes + (i % PPR) * 16u) = v;
        reinterpret_cast<uint4*>(part)[i] = fill4;
      }
    } else {
      flush_rows<ES>(part, dst, row_stride_bytes, FL, 0u, lane);
      __syncwarp();
      for (uint32_t i = lane; i < (FL * RB) / 16u; i += 32u) reinterpret_cast<uint4*>(part)[i] = fill4;
    }
    __syncwarp();
  };

  uint32_t st = tab_abs + (state << stride_log);    // shared address of the state's table entry
  uint32_t tbm = static_cast<uint32_t>(-RB);        // RB * (last row this lane wrote): none yet
  // one pre-walked look-up: emits run + 1 symbols, takes its bits from the low end of x
  auto step = [&](uint32_t x) -> uint32_t {
    const uint32_t ea = lds_u32(st), eb = lds_u32(st + 4u);
    const uint32_t nb = ea & 15u;
    st = tab_abs + (((ea >> 17) | (x & ((1u << nb) - 1u))) << stride_log);
    tbm += ((ea >> 6) & 31u) * RB;
    sts_elem<ES>((tbm & MASK) | ring_lane_abs, eb);
    return nb;
  };
  auto refill_checked = [&]() {
    if (bitpos >= 32u) {
      w0 = w1; w1 = w2;
      w2 = (!STAGED || idx < word_limit) ? load_word(idx) : 0u;
      ++idx;
      bitpos -= 32u;
    }
  };
  auto next_row = [&]() -> int32_t { return (static_cast<int32_t>(tbm) + RB) / RB; };

  // main part: two look-ups share one 32-bit extract (2 * 14 bits at most) and one refill check;
  // it stops short of the lane's end by what a pair can emit at most in this layer (2 * max_adv
  // symbols, max_adv = longest run in the layer's table + 1), so a pair can never emit too many
  const uint32_t pair_max = 2u * max_adv;
  const int32_t lim2 = static_cast<int32_t>(my_count > pair_max - 1 ? my_count - (pair_max - 1) : 0u);
  const int32_t lim1 = static_cast<int32_t>(my_count > max_adv - 1 ? my_count - (max_adv - 1) : 0u);
  uint32_t base = 0;                                // first row not yet written out
  for (;;) {
    const int32_t lim = min(lim2, static_cast<int32_t>(base + RING - pair_max));   // rows
    if (STAGED && park_abs != 0u) {
      uint32_t sp = stage_abs + idx * 4u;
      pair_steps<ES>(st, tbm, bitpos, w0, w1, w2, sp, (lim - 1) * RB, tab_abs, ring_lane_abs, park_abs,
                     1u << stride_log);
      idx = (sp - stage_abs) >> 2;
      if (idx > word_limit) { overran = true; idx = word_limit; }
    } else {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        if (next_row() < lim) {
          const uint32_t x = __funnelshift_r(w0, w1, bitpos);
          const uint32_t nb1 = step(x);
          const uint32_t nb2 = step(x >> nb1);
          bitpos += nb1 + nb2;
          refill_checked();
        }
      }
    }
    const uint32_t tmin = static_cast<uint32_t>(__reduce_min_sync(kFull, next_row()));
    while (tmin >= base + FL) {                     // the slowest lane has left these rows
      write_block(base);
      base += FL;
    }
    if (__all_sync(kFull, next_row() >= lim2)) break;
  }
  // then single pre-walked look-ups while at least 16 symbols are owed to the lane ...
  while (next_row() < lim1) {
    bitpos += step(__funnelshift_r(w0, w1, bitpos));
    refill_checked();
  }
  // ... and the last (up to 15) symbols one at a time: a state whose pre-walked entry has no run
  // is stepped as above; a zero-bit state of the dominant symbol emits that symbol (its value is
  // already in the ring), reads nothing and goes to its one successor, kept in a side table
  while (next_row() < static_cast<int32_t>(my_count)) {
    const uint32_t ea = lds_u32(st);
    if (((ea >> 6) & 31u) == 1u) {
      bitpos += step(__funnelshift_r(w0, w1, bitpos));
      refill_checked();
    } else {
      st = tab_abs + (lds_u16(succ_abs + (((st - tab_abs) >> stride_log) << 1)) << stride_log);
      tbm += RB;
    }
  }
  state = (st - tab_abs) >> stride_log;
  __syncwarp();
  {
    const bool has_part = min_count < rows;         // last row is ragged
    const uint32_t full_rows = (has_part ? rows - 1 : rows) - base;
    uint32_t part_lanes = 0;
    if (has_part) part_lanes = __popc(__ballot_sync(kFull, my_count == rows));
    write_out(base, full_rows, part_lanes);
  }
  __syncwarp();
  uint32_t bad = 0;
  if (state != 0) bad |= ANS_STATUS_BAD_FINAL_STATE;
  // words used must be exactly the lane's run (the last lane's run is followed by < 16 pad bytes)
  const uint32_t bits = (idx - 3u - wbeg) * 32u + bitpos;
  const uint32_t need = (bits + 31u) / 32u;
  const uint32_t have = wend - wbeg;
  if (overran || (last_lane ? (need > have || have - need >= 4u) : (need != have))) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

// =============================================================================================
// Private container, lockstep walk: every look-up emits exactly one symbol (the plain table of
// Section II-A), so the 32 lanes of a warp stay on the same output row.  A row is complete as
// soon as it is decoded and each lane stores its element straight to the output: a row is
// 32 * ES contiguous bytes, whole 32-byte sectors; no ring, no pre-fill, no parking, no tail.
// The price is one look-up per symbol, which pays when look-ups are cheap (a table small enough
// for conflict-free copies) or the pre-walked entries would stand for few symbols anyway.
//
// kFlushRows rows are decoded by one PTX block (row stores at immediate offsets), K look-ups
// sharing one 32-bit extract of the bit window and one refill check: K = 4 when a symbol takes
// at most 8 bits, else 2.  Multiply-high is avoided on purpose (it runs at a fraction of the
// rate of shifts and adds); the bit count is accumulated on the multiply-add pipe, which is
// otherwise idle, by a multiplication with a run-time 1.
// =============================================================================================
#define ANSB_LS_STEP(STOP_, ADDR_)                                \
  "ld.shared.v2.u32 {ea, eb}, [%0];\n\t"                          \
  "shf.l.wrap.b32 m, 0, -1, ea;\n\t"                              \
  "shr.u32 nx, ea, 17;\n\t"                                       \
  "lop3.b32 t, nx, x, m, 0xF4;\n\t"                               \
  "mad.lo.u32 %0, t, %7, %6;\n\t"                                 \
  "shf.r.wrap.b32 x, x, 0, ea;\n\t"                               \
  STOP_ " " ADDR_ ", eb;\n\t"                                     \
  "mad.lo.u32 %1, ea, %9, %1;\n\t"
#define ANSB_LS_BEGIN "shf.r.wrap.b32 x, %2, %3, %1;\n\t"
#define ANSB_LS_END                                               \
  "and.b32 t, %1, 32;\n\t"                                        \
  "setp.ne.u32 q, t, 0;\n\t"                                      \
  "@q mov.u32 %2, %3;\n\t"                                        \
  "@q mov.u32 %3, %4;\n\t"                                        \
  "@q ld.shared.u32 nw, [%5];\n\t"                                \
  "@q mov.u32 %4, nw;\n\t"                                        \
  "@q add.u32 %5, %5, 4;\n\t"                                     \
  "and.b32 %1, %1, 31;\n\t"
#define ANSB_LS_G4(S_, A0, A1, A2, A3)                            \
  ANSB_LS_BEGIN ANSB_LS_STEP(S_, A0) ANSB_LS_STEP(S_, A1) ANSB_LS_STEP(S_, A2) ANSB_LS_STEP(S_, A3) ANSB_LS_END
#define ANSB_LS_G2(S_, A0, A1) ANSB_LS_BEGIN ANSB_LS_STEP(S_, A0) ANSB_LS_STEP(S_, A1) ANSB_LS_END

// st: shared address of the state's entry; bitpos in [0, 32); w0,w1: bit window, w2 the word after
// it; sp: shared address of the word after w2; gp: this lane's element of the block's first row
// in the output (rows are 32 * ES * G bytes apart); one: the value 1, not known at compile time
template <int ES, int K, int G>
__device__ __forceinline__ void lockstep_block(uint32_t& st, uint32_t& bitpos, uint32_t& w0, uint32_t& w1,
                                               uint32_t& w2, uint32_t& sp, uint32_t tab_lane, uint32_t stride,
                                               uint8_t* gp, uint32_t one) {
  constexpr uint32_t RS = 32u * ES * G;
  static_assert(kFlushRows == 16, "the block below is written out for 16 rows");
#define ANSB_LS_BODY4(S_)                                                                   \
      ANSB_LS_G4(S_, "[%8]", "[%8+%10]", "[%8+%11]", "[%8+%12]")                            \
      ANSB_LS_G4(S_, "[%8+%13]", "[%8+%14]", "[%8+%15]", "[%8+%16]")                        \
      ANSB_LS_G4(S_, "[%8+%17]", "[%8+%18]", "[%8+%19]", "[%8+%20]")                        \
      ANSB_LS_G4(S_, "[%8+%21]", "[%8+%22]", "[%8+%23]", "[%8+%24]")
#define ANSB_LS_BODY2(S_)                                                                   \
      ANSB_LS_G2(S_, "[%8]", "[%8+%10]") ANSB_LS_G2(S_, "[%8+%11]", "[%8+%12]")             \
      ANSB_LS_G2(S_, "[%8+%13]", "[%8+%14]") ANSB_LS_G2(S_, "[%8+%15]", "[%8+%16]")         \
      ANSB_LS_G2(S_, "[%8+%17]", "[%8+%18]") ANSB_LS_G2(S_, "[%8+%19]", "[%8+%20]")         \
      ANSB_LS_G2(S_, "[%8+%21]", "[%8+%22]") ANSB_LS_G2(S_, "[%8+%23]", "[%8+%24]")
#define ANSB_LS_ASM(BODY_)                                                                  \
  asm volatile(                                                                             \
      "{\n\t"                                                                               \
      ".reg .pred q;\n\t"                                                                   \
      ".reg .u32 x, ea, eb, m, t, nx, nw;\n\t"                                              \
      BODY_                                                                                 \
      "}"                                                                                   \
      : "+r"(st), "+r"(bitpos), "+r"(w0), "+r"(w1), "+r"(w2), "+r"(sp)                      \
      : "r"(tab_lane), "r"(stride), "l"(gp), "r"(one), "n"(RS * 1), "n"(RS * 2), "n"(RS * 3), \
        "n"(RS * 4), "n"(RS * 5), "n"(RS * 6), "n"(RS * 7), "n"(RS * 8), "n"(RS * 9), "n"(RS * 10), \
        "n"(RS * 11), "n"(RS * 12), "n"(RS * 13), "n"(RS * 14), "n"(RS * 15)                \
      : "memory")
  if (K == 4) {
    if (ES == 1) ANSB_LS_ASM(ANSB_LS_BODY4("st.global.u8"));
    if (ES == 2) ANSB_LS_ASM(ANSB_LS_BODY4("st.global.u16"));
    if (ES == 4) ANSB_LS_ASM(ANSB_LS_BODY4("st.global.u32"));
  } else {
    if (ES == 1) ANSB_LS_ASM(ANSB_LS_BODY2("st.global.u8"));
    if (ES == 2) ANSB_LS_ASM(ANSB_LS_BODY2("st.global.u16"));
    if (ES == 4) ANSB_LS_ASM(ANSB_LS_BODY2("st.global.u32"));
  }
#undef ANSB_LS_ASM
#undef ANSB_LS_BODY2
#undef ANSB_LS_BODY4
}

template <int ES>
__device__ __forceinline__ void stg_elem(uint8_t* p, uint32_t v) {
  if (ES == 1) *p = static_cast<uint8_t>(v);
  if (ES == 2) *reinterpret_cast<uint16_t*>(p) = static_cast<uint16_t>(v);
  if (ES == 4) *reinterpret_cast<uint32_t*>(p) = v;
}

// Decode one sub-stream in lockstep.  tab_abs: this lane's copy of the plain table; stage_abs: the
// staged sub-stream when STAGED; words: the sub-stream in global memory otherwise; rows of one
// sub-stream are `groups` rows of the chunk apart in the output.
template <int ES, bool STAGED>
__device__ __noinline__ uint32_t decode_lockstep(
    uint32_t tab_abs, uint32_t stride_log, uint32_t stage_abs, const uint32_t* __restrict__ words,
    uint32_t ext_words, uint32_t wbeg, uint32_t wend, bool last_lane, uint32_t state, uint32_t my_count,
    uint32_t rows, uint32_t min_count, uint8_t* __restrict__ out_row0, uint32_t groups, uint32_t lane,
    bool wide_steps, uint32_t one) {
  constexpr uint32_t RB = 32u * ES;
  constexpr uint32_t FL = kFlushRows;
  const size_t row_stride_bytes = size_t(RB) * groups;
  // a staged lane may look up to word_limit + 8 words into its buffer (a block advances it by at
  // most 8 words), which holds ext_words + kStagePad / 4
  const uint32_t word_limit = STAGED ? ext_words + 4u : ext_words;
  auto load_word = [&](uint32_t i) -> uint32_t {
    if (STAGED) return lds_u32(stage_abs + i * 4u);
    return i < word_limit ? __ldg(words + i) : 0u;
  };
  uint32_t idx = wbeg;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1), w2 = load_word(idx + 2);
  idx += 3;
  uint32_t bitpos = 0;
  bool overran = false;
  uint32_t st = tab_abs + (state << stride_log);
  uint8_t* gp = out_row0 + size_t(lane) * ES;       // this lane's element of the next row

  // one look-up in plain code: rows outside whole blocks, and sub-streams that were not staged
  auto step = [&]() {
    const uint32_t ea = lds_u32(st), eb = lds_u32(st + 4u);
    const uint32_t nb = ea & 15u;
    const uint32_t x = __funnelshift_r(w0, w1, bitpos);
    st = tab_abs + (((ea >> 17) | (x & ((1u << nb) - 1u))) << stride_log);
    stg_elem<ES>(gp, eb);
    gp += row_stride_bytes;
    bitpos += nb;
    if (bitpos >= 32u) {
      w0 = w1; w1 = w2;
      w2 = (!STAGED || idx < word_limit) ? load_word(idx) : 0u;
      ++idx;
      bitpos -= 32u;
    }
  };

  uint32_t r = 0;
  if (STAGED) {
    uint32_t sp = stage_abs + idx * 4u;
    const uint32_t sp_limit = stage_abs + word_limit * 4u;
    const uint32_t stride = 1u << stride_log;
#define ANSB_LS_LOOP(K_, G_)                                                                \
    while (r + FL <= min_count) {                                                           \
      lockstep_block<ES, K_, G_>(st, bitpos, w0, w1, w2, sp, tab_abs, stride, gp, one);     \
      if (sp > sp_limit) { overran = true; sp = sp_limit; }                                 \
      gp += FL * RB * G_;                                                                   \
      r += FL;                                                                              \
    }
    if (wide_steps) {
      if (groups == 1) { ANSB_LS_LOOP(4, 1) } else if (groups == 2) { ANSB_LS_LOOP(4, 2) }
      else if (groups == 4) { ANSB_LS_LOOP(4, 4) } else if (groups == 8) { ANSB_LS_LOOP(4, 8) }
    } else {
      if (groups == 1) { ANSB_LS_LOOP(2, 1) } else if (groups == 2) { ANSB_LS_LOOP(2, 2) }
      else if (groups == 4) { ANSB_LS_LOOP(2, 4) } else if (groups == 8) { ANSB_LS_LOOP(2, 8) }
    }
#undef ANSB_LS_LOOP
    idx = (sp - stage_abs) >> 2;
  }
  for (; r < min_count; ++r) step();
  if (rows > min_count && my_count == rows) step();   // the ragged last row
  uint32_t bad = 0;
  if (st != tab_abs) bad |= ANS_STATUS_BAD_FINAL_STATE;
  // words used must be exactly the lane's run (the last lane's run is followed by < 16 pad bytes)
  const uint32_t bits = (idx - 3u - wbeg) * 32u + bitpos;
  const uint32_t need = (bits + 31u) / 32u;
  const uint32_t have = wend - wbeg;
  if (overran || (last_lane ? (need > have || have - need >= 4u) : (need != have))) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

// =============================================================================================
// Quads container: the lockstep walk with two changes that the container makes possible.
// A lane owns four adjacent output elements per turn, so the four values of a turn leave in one
// vector store (8 bytes of bf16 per lane, 256 contiguous bytes per warp) instead of four.  And
// the bit window is kept top-aligned (bits are taken from the most significant end), so that
// one funnel shift builds the next state: with q = newX >> nb_bits kept in the entry,
// (q << nb) | (window >> (32 - nb)) needs no mask; a second one drops the bits taken.
//
// shared-memory entry, two words:
//   1- and 2-byte outputs:  a = nb [4:0] | dequantised value [31:16]      b = q
//   4-byte outputs:         a = nb [4:0] | q [31:8]                       b = dequantised value
// =============================================================================================
__device__ __forceinline__ uint2 to_quads_entry(uint32_t g, uint32_t val, bool narrow) {
  const uint32_t nb = entry_nb(g), q = entry_newx(g) >> nb;
  return narrow ? make_uint2(nb | (val << 16), q) : make_uint2(nb | (q << 8), val);
}

#define ANSB_QD_STEP_N(I_)                                        \
  "ld.shared.v2.u32 {ea" I_ ", eb" I_ "}, [%0];\n\t"              \
  "shf.l.wrap.b32 t, x, eb" I_ ", ea" I_ ";\n\t"                  \
  "shf.l.wrap.b32 x, 0, x, ea" I_ ";\n\t"                         \
  "mad.lo.u32 %0, t, %7, %6;\n\t"                                 \
  "mad.lo.u32 %1, ea" I_ ", %9, %1;\n\t"
#define ANSB_QD_STEP_W(I_)                                        \
  "ld.shared.v2.u32 {ea" I_ ", eb" I_ "}, [%0];\n\t"              \
  "shr.u32 nx, ea" I_ ", 8;\n\t"                                  \
  "shf.l.wrap.b32 t, x, nx, ea" I_ ";\n\t"                        \
  "shf.l.wrap.b32 x, 0, x, ea" I_ ";\n\t"                         \
  "mad.lo.u32 %0, t, %7, %6;\n\t"                                 \
  "mad.lo.u32 %1, ea" I_ ", %9, %1;\n\t"
#define ANSB_QD_BEGIN "shf.l.wrap.b32 x, %3, %2, %1;\n\t"
// four look-ups of one turn: one refill check when a symbol takes at most 8 bits, else two
#define ANSB_QD_TURN4(ST_) ANSB_QD_BEGIN ST_("0") ST_("1") ST_("2") ST_("3") ANSB_LS_END
#define ANSB_QD_TURN2(ST_) ANSB_QD_BEGIN ST_("0") ST_("1") ANSB_LS_END ANSB_QD_BEGIN ST_("2") ST_("3") ANSB_LS_END
#define ANSB_QD_OUT1(A_)                                          \
  "prmt.b32 v0, ea0, ea1, 0x0062;\n\t"                            \
  "prmt.b32 v1, ea2, ea3, 0x0062;\n\t"                            \
  "prmt.b32 v0, v0, v1, 0x5410;\n\t"                              \
  "st.global.u32 " A_ ", v0;\n\t"
#define ANSB_QD_OUT2(A_)                                          \
  "prmt.b32 v0, ea0, ea1, 0x7632;\n\t"                            \
  "prmt.b32 v1, ea2, ea3, 0x7632;\n\t"                            \
  "st.global.v2.u32 " A_ ", {v0, v1};\n\t"
#define ANSB_QD_OUT4(A_) "st.global.v4.u32 " A_ ", {eb0, eb1, eb2, eb3};\n\t"

constexpr uint32_t kQuadTurns = 4;     // turns (of four symbols per lane) per trip of the PTX loop

// The hot loop of the quads container: `blocks` times kQuadTurns turns, entirely in PTX (loop
// included, so that nothing is carried through the compiler between trips).  Operands as in
// lockstep_block; gp: this lane's four elements of the first turn; turns are 128 * ES * groups
// bytes apart (immediate offsets when groups == 1); sp is held at sp_limit if a corrupt stream
// drives it that far.
template <int ES, int K>
__device__ __forceinline__ void quads_loop(uint32_t& st, uint32_t& bitpos, uint32_t& w0, uint32_t& w1,
                                           uint32_t& w2, uint32_t& sp, uint32_t tab_lane, uint32_t stride,
                                           uint8_t* gp, uint32_t unit, uint32_t groups, uint32_t blocks,
                                           uint32_t sp_limit) {
  constexpr uint32_t RS = 128u * ES;
#define ANSB_QD_ASM1(LBL_, TURN_, ST_, OUT_)                                                \
  asm volatile(                                                                             \
      "{\n\t"                                                                               \
      ".reg .pred q;\n\t"                                                                   \
      ".reg .u32 x, t, nx, nw, v0, v1, cnt, ea0, ea1, ea2, ea3, eb0, eb1, eb2, eb3;\n\t"     \
      ".reg .u64 gpp;\n\t"                                                                  \
      "mov.u64 gpp, %8;\n\t"                                                                \
      "mov.u32 cnt, %10;\n"                                                                 \
      LBL_ ":\n\t"                                                                          \
      TURN_(ST_) OUT_("[gpp]") TURN_(ST_) OUT_("[gpp+%12]")                                 \
      TURN_(ST_) OUT_("[gpp+%13]") TURN_(ST_) OUT_("[gpp+%14]")                             \
      "add.u64 gpp, gpp, %15;\n\t"                                                          \
      "min.u32 %5, %5, %11;\n\t"                                                            \
      "add.u32 cnt, cnt, -1;\n\t"                                                           \
      "setp.ne.u32 q, cnt, 0;\n\t"                                                          \
      "@q bra " LBL_ ";\n\t"                                                                \
      "}"                                                                                   \
      : "+r"(st), "+r"(bitpos), "+r"(w0), "+r"(w1), "+r"(w2), "+r"(sp)                      \
      : "r"(tab_lane), "r"(stride), "l"(gp), "r"(unit), "r"(blocks), "r"(sp_limit),         \
        "n"(RS * 1), "n"(RS * 2), "n"(RS * 3), "n"(RS * 4)                                  \
      : "memory")
#define ANSB_QD_ASMG(LBL_, TURN_, ST_, OUT_)                                                \
  asm volatile(                                                                             \
      "{\n\t"                                                                               \
      ".reg .pred q;\n\t"                                                                   \
      ".reg .u32 x, t, nx, nw, v0, v1, cnt, ea0, ea1, ea2, ea3, eb0, eb1, eb2, eb3;\n\t"     \
      ".reg .u64 gpp;\n\t"                                                                  \
      "mov.u64 gpp, %8;\n\t"                                                                \
      "mov.u32 cnt, %10;\n"                                                                 \
      LBL_ ":\n\t"                                                                          \
      TURN_(ST_) OUT_("[gpp]") "add.u64 gpp, gpp, %12;\n\t"                                 \
      TURN_(ST_) OUT_("[gpp]") "add.u64 gpp, gpp, %12;\n\t"                                 \
      TURN_(ST_) OUT_("[gpp]") "add.u64 gpp, gpp, %12;\n\t"                                 \
      TURN_(ST_) OUT_("[gpp]") "add.u64 gpp, gpp, %12;\n\t"                                 \
      "min.u32 %5, %5, %11;\n\t"                                                            \
      "add.u32 cnt, cnt, -1;\n\t"                                                           \
      "setp.ne.u32 q, cnt, 0;\n\t"                                                          \
      "@q bra " LBL_ ";\n\t"                                                                \
      "}"                                                                                   \
      : "+r"(st), "+r"(bitpos), "+r"(w0), "+r"(w1), "+r"(w2), "+r"(sp)                      \
      : "r"(tab_lane), "r"(stride), "l"(gp), "r"(unit), "r"(blocks), "r"(sp_limit),         \
        "l"(static_cast<unsigned long long>(RS) * groups)                                   \
      : "memory")
#define ANSB_QD_BOTH(L1_, LG_, TURN_, ST_, OUT_)                                            \
  if (groups == 1) ANSB_QD_ASM1(L1_, TURN_, ST_, OUT_); else ANSB_QD_ASMG(LG_, TURN_, ST_, OUT_)
  if (K == 4) {
    if (ES == 1) { ANSB_QD_BOTH("ANSB_Q41", "ANSB_Q4G", ANSB_QD_TURN4, ANSB_QD_STEP_N, ANSB_QD_OUT1); }
    if (ES == 2) { ANSB_QD_BOTH("ANSB_Q41", "ANSB_Q4G", ANSB_QD_TURN4, ANSB_QD_STEP_N, ANSB_QD_OUT2); }
    if (ES == 4) { ANSB_QD_BOTH("ANSB_Q41", "ANSB_Q4G", ANSB_QD_TURN4, ANSB_QD_STEP_W, ANSB_QD_OUT4); }
  } else {
    if (ES == 1) { ANSB_QD_BOTH("ANSB_Q21", "ANSB_Q2G", ANSB_QD_TURN2, ANSB_QD_STEP_N, ANSB_QD_OUT1); }
    if (ES == 2) { ANSB_QD_BOTH("ANSB_Q21", "ANSB_Q2G", ANSB_QD_TURN2, ANSB_QD_STEP_N, ANSB_QD_OUT2); }
    if (ES == 4) { ANSB_QD_BOTH("ANSB_Q21", "ANSB_Q2G", ANSB_QD_TURN2, ANSB_QD_STEP_W, ANSB_QD_OUT4); }
  }
#undef ANSB_QD_BOTH
#undef ANSB_QD_ASMG
#undef ANSB_QD_ASM1
}

// Decode one sub-stream of the quads container.  full_turns: turns in which every lane of the
// sub-stream owns a whole quad; out_lane: this lane's first output element; a lane's turns are
// 128 * ES * groups bytes apart.
template <int ES, bool STAGED>
__device__ __noinline__ uint32_t decode_quads(
    uint32_t tab_abs, uint32_t stride_log, uint32_t stage_abs, const uint32_t* __restrict__ words,
    uint32_t ext_words, uint32_t wbeg, uint32_t wend, bool last_lane, uint32_t state, uint32_t my_count,
    uint32_t full_turns, uint8_t* __restrict__ out_lane, uint32_t groups, bool wide_steps, uint32_t unit) {
  constexpr bool NARROW = ES != 4;
  constexpr uint32_t QB = 4u * ES;                  // bytes of a quad
  const size_t turn_stride = size_t(128u * ES) * groups;
  const uint32_t word_limit = STAGED ? ext_words + 4u : ext_words;
  auto load_word = [&](uint32_t i) -> uint32_t {
    if (STAGED) return lds_u32(stage_abs + i * 4u);
    return i < word_limit ? __ldg(words + i) : 0u;
  };
  uint32_t idx = wbeg;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1), w2 = load_word(idx + 2);
  idx += 3;
  uint32_t bitpos = 0;
  bool overran = false;
  uint32_t st = tab_abs + (state << stride_log);
  uint32_t k = 0;                                   // symbols this lane has decoded

  uint32_t turn = 0;
  // whole blocks: needs the staged copy, and quads that may leave as one vector store
  if (STAGED && (reinterpret_cast<uintptr_t>(out_lane) & (QB - 1u)) == 0) {
    uint32_t sp = stage_abs + idx * 4u;
    const uint32_t sp_limit = stage_abs + word_limit * 4u;   // a sound lane stays below it
    const uint32_t blocks = full_turns / kQuadTurns;
    if (blocks) {
      if (wide_steps) quads_loop<ES, 4>(st, bitpos, w0, w1, w2, sp, tab_abs, 1u << stride_log, out_lane, unit, groups,
                                        blocks, sp_limit);
      else quads_loop<ES, 2>(st, bitpos, w0, w1, w2, sp, tab_abs, 1u << stride_log, out_lane, unit, groups, blocks,
                             sp_limit);
      if (sp >= sp_limit) overran = true;
      turn = blocks * kQuadTurns;
    }
    idx = (sp - stage_abs) >> 2;
    k = 4u * turn;
  }
  // the rest in plain code, one symbol and one element store at a time
  for (; k < my_count; ++k) {
    const uint32_t ea = lds_u32(st), eb = lds_u32(st + 4u);
    const uint32_t nb = ea & 31u;
    const uint32_t q = NARROW ? eb : ea >> 8, val = NARROW ? ea >> 16 : eb;
    const uint32_t x = __funnelshift_l(w1, w0, bitpos);
    st = tab_abs + (__funnelshift_l(x, q, nb) << stride_log);
    stg_elem<ES>(out_lane + size_t(k >> 2) * turn_stride + (k & 3u) * ES, val);
    bitpos += nb;
    if (bitpos >= 32u) {
      w0 = w1; w1 = w2;
      w2 = (!STAGED || idx < word_limit) ? load_word(idx) : 0u;
      ++idx;
      bitpos -= 32u;
    }
  }
  uint32_t bad = 0;
  if (st != tab_abs) bad |= ANS_STATUS_BAD_FINAL_STATE;
  const uint32_t bits = (idx - 3u - wbeg) * 32u + bitpos;
  const uint32_t need = (bits + 31u) / 32u;
  const uint32_t have = wend - wbeg;
  if (overran || (last_lane ? (need > have || have - need >= 4u) : (need != have))) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

// =============================================================================================
// Interleaved container: the warp's 32 lanes share one sequence of 16-bit units; before each
// round a lane whose buffer holds fewer than 16 bits takes the next unit, its place found by
// ballot + popcount; then every lane decodes one symbol.  Same shared-memory table and staging
// buffer as above.  Every look-up emits exactly one symbol, so a round completes a row of the
// output and every lane stores its element straight to it (32 * ES contiguous bytes per row).
// =============================================================================================
template <int ES>
__device__ __forceinline__ void interleaved_rounds(uint32_t& st, uint32_t& buf, uint32_t& cnt, uint32_t& posaddr,
                                                   uint8_t*& gp, uint32_t n, uint32_t lt, uint32_t limaddr,
                                                   uint32_t tab_abs, uint32_t stride, unsigned long long row_stride) {
#define ANSB_ROUNDS(STOP_)                                                                 \
  asm volatile(                                                                            \
      "{\n\t"                                                                              \
      ".reg .pred p, q;\n\t"                                                               \
      ".reg .u32 b, t, a, u, inc, ea, eb, m, nx, cntr;\n\t"                                \
      "mov.u32 cntr, %5;\n"                                                                \
      "ANSB_RLOOP:\n\t"                                                                    \
      "setp.lt.u32 p, %2, 16;\n\t"                                                         \
      "vote.sync.ballot.b32 b, p, 0xffffffff;\n\t"                                         \
      "and.b32 t, b, %6;\n\t"                                                              \
      "popc.b32 t, t;\n\t"                                                                 \
      "mad.lo.u32 a, t, 2, %3;\n\t"                                                        \
      "min.u32 a, a, %7;\n\t"                                                              \
      "mov.u32 u, 0;\n\t"                                                                  \
      "@p ld.shared.u16 u, [a];\n\t"                                                       \
      "shl.b32 u, u, %2;\n\t"                                                              \
      "or.b32 %1, %1, u;\n\t"                                                              \
      "selp.u32 inc, 16, 0, p;\n\t"                                                        \
      "add.u32 %2, %2, inc;\n\t"                                                           \
      "popc.b32 t, b;\n\t"                                                                 \
      "mad.lo.u32 %3, t, 2, %3;\n\t"                                                       \
      "ld.shared.v2.u32 {ea, eb}, [%0];\n\t"                                               \
      "shf.l.wrap.b32 m, 0, -1, ea;\n\t"                                                   \
      "shr.u32 nx, ea, 17;\n\t"                                                            \
      "lop3.b32 t, nx, %1, m, 0xF4;\n\t"                                                   \
      "mad.lo.u32 %0, t, %9, %8;\n\t"                                                      \
      "shf.r.wrap.b32 %1, %1, 0, ea;\n\t"                                                  \
      "and.b32 t, ea, 15;\n\t"                                                             \
      "sub.u32 %2, %2, t;\n\t"                                                             \
      STOP_ " [%4], eb;\n\t"                                                               \
      "add.u64 %4, %4, %10;\n\t"                                                           \
      "add.u32 cntr, cntr, -1;\n\t"                                                        \
      "setp.ne.u32 q, cntr, 0;\n\t"                                                        \
      "@q bra ANSB_RLOOP;\n\t"                                                             \
      "}"                                                                                  \
      : "+r"(st), "+r"(buf), "+r"(cnt), "+r"(posaddr), "+l"(gp)                            \
      : "r"(n), "r"(lt), "r"(limaddr), "r"(tab_abs), "r"(stride), "l"(row_stride)          \
      : "memory")
  if (ES == 1) ANSB_ROUNDS("st.global.u8");
  if (ES == 2) ANSB_ROUNDS("st.global.u16");
  if (ES == 4) ANSB_ROUNDS("st.global.u32");
#undef ANSB_ROUNDS
}

template <int ES, bool STAGED>
__device__ __noinline__ uint32_t decode_interleaved(
    uint32_t tab_abs, uint32_t stride_log, uint32_t stage_abs, const uint16_t* __restrict__ units, uint32_t unit_cap,
    uint32_t state, uint32_t my_count, uint32_t rows, uint32_t min_count, uint8_t* __restrict__ out_row0,
    size_t row_stride_bytes, uint32_t lane) {
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t st = tab_abs + (state << stride_log);    // shared address of the state's table entry
  uint32_t buf = 0, cnt = 0;                        // the lane's bit buffer and how many bits it holds
  uint32_t pos = 0;                                 // units the warp has taken (same in every lane)
  uint8_t* gp = out_row0 + size_t(lane) * ES;       // this lane's element of the next row

  // one round in plain code: used when the sub-stream was not staged, and for the ragged round
  auto round = [&](bool active) {
    const bool need = active && cnt < 16u;
    const uint32_t b = __ballot_sync(kFull, need);
    if (need) {
      const uint32_t idx = pos + __popc(b & lt);
      uint32_t u = 0;
      if (idx < unit_cap) u = STAGED ? (lds_u32(stage_abs + (idx >> 1) * 4u) >> ((idx & 1u) * 16u)) & 0xFFFFu
                                     : static_cast<uint32_t>(__ldg(units + idx));
      buf |= u << cnt;
      cnt += 16u;
    }
    pos += __popc(b);
    if (active) {
      const uint32_t ea = lds_u32(st), eb = lds_u32(st + 4u);
      const uint32_t nb = ea & 15u;
      st = tab_abs + (((ea >> 17) | (buf & ((1u << nb) - 1u))) << stride_log);
      buf >>= nb;
      cnt -= nb;
      stg_elem<ES>(gp, eb);
    }
    gp += row_stride_bytes;
  };

  if (STAGED && min_count) {                        // rounds in which all 32 lanes decode
    uint32_t posaddr = stage_abs + pos * 2u;
    interleaved_rounds<ES>(st, buf, cnt, posaddr, gp, min_count, lt, stage_abs + unit_cap * 2u, tab_abs,
                           1u << stride_log, static_cast<unsigned long long>(row_stride_bytes));
    pos = (posaddr - stage_abs) >> 1;
  } else {
    for (uint32_t i = 0; i < min_count; ++i) round(true);
  }
  if (rows > min_count) round(my_count == rows);    // the ragged last round
  uint32_t bad = 0;
  if (st != tab_abs) bad |= ANS_STATUS_BAD_FINAL_STATE;
  // the units taken, padded to 16 bytes, must be exactly the sub-stream's extent
  if (((pos * 2u + 15u) & ~15u) != unit_cap * 2u) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

// dynamic shared memory, by absolute shared address: [pad to ring_bytes][rings: NW * ring_bytes]
// [table, in copies][pad to 1 KB][vals 256 words][successor table][mbarriers NW][stages NW * stage_bytes]

template <int LAYOUT, bool LOCK, bool MANY>
__global__ void __launch_bounds__(MANY ? 896 : 512, 1) ans_decode_kernel(const LaunchArgs args) {
  // LOCK: the walks that store rows straight to the output (interleaved, private lockstep, quads).
  // Not LOCK: the private container's pre-walked walk.  MANY: up to 28 warps per CTA on 72
  // registers (the LOCK walks on large layers); otherwise up to 16 warps and no register
  // pressure, which the small CTAs of small-layer models want: a spill there is a cold trip to
  // memory on a path that is all latency.
  constexpr bool kQuads = LAYOUT == ANS_LAYOUT_QUADS;
  constexpr bool kPrivate = LAYOUT != ANS_LAYOUT_INTERLEAVED;   // lanes own their words
  constexpr bool lock = kPrivate && LOCK;           // walked one symbol per look-up (quads always are)
  extern __shared__ __align__(16) uint8_t sm[];
  const uint32_t NW = blockDim.x >> 5;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t sm_abs = smem_u32(sm);
  const uint32_t ring_align = args.ring_bytes ? args.ring_bytes : 16u;
  const uint32_t rings_abs = (sm_abs + ring_align - 1u) & ~(ring_align - 1u);
  const uint32_t tab_abs = rings_abs + NW * args.ring_bytes;
  const uint32_t vals_abs = (tab_abs + ((args.table_words * 4u) << args.rep_log) + 1023u) & ~1023u;
  const uint32_t succ_abs = vals_abs + 1024u;             // private: u16 per state, (2 << max R) bytes
  const uint32_t bars_abs = succ_abs + args.succ_bytes;
  const uint32_t ring_abs = rings_abs + warp * args.ring_bytes;
  const uint32_t stage_abs = bars_abs + NW * 8u + warp * args.stage_bytes;
  uint2* tab = reinterpret_cast<uint2*>(sm + (tab_abs - sm_abs));
  // The table may sit in shared memory in several copies, entry i of copy c at slot i * copies + c.
  // A 64-bit load is served half a warp at a time over 16 bank pairs; with 16 copies every lane
  // of a half-warp has a bank pair of its own and random look-ups no longer collide.
  uint32_t* vals = reinterpret_cast<uint32_t*>(sm + (vals_abs - sm_abs));
  uint16_t* succ = reinterpret_cast<uint16_t*>(sm + (succ_abs - sm_abs));
  uint8_t* ring = sm + (ring_abs - sm_abs);
  uint8_t* stage = sm + (stage_abs - sm_abs);
  const uint32_t bar = bars_abs + warp * 8u;
  __shared__ uint32_t s_dom, s_maxadv;
  uint32_t parity = 0;

  uint64_t cursor = uint64_t(blockIdx.x) * args.items_per_cta;
  const uint64_t cta_end = min(cursor + uint64_t(args.items_per_cta), uint64_t(args.total_work));
  if (cursor >= cta_end) return;
  if (lane == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();

  int l = find_layer(args, cursor);
  uint32_t bad = 0;
  bool gave_up = false;
  const bool begins_in_params = args.n_begin == static_cast<uint32_t>(args.n_layers);
  for (; cursor < cta_end && l < args.n_layers; ++l) {
    const ans_layer_desc L = layer_at(args, l);           // one batch of loads, then registers
    const uint64_t lbeg = begins_in_params ? args.layer_begin[l] : L.work_begin, lend = lbeg + L.work_count;
    if (lend <= cursor) continue;                         // empty layer, or only its padding is left
    if (cursor < lbeg) cursor = lbeg;                     // past the padding after the layer before
    if (cursor >= cta_end) break;
    const uint64_t stop = min(lend, cta_end);
    const int R = L.table_log;
    // copies of this layer's table: a table smaller than the launch's largest uses the room for
    // more of them (the pre-walked walk keeps an extra entry after the table, so it does not)
    const uint32_t rep_log = (kPrivate && !lock) ? args.rep_log
                                                 : min(4u, args.rep_log + (args.max_log - static_cast<uint32_t>(R)));
    const uint32_t reps = 1u << rep_log;
    const uint32_t stride_log = 3u + rep_log;
    const uint32_t tab_lane = tab_abs + (lane & (reps - 1u)) * 8u;
    const uint8_t* blob = static_cast<const uint8_t*>(L.d_table);
    const TableHeader* hdr = reinterpret_cast<const TableHeader*>(blob);
    const uint32_t* g_single = reinterpret_cast<const uint32_t*>(blob + single_offset());
    // private: the pre-walked entries; interleaved: the plain ones (one symbol per look-up)
    const uint32_t* g_multi =
        (kPrivate && !lock) ? reinterpret_cast<const uint32_t*>(blob + multi_offset(R)) : g_single;
    const int dtype = args.d_symbols_override ? ANS_U8 : L.out_dtype;

    const size_t es = dtype == ANS_U8 ? 1 : dtype == ANS_F32 ? 4 : 2;
    const uint32_t W = L.lanes;
    const uint64_t n_sub = uint64_t(L.lanes / 32u) * ((L.n_symbols + L.chunk_symbols - 1) / L.chunk_symbols);

    auto warp_sub = [&](uint64_t gbase, uint64_t& sub) -> bool {
      const uint64_t granule = gbase + warp / kGranule;
      sub = (granule - lbeg) * kGranule + warp % kGranule;
      return granule < stop && sub < n_sub;
    };
    auto start_copy = [&](const Item& it) -> bool {       // true if the sub-stream is being staged
      const bool staged = it.extent > 0 && it.extent + kStagePad <= args.stage_bytes;
      if (staged) {
        __syncwarp();                                     // the last item's readers of the stage are done
        if (lane == 0) {
          const uint32_t bytes = static_cast<uint32_t>(it.extent);
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
          asm volatile(
              "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
              :: "r"(stage_abs), "l"(L.d_stream + it.off0), "r"(bytes), "r"(bar) : "memory");
        }
        for (uint32_t i = lane; i < kStagePad / 4u; i += 32u) reinterpret_cast<uint32_t*>(stage + it.extent)[i] = 0u;
      }
      return staged;
    };
    // Everything the layer's start needs from memory is requested here, before any of it is
    // used, so that it costs one trip and not one per item: the offsets and lane states of the
    // warp's first sub-stream, the table's header, the first batch of table entries.
    constexpr uint32_t kStageBatch = 16;
    const uint32_t n_states = 1u << R;
    auto load_meta = [&](uint64_t sub) -> uint32_t {
      if (kPrivate) return __ldg(static_cast<const uint32_t*>(L.d_lane_meta) + sub * 32 + lane);
      return __ldg(static_cast<const uint16_t*>(L.d_lane_meta) + sub * 32 + lane);
    };
    uint64_t first_sub = 0, first_off0 = 0, first_off1 = 0;
    uint32_t first_meta = 0;
    const bool have_first = warp_sub(cursor, first_sub);
    if (have_first) {
      first_off0 = __ldg(L.d_sub_offsets + first_sub);
      first_off1 = __ldg(L.d_sub_offsets + first_sub + 1);
      first_meta = load_meta(first_sub);
    }
    const uint32_t h_magic = __ldg(&hdr->magic), h_log = __ldg(&hdr->table_log), h_alphabet = __ldg(&hdr->alphabet),
                   h_dominant = __ldg(&hdr->dominant);
    uint32_t g[kStageBatch], g1[kStageBatch];
    auto request_entries = [&](uint32_t b0) {
#pragma unroll
      for (uint32_t k = 0; k < kStageBatch; ++k) {
        const uint32_t i = b0 + k * blockDim.x + threadIdx.x;
        g[k] = i < n_states ? __ldg(g_multi + i) : 0u;
        if (kPrivate && !lock) g1[k] = i < n_states ? __ldg(g_single + i) : 0u;
      }
    };
    request_entries(0);

    // The warp's first sub-stream of this layer: its bulk copy is started now so that it travels
    // while the table is being staged.
    Item first_item;
    bool first_staged = false;
    if (have_first) {
      first_item = make_item(L, first_sub, first_off0, first_off1);
      first_staged = start_copy(first_item);
    }

    __syncthreads();                                      // previous layer's readers of the table are done
    for (uint32_t b0 = 0; b0 < n_states; b0 += blockDim.x * kStageBatch) {
      if (b0 != 0) request_entries(b0);                   // a batch is requested whole before any entry is converted
      if (b0 == 0) {
        for (uint32_t i = threadIdx.x; i < 256u; i += blockDim.x)
          vals[i] = dequant_bits(static_cast<int>(i), L.zero_point, L.scale, dtype);
        if (threadIdx.x == 0) {
          s_dom = h_dominant < 256u ? h_dominant : 0u;    // the ring's fill symbol
          s_maxadv = 1u;
          if (h_magic != kTableMagic || h_log != uint32_t(R) || h_alphabet > (1u << L.bitwidth))
            bad |= ANS_STATUS_BAD_SYMBOL;
        }
        __syncthreads();
      }
      uint32_t longest = 0;
#pragma unroll
      for (uint32_t k = 0; k < kStageBatch; ++k) {
        const uint32_t i = b0 + k * blockDim.x + threadIdx.x;
        if (i < n_states) {
          const uint2 e = kQuads ? to_quads_entry(g[k], vals[entry_sym(g[k])], es != 4)
                                 : to_smem_entry(g[k], vals[entry_sym(g[k])], 32u * static_cast<uint32_t>(es));
          // every lane starts at another copy: the stores of a warp spread over the banks
          for (uint32_t c = 0; c < reps; ++c) tab[(i << rep_log) + ((c + lane) & (reps - 1u))] = e;
          if (kPrivate && !lock) succ[i] = static_cast<uint16_t>(entry_newx(g1[k]));
          longest = max(longest, entry_run(g[k]) + 1u);
        }
      }
      longest = __reduce_max_sync(kFull, longest);
      if (lane == 0 && longest > 1u) atomicMax(&s_maxadv, longest);
    }
    if (threadIdx.x < reps && kPrivate && !lock && R <= kMaxParkLog)
      tab[(n_states << rep_log) + threadIdx.x] =
          make_uint2(n_states << 17, es == 4 ? vals[s_dom] : (vals[s_dom] & 0xFFFFu));
    __syncthreads();

    uint8_t* out_base = args.d_symbols_override ? args.d_symbols_override : static_cast<uint8_t*>(L.d_out);
    const uint32_t dom = vals[s_dom];
    const uint32_t park_abs = R <= kMaxParkLog ? tab_lane + ((n_states << stride_log)) : 0u;
    for (uint64_t gbase = cursor; gbase < stop && !gave_up; gbase += NW / kGranule) {
      uint64_t sub;
      if (!warp_sub(gbase, sub)) continue;
      const bool is_first = gbase == cursor;              // its copy is already under way
      uint64_t off0 = 0, off1 = 0;
      uint32_t meta = first_meta;
      if (!is_first) {                                    // offsets and lane states in one trip
        off0 = __ldg(L.d_sub_offsets + sub);
        off1 = __ldg(L.d_sub_offsets + sub + 1);
        meta = load_meta(sub);
      }
      const Item it = is_first ? first_item : make_item(L, sub, off0, off1);
      uint32_t wbad = it.bad;
      const uint32_t lambda = 32u * it.g + lane;
      // round-robin containers: symbols of this lane, rows of the sub-stream, rows all 32 lanes have.
      // quads: symbols of this lane; rows / min_count count the turns some / all lanes own a whole quad in
      uint32_t my_count, rows, min_count;
      if (kQuads) {
        const uint32_t full = it.nc >> 2, rem = it.nc & 3u;
        my_count = 4u * lane_symbols(full, W, lambda) + ((rem && full % W == lambda) ? rem : 0u);
        rows = lane_symbols(full, W, 32u * it.g);
        min_count = lane_symbols(full, W, 32u * it.g + 31u);
      } else {
        my_count = lane_symbols(it.nc, W, lambda);
        rows = lane_symbols(it.nc, W, 32u * it.g);
        min_count = lane_symbols(it.nc, W, 32u * it.g + 31u);
      }
      const uint32_t ext_words = static_cast<uint32_t>(min(it.extent / 4, uint64_t(0x3FFFFFFFu)));
      const uint8_t* g_bytes = L.d_stream + it.off0;
      const bool staged = is_first ? first_staged : start_copy(it);

      // row 0 of this sub-stream (quads: a row holds four elements per lane)
      uint8_t* out_row0 = out_base + (it.c0 + (kQuads ? 128u : 32u) * it.g) * es;
      const size_t rsb = size_t(W) * es;
      uint32_t state, wbeg = 0, wend = 0;
      if (kPrivate) {
        state = meta & ((1u << R) - 1u);
        wbeg = meta >> 16;
        wend = __shfl_down_sync(kFull, wbeg, 1);
        if (lane == 31) wend = ext_words;
        if (wend > ext_words) { wend = ext_words; wbad |= ANS_STATUS_BAD_LENGTH; }
        if (wbeg > wend) { wbeg = wend; wbad |= ANS_STATUS_BAD_LENGTH; }
      } else {
        state = meta & ((1u << R) - 1u);
      }

      if (staged) {
        const bool ok = mbar_wait(bar, parity);
        parity ^= 1u;
        if (!__all_sync(kFull, ok)) {                     // the copy never landed: stop this warp's work
          bad |= wbad | kStatusTimeout;
          gave_up = true;
          continue;
        }
        __syncwarp();
      }
      if (kPrivate) {
        const uint32_t* words = reinterpret_cast<const uint32_t*>(g_bytes);
#define ANSB_CALL(ES_, ST_)                                                                              \
  wbad |= decode_private<ES_, ST_>(tab_lane, stride_log, succ_abs, ring_abs, stage_abs, park_abs, ring, dom, words, \
                                   ext_words, wbeg, wend, lane == 31, state, my_count, rows, min_count, \
                                   out_row0, rsb, lane, s_maxadv)
#define ANSB_LCALL(ES_, ST_)                                                                             \
  wbad |= decode_lockstep<ES_, ST_>(tab_lane, stride_log, stage_abs, words, ext_words, wbeg, wend, lane == 31, \
                                    state, my_count, rows, min_count, out_row0, W / 32u, lane, R <= 8, args.unit)
#define ANSB_QCALL(ES_, ST_)                                                                             \
  wbad |= decode_quads<ES_, ST_>(tab_lane, stride_log, stage_abs, words, ext_words, wbeg, wend, lane == 31, state, \
                                 my_count, min_count, out_row0 + size_t(lane) * 4u * ES_, W / 32u, R <= 8, args.unit)
        if constexpr (kQuads) {
          if (staged) {
            if (es == 1) ANSB_QCALL(1, true); else if (es == 2) ANSB_QCALL(2, true); else ANSB_QCALL(4, true);
          } else {
            if (es == 1) ANSB_QCALL(1, false); else if (es == 2) ANSB_QCALL(2, false); else ANSB_QCALL(4, false);
          }
        } else if constexpr (lock) {
          if (staged) {
            if (es == 1) ANSB_LCALL(1, true); else if (es == 2) ANSB_LCALL(2, true); else ANSB_LCALL(4, true);
          } else {
            if (es == 1) ANSB_LCALL(1, false); else if (es == 2) ANSB_LCALL(2, false); else ANSB_LCALL(4, false);
          }
        } else {
          if (staged) {
            if (es == 1) ANSB_CALL(1, true); else if (es == 2) ANSB_CALL(2, true); else ANSB_CALL(4, true);
          } else {
            if (es == 1) ANSB_CALL(1, false); else if (es == 2) ANSB_CALL(2, false); else ANSB_CALL(4, false);
          }
        }
#undef ANSB_QCALL
#undef ANSB_LCALL
#undef ANSB_CALL
      } else {
        const uint16_t* units = reinterpret_cast<const uint16_t*>(g_bytes);
        const uint32_t unit_cap = ext_words * 2u;
#define ANSB_CALL(ES_, ST_)                                                                              \
  wbad |= decode_interleaved<ES_, ST_>(tab_lane, stride_log, stage_abs, units, unit_cap, state, my_count, rows, \
                                       min_count, out_row0, rsb, lane)
        if (staged) {
          if (es == 1) ANSB_CALL(1, true); else if (es == 2) ANSB_CALL(2, true); else ANSB_CALL(4, true);
        } else {
          if (es == 1) ANSB_CALL(1, false); else if (es == 2) ANSB_CALL(2, false); else ANSB_CALL(4, false);
        }
#undef ANSB_CALL
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
constexpr int kMaxDevices = 64;
struct LaunchShape { size_t smem = 0; int warps = 0; int per_sm = 0; };
struct DeviceFacts { int sms = 0; int smem_max = 0; LaunchShape shape[8]; };
static DeviceFacts g_facts[kMaxDevices];    // remembered per device; racing writers store equal values

static int launch(const ans_layer_desc* d_descs, const ans_layer_desc* h_descs, int n_layers,
                  uint8_t* d_symbols_override, uint32_t* d_status, cudaStream_t st) {
  int max_log = 1, busy_layers = 0;
  uint64_t total = 0;
  size_t max_avg_sub = 0, max_es = 1;
  const int layout = h_descs[0].layout;
  for (int l = 0; l < n_layers; ++l) {
    const int rc = validate_desc(h_descs[l], d_symbols_override == nullptr);
    if (rc != ANS_OK) return rc;
    if (h_descs[l].layout != layout) return ANS_ERR_UNSUPPORTED;
    if (h_descs[l].work_begin != total || h_descs[l].work_count != granules_of(h_descs[l]))
      return ANS_ERR_INVALID_ARG;                         // ans_plan_batch was not run on this array
    total += h_descs[l].work_count;
    if (h_descs[l].work_count != 0) {
      ++busy_layers;
      const size_t avg = h_descs[l].stream_bytes / subs_of(h_descs[l]);
      if (avg > max_avg_sub) max_avg_sub = avg;
      const size_t es = d_symbols_override ? 1 : elem_size(h_descs[l].out_dtype);
      if (es > max_es) max_es = es;
    }
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
  a.unit = 1u;
  a.max_log = static_cast<uint32_t>(max_log);
  a.table_words = 2u * ((1u << max_log) + 2u);           // two words per state, and a parking entry (one copy)

  // device facts and per-configuration occupancy are looked up once and remembered (plain values,
  // no allocation): a launch of a small model should not spend its time in attribute queries
  int dev = 0, sms = 0, per_sm = 0, smem_max = 0;
  ANSB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ANS_ERR_UNSUPPORTED;
  DeviceFacts& facts = g_facts[dev];
  if (!facts.sms) {
    ANSB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ANSB_CUDA(cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    facts.smem_max = smem_max;
    facts.sms = sms;
  }
  sms = facts.sms;
  smem_max = facts.smem_max;

  const bool quads = layout == ANS_LAYOUT_QUADS;
  const bool priv = layout != ANS_LAYOUT_INTERLEAVED;
  // Layers with many sub-streams share one table among many warps; a model of many small
  // layers runs CTAs of one granule (4 warps) so that each CTA stays inside one layer and
  // several CTAs, each with its own table, share an SM.
  const bool big = total / uint64_t(busy_layers) >= 64;
  // Private container, large layers: tables of up to 512 states (the paper's coder has 256) fit
  // shared memory in many conflict-free copies beside 28 warps' staging buffers, which makes
  // the one-symbol-per-look-up walk the faster one (measured); larger tables, and models of
  // small layers, are walked through the pre-walked entries.
  const bool lock = quads || (priv && big && max_log <= kLockstepMaxLog);
  int warps = 4, launch_which = 0;
  a.succ_bytes = (priv && !lock) ? ((2u << max_log) + 15u) & ~15u : 0u;
  size_t smem = (size_t(a.table_words) + 256) * 4 + a.succ_bytes;
  {
    // per warp: an output ring of kRingRows rows of the widest dtype, and a staging buffer for
    // the largest layer-average sub-stream plus a margin (a longer one is read from global memory)
    // only the pre-walked walk buffers its output; the others store rows straight to it
    const bool direct = lock || !priv;
    const size_t ring = direct ? 0 : size_t(kRingRows) * 32 * max_es;
    size_t want = max_avg_sub + max_avg_sub / 16 + 256 + kStagePad;
    want = (want + 127) & ~size_t(127);
    const size_t fixed = ring + 1024 + smem + 32 * 8;     // alignment slack, table, vals, barriers
    // warps that store straight to the output need few registers and no ring: up to 28 of them,
    // leaving room for the copies
    // (tables of up to 512 states get all 16 copies, which pays for the warps they displace;
    // larger ones about 33 KB in all: 4 copies of 1024 states, ..., 1 from 4096 up; measured)
    const size_t one = size_t(a.table_words) * 4;
    const size_t copies_room = !direct ? 0 : max_log <= 9 ? one * 15
                               : one < (size_t(33) << 10) ? (size_t(33) << 10) - one : 0;
    warps = big ? (direct ? 28 : 16) : 4;
    // a model of small layers that would not fit one wave of 4-warp CTAs (three per SM): the
    // lockstep kernels, light on registers, take two granules side by side rather than in turn
    if (!big && lock && total > uint64_t(3) * sms) warps = 8;
    while (warps > 4 && fixed + copies_room + size_t(warps) * (ring + want) + 1024 > size_t(smem_max)) warps -= 4;
    while (warps > 4 && fixed + size_t(warps) * (ring + want) + 1024 > size_t(smem_max)) warps -= 4;
    const size_t room = size_t(smem_max) > fixed + size_t(warps) * ring + 1024
                            ? (size_t(smem_max) - fixed - size_t(warps) * ring - 1024) / warps : 0;
    size_t stage = (want < room ? want : room) & ~size_t(15);
    if (stage < 256) stage = 0;
    a.stage_bytes = static_cast<uint32_t>(stage);
    a.ring_bytes = static_cast<uint32_t>(ring);
    smem = fixed + size_t(warps) * (ring + stage);
    // Shared memory left over goes to extra copies of the table (fewer bank conflicts on the
    // random look-ups; 16 copies make them conflict-free).  Small CTAs must stay small enough
    // for three of them to share an SM.
    const size_t one_table = size_t(a.table_words) * 4;
    const size_t cap = big ? size_t(smem_max) : size_t(74) << 10;
    while (a.rep_log < 4 && smem + (one_table << a.rep_log) <= cap) {
      smem += one_table << a.rep_log;                     // doubling the copies adds as many again
      ++a.rep_log;
    }
  }
  {
    // which instantiation: the walk, and whether the CTA is one of many warps
    const bool many = warps > 16;
    const int which = (quads ? 0 : lock ? 1 : priv ? 2 : 3) * 2 + (many ? 1 : 0);
    const void* fn = nullptr;
    switch (which) {
      case 0: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_QUADS, true, false>); break;
      case 1: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_QUADS, true, true>); break;
      case 2: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, true, false>); break;
      case 3: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, true, true>); break;
      case 4: case 5: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, false, false>); break;
      case 6: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_INTERLEAVED, true, false>); break;
      default: fn = reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_INTERLEAVED, true, true>); break;
    }
    launch_which = which;
    LaunchShape& shape = facts.shape[which];
    if (shape.smem != smem || shape.warps != warps) {
      ANSB_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
      ANSB_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, warps * 32, smem));
      shape.smem = smem;
      shape.warps = warps;
      shape.per_sm = per_sm;
    }
    per_sm = shape.per_sm;
  }
  if (per_sm < 1) return ANS_ERR_UNSUPPORTED;
  const uint64_t step = uint64_t(warps) / kGranule;       // granules a CTA takes at a time
  if (n_layers <= kParamLayers) {
    // every layer starts on a multiple of `step` in the numbering the CTAs walk: a CTA that meets
    // a new layer starts it with a full round of warps instead of finishing a ragged one first
    a.n_begin = static_cast<uint32_t>(n_layers);
    uint64_t padded = 0;
    for (int l = 0; l < n_layers; ++l) {
      a.layer_begin[l] = static_cast<uint32_t>(padded);
      padded += (uint64_t(h_descs[l].work_count) + step - 1) / step * step;
    }
    if (padded > 0xFFFFFFFFull) return ANS_ERR_UNSUPPORTED;
    total = padded;
    a.total_work = static_cast<uint32_t>(total);
  }
  const uint64_t want_ctas = (total + step - 1) / step;
  const uint64_t grid = want_ctas < uint64_t(sms) * per_sm ? want_ctas : uint64_t(sms) * per_sm;
  uint64_t ipc = (total + grid - 1) / grid;
  ipc = (ipc + step - 1) / step * step;
  a.items_per_cta = static_cast<uint32_t>(ipc);
  const unsigned blocks = static_cast<unsigned>((total + ipc - 1) / ipc);
  const dim3 grid_dim(blocks), block_dim(static_cast<unsigned>(warps) * 32u);
  switch (launch_which) {
    case 0: ans_decode_kernel<ANS_LAYOUT_QUADS, true, false><<<grid_dim, block_dim, smem, st>>>(a); break;
    case 1: ans_decode_kernel<ANS_LAYOUT_QUADS, true, true><<<grid_dim, block_dim, smem, st>>>(a); break;
    case 2: ans_decode_kernel<ANS_LAYOUT_PRIVATE, true, false><<<grid_dim, block_dim, smem, st>>>(a); break;
    case 3: ans_decode_kernel<ANS_LAYOUT_PRIVATE, true, true><<<grid_dim, block_dim, smem, st>>>(a); break;
    case 4: case 5: ans_decode_kernel<ANS_LAYOUT_PRIVATE, false, false><<<grid_dim, block_dim, smem, st>>>(a); break;
    case 6: ans_decode_kernel<ANS_LAYOUT_INTERLEAVED, true, false><<<grid_dim, block_dim, smem, st>>>(a); break;
    default: ans_decode_kernel<ANS_LAYOUT_INTERLEAVED, true, true><<<grid_dim, block_dim, smem, st>>>(a); break;
  }
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
    const uint64_t n = granules_of(d);
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
