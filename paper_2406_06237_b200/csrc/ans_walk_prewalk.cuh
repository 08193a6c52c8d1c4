// Private container walked through its pre-walked entries (ans_decode.cu includes this).
#pragma once

#include "ans_decode_common.cuh"

namespace ansb {

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
      "@q ld.shared.u32 %5, [%6];\n\t"                                                     \
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

}  // namespace ansb
