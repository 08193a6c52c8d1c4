// Private container walked one symbol per look-up (ans_decode.cu includes this).
#pragma once

#include "ans_decode_common.cuh"

namespace ansb {

// =============================================================================================
// Private container, lockstep walk: every look-up emits exactly one symbol (the plain table of
// Section II-A), so the 32 lanes of a warp stay on the same output row.  A row is complete as
// soon as it is decoded and each lane stores its element straight to the output: a row is
// 32 * ES contiguous bytes, whole 32-byte sectors; no ring, no pre-fill, no parking, no tail.
// The price is one look-up per symbol, which pays when look-ups are cheap (a table small enough
// for conflict-free copies) or the pre-walked entries would stand for few symbols anyway.
//
// kFlushRows rows are decoded by one PTX block (row stores at immediate offsets), K look-ups
// sharing one 32-bit extract of the bit window and one refill check: K = 4 when no state of the
// table takes more than 8 bits, else 2.  Multiply-high is avoided on purpose (it runs at a
// fraction of the rate of shifts and adds); the bit count is accumulated on the multiply-add
// pipe, which is otherwise idle, by a multiplication with a run-time 1.
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
  "@q ld.shared.u32 %4, [%5];\n\t"                                \
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

}  // namespace ansb
