// The walk of the strips container's kernels: shared-memory forms of a pre-walked table entry and
// the PTX loop that walks one window of a sub-stream (ans_decode_strips.cu and
// ans_fused_gemm.cu include this).
#pragma once

#include "ans_decode_common.cuh"

namespace ansb {

// shared-memory form of a pre-walked entry.  Two words:
//   1- and 2-byte outputs:  a = nb [4:0] | run [11:8] | value [31:16]    b = q
//   4-byte outputs:         a = nb [4:0] | run [11:8] | q [31:16]        b = value
// q = newX >> nb, so that the next state is (q << nb) | bits: one funnel shift on a bit window
// that is kept top-aligned.  Bits 5-7 of a stay zero: the walk adds all of a to its bit count.
// Or ONE word, for tables of up to 256 states (the paper's sizes) and 1- or 2-byte outputs:
//   value [15:0] | nb [19:16] | run [23:20] | q [31:24]
// Half the bytes, so twice the copies fit and a look-up takes fewer shared-memory wavefronts,
// for one more instruction (the fields have to be cut out; the value is stored as it lies).
__device__ __forceinline__ uint2 to_strip_entry(uint32_t g, uint32_t val, bool narrow) {
  const uint32_t nb = entry_nb(g), q = entry_newx(g) >> nb, run = entry_run(g);
  return narrow ? make_uint2(nb | (run << 8) | (val << 16), q) : make_uint2(nb | (run << 8) | (q << 16), val);
}
__device__ __forceinline__ uint32_t to_strip_entry_short(uint32_t g, uint32_t val) {
  const uint32_t nb = entry_nb(g);
  return (val & 0xFFFFu) | (nb << 16) | (entry_run(g) << 20) | ((entry_newx(g) >> nb) << 24);
}

#define ANSB_SP_BEGIN "shf.l.wrap.b32 x, %3, %2, %1;\n\t"
#define ANSB_SP_END                                               \
  "and.b32 tt, %1, 32;\n\t"                                       \
  "setp.ne.u32 pq, tt, 0;\n\t"                                    \
  "@pq mov.u32 %2, %3;\n\t"                                       \
  "@pq mov.u32 %3, %4;\n\t"                                       \
  "@pq ld.shared.u32 %4, [%5];\n\t"                               \
  "@pq add.u32 %5, %5, 4;\n\t"                                    \
  "and.b32 %1, %1, 31;\n\t"
// One look-up.  %6: the lane's next position; zn: the position of the symbol that ends the run;
// the lane takes the step only if that position is inside the window (and the lane), else it
// keeps its state and waits.
#define ANSB_SP_STEP_N(STS_, ADDR_)                                      \
  "ld.shared.v2.u32 {ea, eb}, [%0];\n\t"                          \
  "bfe.u32 av, ea, 8, 4;\n\t"                                     \
  "add.u32 zn, %6, av;\n\t"                                       \
  "setp.lt.u32 act, zn, %10;\n\t"                                 \
  ADDR_                                                           \
  "shr.u32 vv, ea, 16;\n\t"                                       \
  "@act " STS_ " [ad], vv;\n\t"                                   \
  "@act shf.l.wrap.b32 tt, x, eb, ea;\n\t"                        \
  "@act shf.l.wrap.b32 x, 0, x, ea;\n\t"                          \
  "@act mad.lo.u32 %0, tt, %8, %7;\n\t"                           \
  "@act mad.lo.u32 %1, ea, %11, %1;\n\t"                          \
  "@act add.u32 %6, zn, 1;\n\t"
#define ANSB_SP_STEP_S(STS_, ADDR_)                                      \
  "ld.shared.u32 ea, [%0];\n\t"                                   \
  "bfe.u32 av, ea, 20, 4;\n\t"                                    \
  "add.u32 zn, %6, av;\n\t"                                       \
  "setp.lt.u32 act, zn, %10;\n\t"                                 \
  ADDR_                                                           \
  "@act " STS_ " [ad], ea;\n\t"                                   \
  "bfe.u32 eb, ea, 16, 4;\n\t"                                    \
  "shr.u32 av, ea, 24;\n\t"                                       \
  "@act shf.l.wrap.b32 tt, x, av, eb;\n\t"                        \
  "@act shf.l.wrap.b32 x, 0, x, eb;\n\t"                          \
  "@act mad.lo.u32 %0, tt, %8, %7;\n\t"                           \
  "@act add.u32 %1, %1, eb;\n\t"                                  \
  "@act add.u32 %6, zn, 1;\n\t"
#define ANSB_SP_STEP_W(STS_, ADDR_)                                      \
  "ld.shared.v2.u32 {ea, eb}, [%0];\n\t"                          \
  "bfe.u32 av, ea, 8, 4;\n\t"                                     \
  "add.u32 zn, %6, av;\n\t"                                       \
  "setp.lt.u32 act, zn, %10;\n\t"                                 \
  ADDR_                                                           \
  "shr.u32 vv, ea, 16;\n\t"                                       \
  "@act " STS_ " [ad], eb;\n\t"                                   \
  "@act shf.l.wrap.b32 tt, x, vv, ea;\n\t"                        \
  "@act shf.l.wrap.b32 x, 0, x, ea;\n\t"                          \
  "@act mad.lo.u32 %0, tt, %8, %7;\n\t"                           \
  "@act mad.lo.u32 %1, ea, %11, %1;\n\t"                          \
  "@act add.u32 %6, zn, 1;\n\t"

// where the symbol at position zn goes in the window.  Strips: a row is one symbol of every lane.
// Channels: a row is one piece of E symbols of every lane; zn / E by a multiplication (%15 =
// 2^32 / E rounded up, exact for positions below 2^32 / E), %16 = 31 * E * ES.
#define ANSB_SP_ADDR_STRIPS "mad.lo.u32 ad, zn, %13, %9;\n\t"
#define ANSB_SP_ADDR_PIECES                                       \
  "mul.hi.u32 tt, zn, %15;\n\t"                                   \
  "mad.lo.u32 ad, tt, %16, %9;\n\t"                               \
  "mad.lo.u32 ad, zn, %14, ad;\n\t"

// The walk of one window, entirely in PTX (loop included).  Groups of K look-ups share one
// 32-bit extract of the bit window and one refill check: K = 4 when no state of the table takes
// more than 8 bits, else 2.  The loop ends when no lane took the last look-up of a group; every
// look-up a lane takes moves its position on, so a window costs at most its symbols in trips.
//   st: shared address of the state's entry      z: the lane's next position (symbols it has decoded)
//   abase: window address of the lane's first symbol, minus the window's first row (a row holds one
//          symbol of every lane)
//   lim: first position the lane may not write (end of the window, or of the lane)
template <int ES, int K, bool SHORT, bool PIECES>
__device__ __forceinline__ void strip_window_walk(uint32_t& st, uint32_t& bitpos, uint32_t& w0, uint32_t& w1,
                                                  uint32_t& w2, uint32_t& sp, uint32_t& z, uint32_t tab_lane,
                                                  uint32_t stride, uint32_t abase, uint32_t lim, uint32_t unit,
                                                  uint32_t sp_limit, uint32_t magic, uint32_t row_skip) {
#define ANSB_SP_ASM(LBL_, BODY_, MORE_)                                                     \
  asm volatile(                                                                             \
      "{\n\t"                                                                               \
      ".reg .pred act, pq, pany;\n\t"                                                       \
      ".reg .u32 x, ea, eb, av, zn, tt, ad, vv, nw;\n"                                      \
      LBL_ ":\n\t"                                                                          \
      BODY_                                                                                 \
      "vote.sync.any.pred pany, act, 0xffffffff;\n\t"                                       \
      "@pany bra " LBL_ ";\n\t"                                                             \
      "min.u32 %5, %5, %12;\n\t"                                                            \
      "}"                                                                                   \
      : "+r"(st), "+r"(bitpos), "+r"(w0), "+r"(w1), "+r"(w2), "+r"(sp), "+r"(z)             \
      : "r"(tab_lane), "r"(stride), "r"(abase), "r"(lim), "r"(unit), "r"(sp_limit),         \
        "n"(32 * ES), "n"(ES) MORE_()                                                       \
      : "memory")
#define ANSB_SP_G4(ST_, STS_, AD_) ANSB_SP_BEGIN ST_(STS_, AD_) ST_(STS_, AD_) ST_(STS_, AD_) ST_(STS_, AD_) ANSB_SP_END
#define ANSB_SP_G2(ST_, STS_, AD_) ANSB_SP_BEGIN ST_(STS_, AD_) ST_(STS_, AD_) ANSB_SP_END
#define ANSB_SP_NONE()
#define ANSB_SP_PIECE_OPS() , "r"(magic), "r"(row_skip)
#define ANSB_SP_ALL(AD_, P_, MORE_)                                                              \
  if (SHORT) {                                             /* (tables of up to 256 states: no state takes more than 8 bits) */ \
    if (ES == 1) ANSB_SP_ASM("ANSB_SPS1" P_, ANSB_SP_G4(ANSB_SP_STEP_S, "st.shared.u8", AD_), MORE_);     \
    if (ES == 2) ANSB_SP_ASM("ANSB_SPS2" P_, ANSB_SP_G4(ANSB_SP_STEP_S, "st.shared.u16", AD_), MORE_);    \
  } else if (K == 4) {                                                                           \
    if (ES == 1) ANSB_SP_ASM("ANSB_SP41" P_, ANSB_SP_G4(ANSB_SP_STEP_N, "st.shared.u8", AD_), MORE_);     \
    if (ES == 2) ANSB_SP_ASM("ANSB_SP42" P_, ANSB_SP_G4(ANSB_SP_STEP_N, "st.shared.u16", AD_), MORE_);    \
    if (ES == 4) ANSB_SP_ASM("ANSB_SP44" P_, ANSB_SP_G4(ANSB_SP_STEP_W, "st.shared.u32", AD_), MORE_);    \
  } else {                                                                                       \
    if (ES == 1) ANSB_SP_ASM("ANSB_SP21" P_, ANSB_SP_G2(ANSB_SP_STEP_N, "st.shared.u8", AD_), MORE_);     \
    if (ES == 2) ANSB_SP_ASM("ANSB_SP22" P_, ANSB_SP_G2(ANSB_SP_STEP_N, "st.shared.u16", AD_), MORE_);    \
    if (ES == 4) ANSB_SP_ASM("ANSB_SP24" P_, ANSB_SP_G2(ANSB_SP_STEP_W, "st.shared.u32", AD_), MORE_);    \
  }
  if (PIECES) { ANSB_SP_ALL(ANSB_SP_ADDR_PIECES, "P", ANSB_SP_PIECE_OPS) } else { ANSB_SP_ALL(ANSB_SP_ADDR_STRIPS, "", ANSB_SP_NONE) }
#undef ANSB_SP_ALL
#undef ANSB_SP_PIECE_OPS
#undef ANSB_SP_NONE
#undef ANSB_SP_G2
#undef ANSB_SP_G4
#undef ANSB_SP_ASM
}

__device__ __forceinline__ uint4 lds_v4(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts_v4(uint32_t a, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" :: "r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

}  // namespace ansb
