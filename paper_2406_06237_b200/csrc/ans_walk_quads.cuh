// Quads container (ans_decode.cu includes this).
#pragma once

#include "ans_walk_lockstep.cuh"   // shares the refill macro

namespace ansb {

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
// or, for 1-byte outputs, ONE word: nb [4:0] | q [21:8] | value [31:24].  Half the bytes per
// table, so twice the copies fit: it pays where copies are short (tables of 2^11 states and up,
// whose random look-ups collide), at the price of one more instruction per look-up.
// 2-byte outputs have a one-word form too, for tables of 2^10 to 2^12 states:
// nb [3:0] | q [15:4] | value [31:16] (two more instructions per look-up, half the wavefronts).
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
#define ANSB_QD_STEP_S(I_)                                        \
  "ld.shared.u32 ea" I_ ", [%0];\n\t"                             \
  "bfe.u32 nx, ea" I_ ", 8, 14;\n\t"                              \
  "shf.l.wrap.b32 t, x, nx, ea" I_ ";\n\t"                        \
  "shf.l.wrap.b32 x, 0, x, ea" I_ ";\n\t"                         \
  "mad.lo.u32 %0, t, %7, %6;\n\t"                                 \
  "mad.lo.u32 %1, ea" I_ ", %9, %1;\n\t"
#define ANSB_QD_STEP_S2(I_)                                       \
  "ld.shared.u32 ea" I_ ", [%0];\n\t"                             \
  "and.b32 nbb, ea" I_ ", 15;\n\t"                                \
  "bfe.u32 nx, ea" I_ ", 4, 12;\n\t"                              \
  "shf.l.wrap.b32 t, x, nx, nbb;\n\t"                            \
  "shf.l.wrap.b32 x, 0, x, nbb;\n\t"                             \
  "mad.lo.u32 %0, t, %7, %6;\n\t"                                 \
  "add.u32 %1, %1, nbb;\n\t"
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
// (the stores carry the streaming hint: an output line is written once and not read again by
// this kernel, and evicting it first leaves L2 to the compressed bytes and to the other writes)
#define ANSB_QD_OUT1(A_)                                          \
  "prmt.b32 v0, ea0, ea1, 0x0062;\n\t"                            \
  "prmt.b32 v1, ea2, ea3, 0x0062;\n\t"                            \
  "prmt.b32 v0, v0, v1, 0x5410;\n\t"                              \
  "st.global.cs.u32 " A_ ", v0;\n\t"
#define ANSB_QD_OUT1S(A_)                                         \
  "prmt.b32 v0, ea0, ea1, 0x0073;\n\t"                            \
  "prmt.b32 v1, ea2, ea3, 0x0073;\n\t"                            \
  "prmt.b32 v0, v0, v1, 0x5410;\n\t"                              \
  "st.global.cs.u32 " A_ ", v0;\n\t"
#define ANSB_QD_OUT2(A_)                                          \
  "prmt.b32 v0, ea0, ea1, 0x7632;\n\t"                            \
  "prmt.b32 v1, ea2, ea3, 0x7632;\n\t"                            \
  "st.global.cs.v2.u32 " A_ ", {v0, v1};\n\t"
#define ANSB_QD_OUT4(A_) "st.global.cs.v4.u32 " A_ ", {eb0, eb1, eb2, eb3};\n\t"

constexpr uint32_t kQuadTurns = 4;     // turns (of four symbols per lane) per trip of the PTX loop

// The hot loop of the quads container: `blocks` times kQuadTurns turns, entirely in PTX (loop
// included, so that nothing is carried through the compiler between trips).  Operands as in
// lockstep_block; gp: this lane's four elements of the first turn; turns are 128 * ES * groups
// bytes apart (immediate offsets when groups == 1); sp is held at sp_limit if a corrupt stream
// drives it that far.
template <int ES, int K, bool SHORT = false>
__device__ __forceinline__ void quads_loop(uint32_t& st, uint32_t& bitpos, uint32_t& w0, uint32_t& w1,
                                           uint32_t& w2, uint32_t& sp, uint32_t tab_lane, uint32_t stride,
                                           uint8_t* gp, uint32_t unit, uint32_t groups, uint32_t blocks,
                                           uint32_t sp_limit) {
  constexpr uint32_t RS = 128u * ES;
#define ANSB_QD_ASM1(LBL_, TURN_, ST_, OUT_)                                                \
  asm volatile(                                                                             \
      "{\n\t"                                                                               \
      ".reg .pred q;\n\t"                                                                   \
      ".reg .u32 x, t, nx, nbb, nw, v0, v1, cnt, ea0, ea1, ea2, ea3, eb0, eb1, eb2, eb3;\n\t" \
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
      ".reg .u32 x, t, nx, nbb, nw, v0, v1, cnt, ea0, ea1, ea2, ea3, eb0, eb1, eb2, eb3;\n\t" \
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
  if (SHORT && ES == 2) {     // one-word entries, 2-byte outputs
    if (K == 4) { ANSB_QD_BOTH("ANSB_QT41", "ANSB_QT4G", ANSB_QD_TURN4, ANSB_QD_STEP_S2, ANSB_QD_OUT2); }
    else { ANSB_QD_BOTH("ANSB_QT21", "ANSB_QT2G", ANSB_QD_TURN2, ANSB_QD_STEP_S2, ANSB_QD_OUT2); }
  } else if (SHORT) {     // one-word entries, 1-byte outputs
    if (K == 4) { ANSB_QD_BOTH("ANSB_QS41", "ANSB_QS4G", ANSB_QD_TURN4, ANSB_QD_STEP_S, ANSB_QD_OUT1S); }
    else { ANSB_QD_BOTH("ANSB_QS21", "ANSB_QS2G", ANSB_QD_TURN2, ANSB_QD_STEP_S, ANSB_QD_OUT1S); }
  } else if (K == 4) {
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
template <int ES, bool STAGED, bool SHORT = false>
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
      if (wide_steps) quads_loop<ES, 4, SHORT>(st, bitpos, w0, w1, w2, sp, tab_abs, 1u << stride_log, out_lane, unit,
                                               groups, blocks, sp_limit);
      else quads_loop<ES, 2, SHORT>(st, bitpos, w0, w1, w2, sp, tab_abs, 1u << stride_log, out_lane, unit, groups,
                                    blocks, sp_limit);
      if (sp >= sp_limit) overran = true;
      turn = blocks * kQuadTurns;
    }
    idx = (sp - stage_abs) >> 2;
    k = 4u * turn;
  }
  // the rest in plain code, one symbol and one element store at a time
  for (; k < my_count; ++k) {
    const uint32_t ea = lds_u32(st), eb = SHORT ? 0u : lds_u32(st + 4u);
    constexpr bool SHORT2 = SHORT && ES == 2;
    const uint32_t nb = SHORT2 ? ea & 15u : ea & 31u;
    const uint32_t q = SHORT2 ? (ea >> 4) & 0xFFFu : SHORT ? (ea >> 8) & 0x3FFFu : NARROW ? eb : ea >> 8;
    const uint32_t val = SHORT2 ? ea >> 16 : SHORT ? ea >> 24 : NARROW ? ea >> 16 : eb;
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

}  // namespace ansb
