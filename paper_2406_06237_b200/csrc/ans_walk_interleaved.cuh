// Interleaved container (ans_decode.cu includes this).
#pragma once

#include "ans_decode_common.cuh"

namespace ansb {

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

}  // namespace ansb
