// Decode fused into its consumer: Y = X * W^T with W read in compressed form, for sm_100a.
//
// Paper Section I and Section III-C: the weights stay compressed in memory and are decompressed
// just before the computation that uses them, so that the decoded weights never travel to or from
// DRAM.  Here the consumer is a bf16 matrix product on the 5th-generation tensor cores: a CTA
// decodes 64 x 64 blocks of W (tANS states of a sub-stream's 32 lanes walked in step, Section
// II-A; dequantised to bf16, Section II-B) straight into shared memory in the layout
// tcgen05.mma reads its B operand from, and multiplies them with the matching 128 x 64 slices
// of X into a 128 x 64 fp32 accumulator in tensor memory.
//
// W (N x K, row n = output feature) must be stored for this call in blocks of 64 x 64:
// block (n / 64, k / 64) is 4096 consecutive symbols, blocks ordered [N / 64][K / 64]; coded in
// the strips container with chunk_symbols = 4096 and 32 lanes, so that one sub-stream is one
// block.  Inside a block the symbols lie in the order the tensor core reads the tile from shared
// memory (rows of 64, the eight 8-element pieces of row r exchanged by r mod 8: tile_offset
// below), so that symbol q of the block is simply the q-th bf16 of the tile.  X is M x K bf16 row-major, M <= 128; Y is
// M x N fp32 row-major.
//
// One CTA per block row of W (64 output features).  Warps 0-3 produce: warp w takes the blocks
// k / 64 = w, w + 4, ... of its block row, copies the slice of X and decodes the block of W into
// stage w, and hands the stage over through an mbarrier; warp 4 owns the tensor memory and issues
// the tcgen05.mma instructions in block order (four of K = 16 per stage), committing each stage
// back to its producer; at the end warps 0-3 read the accumulator with tcgen05.ld and store it.
// Every wait is bounded; a wait that runs out sets a status bit and the kernel carries on to its
// end (tensor memory is freed on every path).
#include "ans_decode_common.cuh"
#include "ans_walk_strips.cuh"

namespace ansb {

constexpr uint32_t kFgBlock = 64;                 // W is cut into kFgBlock x kFgBlock blocks
constexpr uint32_t kFgStages = 4;                 // = producer warps
constexpr uint32_t kFgATile = 128 * 128;          // bytes: 128 rows of X, 64 bf16 each
constexpr uint32_t kFgBTile = 64 * 128;           // bytes: 64 rows of W, 64 bf16 each
constexpr uint32_t kFgHeader = 64;                // bytes: 32 lanes x 16-bit length (strips container)
constexpr uint32_t kFgCols = 64;                  // tensor-memory columns: 64 fp32 accumulators per row

struct FgArgs {
  const uint8_t* blob;          // W's decode table
  const uint8_t* stream;
  const uint64_t* sub_offsets;
  uint64_t stream_bytes;
  const uint16_t* x;            // bf16 [M][K]
  float* y;                     // [M][N]
  uint32_t M, N, K;
  uint32_t R, zero_point, bitwidth;
  float scale;
  uint32_t* d_status;
};

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

// A wait on an mbarrier phase with a limit in clock cycles (about 0.1 s); once any wait of the
// thread has run out (a bit in `bad`), later ones only look once, so that a broken run ends fast.
// try_wait lets the hardware park the thread for a while instead of having it poll: a waiting
// warp then leaves the issue slots to the warps that decode.
__device__ __forceinline__ bool fg_wait(uint32_t bar, uint32_t parity, uint32_t bad) {
  const long long t0 = clock64();
  for (;;) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    if ((bad & kStatusTimeout) || clock64() - t0 > 200000000ll) return false;
  }
}

// where element (row, k) of a tile of 64 bf16 per row lies: rows of 128 bytes, eight rows to a
// 1 KB group, the 16-byte pieces of a row exchanged by the row's number in its group (the
// 128-byte swizzle of the tensor-core operand layouts, K-major)
__device__ __forceinline__ uint32_t tile_offset(uint32_t row, uint32_t k) {
  return (row >> 3) * 1024u + (row & 7u) * 128u + ((((k >> 3) ^ row) & 7u) << 4) + (k & 7u) * 2u;
}

// shared-memory operand descriptor: start address, 16-byte units; leading offset 1 (unused for a
// swizzled K-major tile); stride between 8-row groups 1024 bytes; descriptor version 1;
// 128-byte swizzle
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr) {
  return uint64_t((smem_addr & 0x3FFFFu) >> 4) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) |
         (uint64_t(1) << 46) | (uint64_t(2) << 61);
}

// instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, N = 64, M = 128
constexpr uint32_t kFgIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kFgBlock >> 3) << 17) | ((128u >> 4) << 24);

// Decode one 64 x 64 block (one sub-stream of the strips container, 128 symbols per lane, lanes in
// step) into the B tile at b_abs.  tab: one word per state (symbol, nb_bits, newX); vals: the
// dequantised bf16 of every symbol.  Returns status bits.
__device__ __noinline__ uint32_t decode_block(const FgArgs& a, uint64_t sub, uint32_t tab_abs, uint32_t vals_abs,
                                              uint32_t b_abs, uint32_t lane) {
  uint32_t bad = 0;
  uint64_t off0 = __ldg(a.sub_offsets + sub), off1 = __ldg(a.sub_offsets + sub + 1);
  if (off1 < off0 || off1 > a.stream_bytes || ((off0 | off1) & 15u) || off1 - off0 < kFgHeader || off1 - off0 > 0x3FFFFFFFull) {
    // unusable offsets: the block is left as zeros
    for (uint32_t i = lane * 16u; i < kFgBTile; i += 512u)
      asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" :: "r"(b_abs + i), "r"(0u) : "memory");
    return ANS_STATUS_BAD_LENGTH;
  }
  const uint32_t* words = reinterpret_cast<const uint32_t*>(a.stream + off0);
  const uint32_t ext_words = static_cast<uint32_t>((off1 - off0) >> 2);
  auto load_word = [&](uint32_t i) -> uint32_t { return i < ext_words ? __ldg(words + i) : 0u; };
  const uint32_t hw = load_word(lane >> 1);
  const uint32_t len = (lane & 1u) ? hw >> 16 : hw & 0xFFFFu;
  uint32_t incl = len;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t up = __shfl_up_sync(kFull, incl, d);
    if (lane >= static_cast<uint32_t>(d)) incl += up;
  }
  const uint32_t total_bits = __shfl_sync(kFull, incl, 31);
  if ((((kFgHeader / 4u + ((total_bits + 31u) >> 5)) + 3u) & ~3u) != ext_words) bad |= ANS_STATUS_BAD_LENGTH;
  const uint32_t bit0 = kFgHeader * 8u + (incl - len);
  uint32_t idx = bit0 >> 5, bitpos = bit0 & 31u;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1);
  idx += 2;
  auto take = [&](uint32_t nb) -> uint32_t {           // the next nb bits, most significant first
    const uint32_t x = __funnelshift_l(w1, w0, bitpos);
    const uint32_t v = nb ? x >> (32u - nb) : 0u;
    bitpos += nb;
    if (bitpos >= 32u) { w0 = w1; w1 = load_word(idx); ++idx; bitpos -= 32u; }
    return v;
  };
  uint32_t state = take(a.R);
  constexpr uint32_t kPerLane = kFgBlock * kFgBlock / 32u;
  for (uint32_t t = 0; t < kPerLane; ++t) {
    const uint32_t e = lds_u32(tab_abs + state * 4u);
    const uint32_t q = t * 32u + lane;                   // the symbol's place in the block = in the tile
    const uint32_t val = lds_u32(vals_abs + (e & 0xFFu) * 4u);
    sts_elem<2>(b_abs + q * 2u, val);
    state = (e >> 16) + take((e >> 8) & 15u);
  }
  if (state != 0) bad |= ANS_STATUS_BAD_FINAL_STATE;
  if ((idx - 2u) * 32u + bitpos - bit0 != len) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

__global__ void __launch_bounds__(160, 1) ans_decode_gemm_kernel(const FgArgs a) {
  extern __shared__ uint8_t sm_raw[];
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  // [A tiles][B tiles], 1 KB aligned; [table 4 << R][values 1 KB][barriers]
  const uint32_t base = (smem_u32(sm_raw) + 1023u) & ~1023u;
  const uint32_t a_abs = base, b_abs = base + kFgStages * kFgATile;
  const uint32_t tab_abs = b_abs + kFgStages * kFgBTile;
  const uint32_t vals_abs = tab_abs + (4u << a.R);
  const uint32_t bars_abs = vals_abs + 1024u;
  const uint32_t full_bar = bars_abs, empty_bar = bars_abs + 8u * kFgStages, done_bar = bars_abs + 16u * kFgStages;
  const uint32_t slot_abs = done_bar + 8u;
  uint32_t bad = 0;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < kFgStages; ++s) { mbar_init(full_bar + 8u * s, 1); mbar_init(empty_bar + 8u * s, 1); }
    mbar_init(done_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 4) {                                         // this warp owns the tensor memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(slot_abs), "r"(kFgCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // the table, one word per state, and the dequantised value of every symbol
  {
    const uint32_t* g_single = reinterpret_cast<const uint32_t*>(a.blob + single_offset());
    for (uint32_t i = threadIdx.x; i < (1u << a.R); i += blockDim.x)
      asm volatile("st.shared.u32 [%0], %1;" :: "r"(tab_abs + i * 4u), "r"(__ldg(g_single + i)) : "memory");
    for (uint32_t s = threadIdx.x; s < 256u; s += blockDim.x)
      asm volatile("st.shared.u32 [%0], %1;" :: "r"(vals_abs + s * 4u),
                   "r"(dequant_bits(static_cast<int>(s), static_cast<int>(a.zero_point), a.scale, ANS_BF16)) : "memory");
    const TableHeader* hdr = reinterpret_cast<const TableHeader*>(a.blob);
    if (threadIdx.x == 0 && (__ldg(&hdr->magic) != kTableMagic || __ldg(&hdr->table_log) != a.R ||
                             __ldg(&hdr->alphabet) > (1u << a.bitwidth)))
      bad |= ANS_STATUS_BAD_SYMBOL;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = lds_u32(slot_abs);

  const uint32_t nb_row = blockIdx.x;                      // block row of W: output features 64 nb_row ...
  const uint32_t KB = a.K / kFgBlock;
  if (warp < kFgStages) {
    // ---- producers --------------------------------------------------------------------------
    const uint32_t my_a = a_abs + warp * kFgATile, my_b = b_abs + warp * kFgBTile;
    for (uint32_t kb = warp, it = 0; kb < KB; kb += kFgStages, ++it) {
      if (it > 0 && !__all_sync(kFull, fg_wait(empty_bar + 8u * warp, (it - 1u) & 1u, bad))) bad |= kStatusTimeout;
      // the slice of X: rows beyond M are zeros
      for (uint32_t i = lane; i < 128u * 8u; i += 32u) {
        const uint32_t r = i >> 3, c = i & 7u;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (r < a.M) v = __ldg(reinterpret_cast<const uint4*>(a.x + size_t(r) * a.K + size_t(kb) * kFgBlock + c * 8u));
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                     :: "r"(my_a + tile_offset(r, c * 8u)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
      }
      bad |= decode_block(a, uint64_t(nb_row) * KB + kb, tab_abs, vals_abs, my_b, lane);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads shared memory through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8u * warp);
    }
  } else if (lane == 0) {
    // ---- the thread that issues the matrix instructions ----------------------------------------
    for (uint32_t kb = 0; kb < KB; ++kb) {
      const uint32_t s = kb & (kFgStages - 1u), it = kb / kFgStages;
      if (!fg_wait(full_bar + 8u * s, it & 1u, bad)) bad |= kStatusTimeout;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint64_t da = operand_desc(a_abs + s * kFgATile), db = operand_desc(b_abs + s * kFgBTile);
#pragma unroll
      for (uint32_t j = 0; j < kFgBlock / 16u; ++j) {      // K = 16 per instruction: 32 bytes further along the rows
        const uint32_t accumulate = (kb | j) ? 1u : 0u;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
            :: "r"(tmem), "l"(da + 2u * j), "l"(db + 2u * j), "r"(kFgIdesc), "r"(accumulate), "r"(0u) : "memory");
      }
      // the stage is free again once these have read it
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(empty_bar + 8u * s) : "memory");
    }
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(done_bar) : "memory");
  }

  // ---- the accumulator: row m of Y in lane m of the tensor memory, 64 columns -------------------
  if (warp < 4) {
    __syncwarp();
    if (!__all_sync(kFull, fg_wait(done_bar, 0, bad))) bad |= kStatusTimeout;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t row = warp * 32u + lane;
    float* yrow = a.y + size_t(row) * a.N + size_t(nb_row) * kFgBlock;
#pragma unroll
    for (uint32_t c0 = 0; c0 < kFgCols; c0 += 8u) {
      uint32_t r0, r1, r2, r3, r4, r5, r6, r7;
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                   : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5), "=r"(r6), "=r"(r7)
                   : "r"(tmem + ((warp * 32u) << 16) + c0) : "memory");
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (row < a.M) {
        *reinterpret_cast<uint4*>(yrow + c0) = make_uint4(r0, r1, r2, r3);
        *reinterpret_cast<uint4*>(yrow + c0 + 4) = make_uint4(r4, r5, r6, r7);
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 4) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kFgCols) : "memory");
  }
  bad = __reduce_or_sync(kFull, bad);
  if (lane == 0 && bad && a.d_status) atomicOr(a.d_status, bad);
}

// ---------------------------------------------------------------------------------------------
// The wide form, for tables of up to 256 states (the paper's sizes) and N a multiple of 256.
//
// The work is cut into units: 256 output features (four block rows of W) by one step of 64 along
// K; the units, ordered by features and then by K, are dealt to the CTAs (one per SM) in equal
// contiguous ranges.  A range is a sequence of segments, each a run of K steps under the same 256
// features: a segment is accumulated in tensor memory and then leaves for Y, by plain stores if
// it covers all of K and by fp32 atomic adds (into a Y zeroed beforehand) if not.  Two
// accumulators take turns, so that a segment is stored while the next is being multiplied.
// A stage holds a 128 x 64 slice of X and the four 64 x 64 blocks of W under it.  Sixteen producer
// warps take the blocks of the range in turn (row i = warp mod 4 of unit warp / 4, + 4, ...) and
// decode them with the strips kernel's walk (pre-walked table: a look-up stands for a run of the
// dominant symbol plus one symbol, Section II-A) into the tile, pre-filled with the dominant
// value.  The sub-stream's bytes come into shared memory by asynchronous copies issued one block
// ahead.  Warp 16 issues one tcgen05.mma of N = 256 per 16 columns of K; warps 17-20 read the
// finished accumulators with tcgen05.ld.
// ---------------------------------------------------------------------------------------------
// The kernel has two forms.  NM = 0: X is the 128-row operand (any M up to 128) and the 256 rows of W
// are the N = 256 operand, as described above.  NM = 16 or 32, for M up to NM: the operands are
// exchanged, Y^T = W X^T: the 256 rows of W are two 128-row operands and the NM rows of X (a tile
// of NM * 128 bytes instead of 16 KB) the N = NM operand of both; the shared memory that X no
// longer takes holds a fifth stage, so twenty producers decode instead of sixteen, and a row of
// the accumulator is a feature, so that a warp stores 32 consecutive floats of a row of Y.
constexpr uint32_t kF2Rows = 4;                   // block rows of W per CTA
constexpr uint32_t kF2BTile = kF2Rows * kFgBTile; // bytes: 256 rows of W, 64 bf16 each
constexpr uint32_t kF2Cols = kF2Rows * kFgBlock;  // features per unit
template <uint32_t NM>
struct F2Shape {
  // (NM = 0: three stages would leave room for 32 copies of the table, but twelve tiles in flight
  // instead of sixteen: measured slower)
  static constexpr uint32_t kStages = NM ? 5 : 4;
  static constexpr uint32_t kProducers = kStages * kF2Rows;
  static constexpr uint32_t kThreads = (kProducers + 1 + 4) * 32;   // producers, the issuing warp, four warps that store
  static constexpr uint32_t kXRows = NM ? NM : 128;                 // rows of X in a stage
  static constexpr uint32_t kXTile = kXRows * 128;                  // bytes
  static constexpr uint32_t kAccCols = NM ? 2 * NM : kF2Cols;       // tensor-memory columns of one accumulator (there are two)
  // instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, M = 128, N = NM or 256
  static constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (((NM ? NM : kF2Cols) >> 3) << 17) | ((128u >> 4) << 24);
};
constexpr uint32_t kF2Pad = 256;                  // zero bytes after a staged sub-stream: more than a lane can
                                                  // advance in the 128 look-ups of a block (8 bits each at most)

struct F2Args {
  FgArgs g;
  uint32_t units;               // work units in all: (N / 256) * (K / 64), one per 256 x 64 piece of W
  uint32_t stage_bytes;         // per producer: room for a sub-stream's bytes and the padding
  uint32_t rep_log;             // copies of the table, log2
  uint32_t unit;                // the value 1
};

// Decode one block (one sub-stream: 128 symbols per lane) into the tile at tile_abs, which holds
// the dominant value everywhere.  The sub-stream's words are in shared memory at
// stage_abs (staged, zero words after them) or in global memory.  Returns status bits.
__device__ __noinline__ uint32_t decode_block_wide(uint32_t tab_lane, uint32_t stride_log, uint32_t succ_abs,
                                                   uint32_t tile_abs, uint32_t stage_abs,
                                                   const uint32_t* __restrict__ words, uint32_t ext_words, bool staged,
                                                   uint32_t R, uint32_t unit, uint32_t lane) {
  constexpr uint32_t count = kFgBlock * kFgBlock / 32u;
  const uint32_t word_limit = staged ? ext_words + 4u : ext_words;
  auto load_word = [&](uint32_t i) -> uint32_t {
    if (staged) return lds_u32(stage_abs + min(i, word_limit + 8u) * 4u);
    return i < word_limit ? __ldg(words + i) : 0u;
  };
  uint32_t bad = 0;
  const uint32_t hw = load_word(lane >> 1);
  const uint32_t len = (lane & 1u) ? hw >> 16 : hw & 0xFFFFu;
  uint32_t incl = len;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t up = __shfl_up_sync(kFull, incl, d);
    if (lane >= static_cast<uint32_t>(d)) incl += up;
  }
  const uint32_t total_bits = __shfl_sync(kFull, incl, 31);
  if (ext_words < kFgHeader / 4u || (((kFgHeader / 4u + ((total_bits + 31u) >> 5)) + 3u) & ~3u) != ext_words)
    bad |= ANS_STATUS_BAD_LENGTH;
  const uint32_t bit0 = kFgHeader * 8u + (incl - len);
  uint32_t idx = bit0 >> 5, bitpos = bit0 & 31u;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1), w2 = load_word(idx + 2);
  idx += 3;
  uint32_t state = __funnelshift_l(w1, w0, bitpos) >> (32u - R);   // the string begins with the state, R bits
  bitpos += R;
  if (bitpos >= 32u) { w0 = w1; w1 = w2; w2 = load_word(idx); ++idx; bitpos -= 32u; }
  const uint32_t stride = 1u << stride_log;
  uint32_t st = tab_lane + (state << stride_log);
  uint32_t z = 0;
  const uint32_t abase = tile_abs + lane * 2u;             // position z of this lane: symbol 32 z + lane of the block
  if (staged) {
    const uint32_t sp_limit = stage_abs + word_limit * 4u;
    uint32_t sp = min(stage_abs + min(idx, word_limit) * 4u, sp_limit);
    strip_window_walk<2, 4, true, false>(st, bitpos, w0, w1, w2, sp, z, tab_lane, stride, abase, count, unit, sp_limit, 0u, 0u);
    if (sp >= sp_limit) bad |= ANS_STATUS_BAD_LENGTH;
    idx = (sp - stage_abs) >> 2;
  } else {
    bool any = true;
    while (any) {
      const uint32_t ea = lds_u32(st);
      const uint32_t nb = (ea >> 16) & 15u, zn = z + ((ea >> 20) & 15u);
      const bool act = zn < count;
      if (act) {
        sts_elem<2>(abase + zn * 64u, ea);
        const uint32_t x = __funnelshift_l(w1, w0, bitpos);
        st = tab_lane + (__funnelshift_l(x, ea >> 24, nb) << stride_log);
        z = zn + 1u;
        bitpos += nb;
        if (bitpos >= 32u) { w0 = w1; w1 = w2; w2 = load_word(idx); ++idx; bitpos -= 32u; }
      }
      any = __any_sync(kFull, act);
    }
  }
  // what is left of the lane lies inside the run of the entry it stopped at
  uint32_t s = (st - tab_lane) >> stride_log;
  for (uint32_t left = count - z; left != 0 && left <= uint32_t(kMaxRun); --left) s = lds_u16(succ_abs + s * 2u);
  if (count - z > uint32_t(kMaxRun) || s != 0) bad |= ANS_STATUS_BAD_FINAL_STATE;
  if ((idx - 3u) * 32u + bitpos - bit0 != len) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

template <uint32_t NM>
__global__ void __launch_bounds__(F2Shape<NM>::kThreads, 1) ans_decode_gemm_wide_kernel(const F2Args args) {
  using Shape = F2Shape<NM>;
  constexpr uint32_t kF2Stages = Shape::kStages, kF2Producers = Shape::kProducers;
  extern __shared__ uint8_t sm_raw[];
  const FgArgs& a = args.g;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  // [A tiles][B tiles], 1 KB aligned; [table copies][successors][byte stages][barriers]
  const uint32_t base = (smem_u32(sm_raw) + 1023u) & ~1023u;
  const uint32_t a_abs = base, b_abs = base + kF2Stages * Shape::kXTile;   // (a: the slices of X; b: the tiles of W)
  const uint32_t tab_abs = b_abs + kF2Stages * kF2BTile;
  const uint32_t stride_log = 2u + args.rep_log;
  const uint32_t succ_abs = tab_abs + (1u << (a.R + stride_log));
  const uint32_t succ_bytes = max(2u << a.R, 16u);
  const uint32_t stages_abs = succ_abs + succ_bytes;
  const uint32_t bars_abs = stages_abs + kF2Producers * args.stage_bytes;
  // A wait on an mbarrier tells the current phase from the one before it and no more.  The thread
  // that issues the products takes the steps in order, but a producer may be several steps ahead
  // of the others; so a stage has two "empty" barriers used in turn (fill u of stage s frees
  // barrier 2 s + u mod 2): the phase before the one a producer waits for then lies nine steps
  // back, and the producer has seen step j - 7 consumed when it took its last block.
  const uint32_t full_bar = bars_abs, empty_bar = bars_abs + 8u * kF2Stages;
  const uint32_t acc_full = bars_abs + 24u * kF2Stages, acc_empty = acc_full + 16u;   // two accumulators
  const uint32_t slot_abs = acc_empty + 16u;
  uint32_t bad = 0;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < kF2Stages; ++s) {
      mbar_init(full_bar + 8u * s, kF2Rows);
      mbar_init(empty_bar + 16u * s, 1);
      mbar_init(empty_bar + 16u * s + 8u, 1);
    }
    for (uint32_t b = 0; b < 2u; ++b) { mbar_init(acc_full + 8u * b, 1); mbar_init(acc_empty + 8u * b, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kF2Producers) {                              // this warp owns the tensor memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(slot_abs), "r"(2u * Shape::kAccCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // the pre-walked table in one-word entries, the bf16 value folded in, copies side by side
  const TableHeader* hdr = reinterpret_cast<const TableHeader*>(a.blob);
  const uint32_t h_dominant = __ldg(&hdr->dominant);
  {
    const uint32_t* g_single = reinterpret_cast<const uint32_t*>(a.blob + single_offset());
    const uint32_t* g_multi = reinterpret_cast<const uint32_t*>(a.blob + multi_offset(static_cast<int>(a.R)));
    for (uint32_t i = threadIdx.x; i < (1u << a.R); i += blockDim.x) {
      const uint32_t gm = __ldg(g_multi + i), gs = __ldg(g_single + i);
      const uint32_t val = dequant_bits(static_cast<int>(entry_sym(gm)), static_cast<int>(a.zero_point), a.scale, ANS_BF16);
      const uint32_t e = to_strip_entry_short(gm, val);
      if (stride_log >= 4u) {                              // 16 bytes at a time, every lane starting at another piece
        const uint32_t pieces = 1u << (stride_log - 4u), turn = lane & (pieces - 1u);
#pragma unroll
        for (uint32_t q = 0; q < 8u; ++q)
          if (q < pieces) sts_v4(tab_abs + (i << stride_log) + ((q ^ turn) << 4), make_uint4(e, e, e, e));
      } else {
        for (uint32_t c = 0; c < (1u << args.rep_log); ++c)
          asm volatile("st.shared.u32 [%0], %1;" :: "r"(tab_abs + (i << stride_log) + c * 4u), "r"(e) : "memory");
      }
      asm volatile("st.shared.u16 [%0], %1;" :: "r"(succ_abs + i * 2u), "r"(entry_newx(gs)) : "memory");
    }
    if (threadIdx.x == 0 && (__ldg(&hdr->magic) != kTableMagic || __ldg(&hdr->table_log) != a.R ||
                             __ldg(&hdr->alphabet) > (1u << a.bitwidth)))
      bad |= ANS_STATUS_BAD_SYMBOL;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = lds_u32(slot_abs);

  const uint32_t KB = a.K / kFgBlock;
  // this CTA's units [u0, u0 + nu)
  const uint32_t u0 = static_cast<uint32_t>(uint64_t(args.units) * blockIdx.x / gridDim.x);
  const uint32_t nu = static_cast<uint32_t>(uint64_t(args.units) * (blockIdx.x + 1u) / gridDim.x) - u0;
  if (warp < kF2Producers) {
    // ---- producers --------------------------------------------------------------------------
    const uint32_t i = warp % kF2Rows, j0 = warp / kF2Rows;
    constexpr uint32_t kStep = kF2Producers / kF2Rows;     // units between two blocks of a warp
    static_assert(kStep <= 2 * kF2Stages, "a producer must have seen the phase before the one it waits for");
    static_assert(kStep == kF2Stages, "a producer keeps to one stage");
    const uint32_t my_stage = stages_abs + warp * args.stage_bytes;
    const uint32_t tab_lane = tab_abs + ((lane & ((1u << args.rep_log) - 1u)) << 2);
    const uint32_t dom = dequant_bits(static_cast<int>(h_dominant < 256u ? h_dominant : 0u), static_cast<int>(a.zero_point),
                                      a.scale, ANS_BF16);
    const uint32_t fill = (dom & 0xFFFFu) * 0x10001u;
    const uint4 fill4 = make_uint4(fill, fill, fill, fill);
    // the sub-stream of this warp's row of unit u: block (4 tile + i, step) of W
    auto sub_of = [&](uint32_t u) -> uint64_t {
      const uint32_t tile = u / KB;
      return uint64_t(tile * kF2Rows + i) * KB + (u - tile * KB);
    };

    // the extent of a sub-stream, checked; its bytes requested into the warp's stage when they fit
    uint64_t off0 = 0;
    uint32_t extent = 0;
    bool staged = false;
    auto locate = [&](uint64_t o0, uint64_t o1) {
      off0 = o0;
      extent = static_cast<uint32_t>(o1 - o0);
      if (o1 < o0 || o1 > a.stream_bytes || ((o0 | o1) & 15u) || o1 - o0 < kFgHeader || o1 - o0 > 0x3FFFFFFFull) {
        extent = 0;
        off0 = 0;
        bad |= ANS_STATUS_BAD_LENGTH;
      }
      staged = extent > 0 && extent + kF2Pad <= args.stage_bytes;
      if (staged) {
        const uint8_t* src = a.stream + off0;
        for (uint32_t o = lane * 16u; o < extent; o += 512u)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(my_stage + o), "l"(src + o) : "memory");
        for (uint32_t q = lane; q < kF2Pad / 4u; q += 32u)
          asm volatile("st.shared.u32 [%0], %1;" :: "r"(my_stage + extent + q * 4u), "r"(0u) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint64_t n0 = 0, n1 = 0;                               // offsets of the block after this one
    if (j0 < nu) {
      const uint64_t sub = sub_of(u0 + j0);
      locate(__ldg(a.sub_offsets + sub), __ldg(a.sub_offsets + sub + 1));
    }
    for (uint32_t j = j0; j < nu; j += kStep) {
      const bool more = j + kStep < nu;
      if (more) {
        const uint64_t sub = sub_of(u0 + j + kStep);
        n0 = __ldg(a.sub_offsets + sub);
        n1 = __ldg(a.sub_offsets + sub + 1);
      }
      const uint32_t s = j % kF2Stages, use = j / kF2Stages;   // the stage and how often it has been filled before
      const uint32_t my_a = a_abs + s * Shape::kXTile, my_b = b_abs + s * kF2BTile + i * kFgBTile;
      const uint32_t kb = (u0 + j) % KB;
      if (use > 0 && !__all_sync(kFull, fg_wait(empty_bar + 16u * s + 8u * ((use - 1u) & 1u), ((use - 1u) >> 1) & 1u, bad)))
        bad |= kStatusTimeout;
      // this warp's quarter of the slice of X: rows beyond M are zeros
      constexpr uint32_t kQuarter = Shape::kXRows / kF2Rows;   // rows
#pragma unroll
      for (uint32_t q = 0; q < (kQuarter * 8u + 31u) / 32u; ++q) {
        const uint32_t idx = q * 32u + lane, c = idx & 7u, r = i * kQuarter + (idx >> 3);
        if (idx < kQuarter * 8u) {
          const uint32_t bytes = r < a.M ? 16u : 0u;
          const uint16_t* src = a.x + size_t(r < a.M ? r : 0u) * a.K + size_t(kb) * kFgBlock + c * 8u;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(my_a + tile_offset(r, c * 8u)), "l"(src), "r"(bytes) : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      for (uint32_t o = lane * 16u; o < kFgBTile; o += 512u) sts_v4(my_b + o, fill4);
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncwarp();
      if (extent)
        bad |= decode_block_wide(tab_lane, stride_log, succ_abs, my_b, my_stage,
                                 reinterpret_cast<const uint32_t*>(a.stream + off0), extent >> 2, staged, a.R, args.unit, lane);
      __syncwarp();
      // the warp's bytes are used up: the next block's may come
      if (more) locate(n0, n1);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads shared memory through the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar + 8u * s);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else if (warp == kF2Producers) {
    // ---- the thread that issues the matrix instructions ----------------------------------------
    if (lane == 0) {
      uint32_t seg = 0;
      for (uint32_t j = 0; j < nu; ++j) {
        const uint32_t s = j % kF2Stages, use = j / kF2Stages;
        const uint32_t kb = (u0 + j) % KB;
        const bool first = j == 0 || kb == 0, last = j + 1u == nu || kb + 1u == KB;
        const uint32_t buf = seg & 1u;
        if (first && seg >= 2u) {                          // the accumulator must have been read out
          if (!fg_wait(acc_empty + 8u * buf, ((seg >> 1) - 1u) & 1u, bad)) bad |= kStatusTimeout;
        }
        if (!fg_wait(full_bar + 8u * s, use & 1u, bad)) bad |= kStatusTimeout;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t dx = operand_desc(a_abs + s * Shape::kXTile), dw = operand_desc(b_abs + s * kF2BTile);
#pragma unroll
        for (uint32_t k = 0; k < kFgBlock / 16u; ++k) {    // K = 16 per instruction: 32 bytes further along the rows
          const uint32_t accumulate = (!first || k) ? 1u : 0u;
#pragma unroll
          for (uint32_t h = 0; h < (NM ? 2u : 1u); ++h) {
            // NM = 0: D[m][n] = X (128 rows) times the 256 rows of W.  Else D[n][m], one product for
            // each half of the rows of W (128 rows = 16 KB further on), side by side in the accumulator
            const uint64_t da = NM ? dw + uint64_t(h * (128u * 128u >> 4)) : dx, db = NM ? dx : dw;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                :: "r"(tmem + buf * Shape::kAccCols + h * NM), "l"(da + 2u * k), "l"(db + 2u * k), "r"(Shape::kIdesc),
                   "r"(accumulate), "r"(0u) : "memory");
          }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                     :: "r"(empty_bar + 16u * s + 8u * (use & 1u)) : "memory");
        if (last) {
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(acc_full + 8u * buf) : "memory");
          ++seg;
        }
      }
    }
  } else {
    // ---- the accumulators: row m of Y in lane m of the tensor memory, 256 columns ------------------
    const uint32_t quarter = warp & 3u;                    // the lanes of tensor memory this warp may read
    const uint32_t row = quarter * 32u + lane;
    uint32_t seg = 0;
    for (uint32_t j = 0; j < nu; ++seg) {
      const uint32_t tile = (u0 + j) / KB, kb = (u0 + j) - tile * KB;
      const uint32_t len = min(KB - kb, nu - j);
      const bool add = len != KB;                          // part of K only: the parts meet in Y
      const uint32_t buf = seg & 1u;
      if (!__all_sync(kFull, fg_wait(acc_full + 8u * buf, (seg >> 1) & 1u, bad))) bad |= kStatusTimeout;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if constexpr (NM == 0) {
        float* yrow = a.y + size_t(row) * a.N + size_t(tile) * kF2Cols;
#pragma unroll 4
        for (uint32_t c0 = 0; c0 < (quarter * 32u < a.M ? kF2Cols : 0u); c0 += 8u) {   // (a warp whose rows are all beyond M has nothing to store)
          uint32_t r0, r1, r2, r3, r4, r5, r6, r7;
          asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                       : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5), "=r"(r6), "=r"(r7)
                       : "r"(tmem + ((quarter * 32u) << 16) + buf * kF2Cols + c0) : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (row < a.M) {
            if (add) {
              atomicAdd(reinterpret_cast<float4*>(yrow + c0),
                        make_float4(__uint_as_float(r0), __uint_as_float(r1), __uint_as_float(r2), __uint_as_float(r3)));
              atomicAdd(reinterpret_cast<float4*>(yrow + c0 + 4),
                        make_float4(__uint_as_float(r4), __uint_as_float(r5), __uint_as_float(r6), __uint_as_float(r7)));
            } else {
              *reinterpret_cast<uint4*>(yrow + c0) = make_uint4(r0, r1, r2, r3);
              *reinterpret_cast<uint4*>(yrow + c0 + 4) = make_uint4(r4, r5, r6, r7);
            }
          }
        }
      } else {
        // lane n of the tensor memory holds feature n of a half, its columns the rows of X: the
        // warp's 32 lanes store 32 consecutive floats of one row of Y at a time
#pragma unroll
        for (uint32_t h = 0; h < 2u; ++h) {
          float* ycol = a.y + size_t(tile) * kF2Cols + h * 128u + row;
#pragma unroll
          for (uint32_t c0 = 0; c0 < NM; c0 += 16u) {
            uint32_t r[16];
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                           "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                         : "r"(tmem + ((quarter * 32u) << 16) + buf * Shape::kAccCols + h * NM + c0) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (uint32_t m = 0; m < 16u; ++m) {
              if (c0 + m < a.M) {
                if (add) atomicAdd(ycol + size_t(c0 + m) * a.N, __uint_as_float(r[m]));
                else ycol[size_t(c0 + m) * a.N] = __uint_as_float(r[m]);
              }
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + 8u * buf);
      j += len;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kF2Producers) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(2u * Shape::kAccCols) : "memory");
  }
  bad = __reduce_or_sync(kFull, bad);
  if (lane == 0 && bad && a.d_status) atomicOr(a.d_status, bad);
}

}  // namespace ansb

namespace ansb {

// Launch the wide form NM (see F2Shape).  Returns ANS_OK, an error, or 1 if the form does not
// fit this device's shared memory.
template <uint32_t NM>
static int launch_wide(const FgArgs& a, const ans_layer_desc& d, int sms, int smem_max, cudaStream_t st) {
  using Shape = F2Shape<NM>;
  const uint32_t M = a.M, N = a.N, K = a.K;
  // room for a sub-stream of up to 1.25 times the average plus the padding per producer, less if
  // shared memory is short (a sub-stream that does not fit is read from global memory); what
  // shared memory is left goes to copies of the table
  const uint64_t n_sub = uint64_t(N / 64) * uint64_t(K / 64);
  size_t stage = static_cast<size_t>(d.stream_bytes / n_sub);
  stage = (stage + stage / 4 + 128 + kF2Pad + 127) & ~size_t(127);
  const size_t succ = (size_t(2) << d.table_log) < 16 ? 16 : (size_t(2) << d.table_log);
  const size_t one_table = size_t(4) << d.table_log;
  const size_t rest = 1024 + Shape::kStages * (Shape::kXTile + kF2BTile) + succ + 256;
  const size_t room = static_cast<size_t>(smem_max) > rest + one_table ? static_cast<size_t>(smem_max) - rest - one_table : 0;
  if (Shape::kProducers * stage > room) stage = (room / Shape::kProducers) & ~size_t(127);
  const size_t fixed = rest + Shape::kProducers * stage;
  if (stage < 512) return 1;
  uint32_t rep_log = 0;
  while (rep_log < 5 && fixed + (one_table << (rep_log + 1)) <= static_cast<size_t>(smem_max)) ++rep_log;
  const uint32_t KB = K / 64, tiles = N / kF2Cols;
  const uint64_t units = uint64_t(tiles) * KB;
  if (units > 0x7FFFFFFFull) return ANS_ERR_UNSUPPORTED;
  // CTAs: one per SM with the units dealt evenly, or, if that saves no round of the producers
  // (a stage's worth of units is decoded at a time), a whole number of CTAs per 256 features, so
  // that no range crosses from one accumulator's features to the next
  uint32_t ctas = units < static_cast<uint64_t>(sms) ? static_cast<uint32_t>(units) : static_cast<uint32_t>(sms);
  {
    uint32_t per_tile = static_cast<uint32_t>(sms) / tiles;
    if (per_tile > KB) per_tile = KB;
    const uint32_t aligned = tiles * per_tile;
    constexpr uint32_t kAtATime = Shape::kStages;
    auto rounds = [&](uint32_t n) { return ((units + n - 1) / n + kAtATime - 1) / kAtATime; };
    if (aligned >= 1 && rounds(aligned) <= rounds(ctas)) {
      // and no more CTAs than that number of rounds needs: fewer partial sums to add
      while (per_tile > 1 && rounds(tiles * (per_tile - 1)) == rounds(aligned)) --per_tile;
      ctas = tiles * per_tile;
    }
  }
  // Y is zeroed first if any range ends inside the K steps of its 256 features (those parts are added)
  bool whole = true;
  for (uint32_t c = 1; c < ctas && whole; ++c) whole = (units * c / ctas) % KB == 0;
  F2Args w{};
  w.g = a;
  w.units = static_cast<uint32_t>(units);
  w.stage_bytes = static_cast<uint32_t>(stage);
  w.rep_log = rep_log;
  w.unit = 1u;
  const size_t smem = fixed + (one_table << rep_log);
  if (!whole) ANSB_CUDA(cudaMemsetAsync(a.y, 0, size_t(M) * size_t(N) * sizeof(float), st));
  ANSB_CUDA(cudaFuncSetAttribute(ans_decode_gemm_wide_kernel<NM>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  ans_decode_gemm_wide_kernel<NM><<<ctas, Shape::kThreads, smem, st>>>(w);
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}

}  // namespace ansb

using namespace ansb;

ANS_EXPORT int ans_decode_gemm_bf16(const ans_layer_desc* h_desc, const void* d_x, int M, int N, int K, float* d_y,
                                    uint32_t* d_status, void* stream) {
  ApiRange range("ans_decode_gemm_bf16");
  if (!h_desc || !d_x || !d_y || !d_status) return ANS_ERR_INVALID_ARG;
  const ans_layer_desc& d = *h_desc;
  int rc = validate_desc(d, false);
  if (rc != ANS_OK) return rc;
  if (d.layout != ANS_LAYOUT_STRIPS || d.chunk_symbols != kFgBlock * kFgBlock || d.lanes != 32 || d.table_log > 12)
    return ANS_ERR_UNSUPPORTED;
  if (M < 1 || M > 128 || N < 64 || K < 64 || N % 64 || K % 64 || N > (1 << 20) || K > (1 << 20)) return ANS_ERR_UNSUPPORTED;
  if (d.n_symbols != uint64_t(N) * uint64_t(K)) return ANS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 15) || (reinterpret_cast<uintptr_t>(d_y) & 15)) return ANS_ERR_INVALID_ARG;
  FgArgs a{};
  a.blob = static_cast<const uint8_t*>(d.d_table);
  a.stream = d.d_stream;
  a.sub_offsets = d.d_sub_offsets;
  a.stream_bytes = d.stream_bytes;
  a.x = static_cast<const uint16_t*>(d_x);
  a.y = d_y;
  a.M = static_cast<uint32_t>(M);
  a.N = static_cast<uint32_t>(N);
  a.K = static_cast<uint32_t>(K);
  a.R = static_cast<uint32_t>(d.table_log);
  a.zero_point = static_cast<uint32_t>(d.zero_point);
  a.bitwidth = static_cast<uint32_t>(d.bitwidth);
  a.scale = d.scale;
  a.d_status = d_status;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int dev = 0, sms = 0, smem_max = 0;
  ANSB_CUDA(cudaGetDevice(&dev));
  ANSB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ANSB_CUDA(cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
  if (d.table_log <= 8 && N % static_cast<int>(kF2Cols) == 0) {
    // the wide forms: the one with the operands exchanged when X has few rows
    const int rc2 = M <= 16 ? launch_wide<16>(a, d, sms, smem_max, st)
                  : M <= 32 ? launch_wide<32>(a, d, sms, smem_max, st) : launch_wide<0>(a, d, sms, smem_max, st);
    if (rc2 != 1) return rc2;                              // (1: shared memory too short for it)
  }
  const size_t smem = 1024 + kFgStages * (kFgATile + kFgBTile) + (size_t(4) << d.table_log) + 1024 + 128;
  ANSB_CUDA(cudaFuncSetAttribute(ans_decode_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  ans_decode_gemm_kernel<<<static_cast<unsigned>(N / 64), 160, smem, st>>>(a);
  ANSB_CUDA(cudaGetLastError());
  return ANS_OK;
}
