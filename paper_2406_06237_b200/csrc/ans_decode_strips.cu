// Decode (+ dequantise) kernel of the strips container, for sm_100a.
//
// Paper Section II-A: some transitions of the automaton take no bits; they belong to the one
// symbol that owns more than half of the states and are what carries the rate under one bit per
// weight.  The pre-walked table folds such chains into the entry that starts them: one look-up
// stands for `run` copies of the dominant symbol followed by one more symbol (state -> symbol,
// nb_bits, newX as in Fig. 2, after `run` unlabeled transitions).  Section III-B: one table per
// layer, a vector of states; here a warp holds the 32 states of a sub-stream.
//
// The container keeps a sub-stream's symbols in one contiguous strip of the layer, dealt to the
// 32 lanes round-robin, so a look-up that emits several symbols only moves a lane's own
// position: nothing has to be kept in step.  A warp collects a window of its strip in shared
// memory, pre-filled with the dominant symbol's value; a lane only writes the symbol that ends a
// run; a full window is contiguous in the output and leaves in 16-byte stores.
//
// The channels container (Section III-B: one stream per input channel of a tensor stored
// O x I x H x W) is walked by the same kernel: a row of the window is then one piece (H * W
// symbols) of every lane, rows lie a whole tensor row apart in the output, and a window leaves in
// one bulk store per row.
//
// One CTA = one work item of the batch plan (up to four consecutive sub-streams of ONE layer,
// a warp each).  Up to kStripParamLayers layer records travel in the kernel parameters, so a
// CTA reaches its layer without a trip to memory; the trips that remain are the sub-stream's
// offsets (then its bytes, one bulk copy) and, beside them, the layer's table.
#include "ans_decode_common.cuh"
#include "ans_walk_strips.cuh"

namespace ansb {

constexpr int kStripWarps = static_cast<int>(kGranule);   // sub-streams (warps) per CTA
constexpr int kStripParamLayers = 64;                     // layers of one launch
constexpr uint32_t kStripHeader = 64;                     // bytes: 32 lanes x 16-bit length
constexpr uint32_t kStripWindow = 4096;                   // bytes of output a warp collects before writing them out
constexpr uint32_t kStripBatch = 8;                       // table entries a thread requests at a time
constexpr uint32_t kStripCtaTable = 2048;                 // launches of up to this many CTAs carry a CTA -> layer table
constexpr uint32_t kStripPad = 256;                       // readable bytes after a staged sub-stream: more than a lane
                                                          // can advance while it walks one window (128 symbols of 14 bits)
static_assert(kStripWindow / 32 * 14 / 8 + 32 <= kStripPad, "a window's walk must stay inside the padding");

struct StripLayer {                // what the kernel needs of one layer, 64 bytes
  const uint8_t* blob;             // table blob
  const uint8_t* stream;
  const uint64_t* sub_offsets;
  uint8_t* out;
  uint64_t stream_bytes;
  uint64_t n_symbols;
  uint32_t chunk_symbols;
  uint32_t n_sub;
  float scale;
  uint32_t packed;                 // zero_point [7:0] | table_log [11:8] | bitwidth [15:12] | dtype [17:16] | lanes / 32 [24:18]
                                   // | piece_symbols [31:25] (channels container; 0: strips)
};

struct StripArgs {
  StripLayer layer[kStripParamLayers];
  uint32_t cta_begin[kStripParamLayers + 1];   // first CTA of each layer
  int n_layers;
  uint32_t* d_status;
  uint32_t table_bytes;            // shared-memory bytes reserved for the table copies
  uint32_t max_log;
  uint32_t succ_bytes;             // shared-memory bytes of the successor table (2 << max_log, at least 16)
  uint32_t stage_bytes;            // per-warp staging buffer for the sub-stream's bytes
  uint32_t unit;                   // the value 1 (keeps a multiply-add a multiply-add)
  uint32_t ctas;                   // CTAs of the launch
  uint32_t early;                  // 1: every layer's inputs were settled before the preceding work began;
                                   // 2: and the preceding work does not touch the outputs
  uint8_t cta_layer[kStripCtaTable];   // layer of every CTA when ctas <= kStripCtaTable: one look-up instead of a search
};

struct StripGeom {                 // one sub-stream's place in the output
  uint32_t count;                  // symbols of this lane
  uint32_t rows;                   // rows of the sub-stream (a row: E symbols of every lane, contiguous in the output)
  uint32_t E;                      // symbols of a lane per row: 1 for strips, the piece for channels
  uint32_t last_row_bytes;         // bytes of the last row (strips: it may be short)
  uint32_t row_stride;             // bytes from one row to the next in the output
};

// Decode one sub-stream.  win_abs: the warp's window (kStripWindow bytes, holding `fill`);
// words: the sub-stream in shared memory (STAGED, at stage_abs) or in global memory.
template <int ES, bool STAGED, bool SHORT, bool PIECES>
__device__ __noinline__ uint32_t decode_strip(
    uint32_t tab_lane, uint32_t stride_log, uint32_t succ_abs, uint32_t win_abs, uint32_t stage_abs,
    const uint32_t* __restrict__ words, uint32_t ext_words, uint32_t R, uint32_t count, uint32_t rows, uint32_t piece,
    uint32_t last_row_bytes, uint32_t row_stride, uint8_t* __restrict__ out_strip,
    uint32_t fill, bool wide_steps, uint32_t unit, uint32_t lane_early) {
  // lane_early: the lane, and in bit 8 whether the wait for the preceding work on the stream is
  // still to come (it then comes before the first byte is written; bit 9: no wait is needed)
  const uint32_t lane = lane_early & 31u;
  const uint32_t E = PIECES ? piece : 1u;
  const uint32_t magic = PIECES ? 0xFFFFFFFFu / piece + 1u : 0u;   // 2^32 / E rounded up (E >= 2)
  const uint32_t RB = 32u * ES * E;                        // bytes of a row
  const uint32_t P = kStripWindow / RB;                    // rows of a window
  const uint32_t word_limit = STAGED ? ext_words + 4u : ext_words;
  auto load_word = [&](uint32_t i) -> uint32_t {     // (staged: the words after the sub-stream are zero, up to kStripPad)
    if (STAGED) return lds_u32(stage_abs + min(i, word_limit + 8u) * 4u);
    return i < word_limit ? __ldg(words + i) : 0u;
  };
  uint32_t bad = 0;


  // the lanes' bit lengths head the sub-stream; their running sum places every lane's string
  const uint32_t hw = load_word(lane >> 1);
  const uint32_t len = (lane & 1u) ? hw >> 16 : hw & 0xFFFFu;
  uint32_t incl = len;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t up = __shfl_up_sync(kFull, incl, d);
    if (lane >= static_cast<uint32_t>(d)) incl += up;
  }
  const uint32_t total_bits = __shfl_sync(kFull, incl, 31);
  // the sub-stream must be exactly its header, the words its bits need, and the padding
  if (ext_words < kStripHeader / 4u || (((kStripHeader / 4u + ((total_bits + 31u) >> 5)) + 3u) & ~3u) != ext_words)
    bad |= ANS_STATUS_BAD_LENGTH;
  const uint32_t bit0 = kStripHeader * 8u + (incl - len);
  uint32_t idx = bit0 >> 5, bitpos = bit0 & 31u;
  uint32_t w0 = load_word(idx), w1 = load_word(idx + 1), w2 = load_word(idx + 2);
  idx += 3;
  uint32_t state = 0;
  if (count) {                                             // the string begins with the state, R bits
    state = __funnelshift_l(w1, w0, bitpos) >> (32u - R);
    bitpos += R;
    if (bitpos >= 32u) { w0 = w1; w1 = w2; w2 = load_word(idx); ++idx; bitpos -= 32u; }
  }
  const uint32_t stride = 1u << stride_log;
  uint32_t st = tab_lane + (state << stride_log);
  uint32_t z = 0;                                          // the lane's next position
  const uint32_t sp_limit = stage_abs + word_limit * 4u;
  uint32_t sp = min(stage_abs + min(idx, word_limit) * 4u, sp_limit);   // (lengths that lead outside are flagged below)
  const bool vec_ok = (reinterpret_cast<uintptr_t>(out_strip) & 15u) == 0;
  const uint4 fill4 = make_uint4(fill, fill, fill, fill);

  for (uint32_t t0 = 0; t0 < rows; t0 += P) {
    const uint32_t lim = min((t0 + P) * E, count);
    const uint32_t abase = win_abs + lane * ES * E - t0 * RB;
    __syncwarp();
    if (STAGED) {
      if (SHORT || wide_steps)
        strip_window_walk<ES, 4, SHORT, PIECES>(st, bitpos, w0, w1, w2, sp, z, tab_lane, stride, abase, lim, unit, sp_limit,
                                                magic, 31u * E * ES);
      else
        strip_window_walk<ES, 2, false, PIECES>(st, bitpos, w0, w1, w2, sp, z, tab_lane, stride, abase, lim, unit, sp_limit,
                                                magic, 31u * E * ES);
    } else {                                               // the same walk in plain code, words from global memory
      bool any = true;
      while (any) {
        const uint32_t ea = lds_u32(st), eb = SHORT ? 0u : lds_u32(st + 4u);
        const uint32_t nb = SHORT ? (ea >> 16) & 15u : ea & 31u, zn = z + (SHORT ? (ea >> 20) & 15u : (ea >> 8) & 15u);
        const bool act = zn < lim;
        if (act) {
          const uint32_t q = SHORT ? ea >> 24 : ES == 4 ? ea >> 16 : eb, val = SHORT ? ea : ES == 4 ? eb : ea >> 16;
          sts_elem<ES>(PIECES ? abase + zn * ES + (zn / E) * (31u * E * ES) : abase + zn * RB, val);
          const uint32_t x = __funnelshift_l(w1, w0, bitpos);
          st = tab_lane + (__funnelshift_l(x, q, nb) << stride_log);
          z = zn + 1u;
          bitpos += nb;
          if (bitpos >= 32u) { w0 = w1; w1 = w2; w2 = load_word(idx); ++idx; bitpos -= 32u; }
        }
        any = __any_sync(kFull, act);
      }
    }
    __syncwarp();
    // the window is complete: write it out and fill it again.  Its rows are contiguous in the
    // output for strips (one bulk store); for channels every row is a store of its own.
    if (t0 == 0 && ((lane_early >> 8) & 1u)) asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t wrows = min(P, rows - t0);
    const uint32_t wbytes = (wrows - 1u) * RB + (t0 + wrows == rows ? last_row_bytes : RB);
    uint8_t* gdst = out_strip + size_t(t0) * row_stride;
    const bool more = t0 + P < rows;
    if (vec_ok && (wbytes & 15u) == 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (row_stride == RB) {                          // rows side by side in the output: one store
        if (lane == 0) {
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" :: "l"(gdst), "r"(win_abs), "r"(wbytes) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        }
      } else {
        bool mine = false;
        for (uint32_t r = lane; r < wrows; r += 32u) {
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                       :: "l"(gdst + size_t(r) * row_stride), "r"(win_abs + r * RB), "r"(RB) : "memory");
          mine = true;
        }
        if (mine) {
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        }
      }
      __syncwarp();
      if (more)
        for (uint32_t i = lane * 16u; i < kStripWindow; i += 512u) sts_v4(win_abs + i, fill4);
    } else {
      // ragged ends (a layer's last strip) and outputs off a 16-byte boundary leave through registers
      for (uint32_t r = 0; r < wrows; ++r) {
        const uint32_t rb = (t0 + r + 1u == rows) ? last_row_bytes : RB;
        uint8_t* grow = gdst + size_t(r) * row_stride;
        for (uint32_t i = lane * ES; i < rb; i += 32u * ES) {
          const uint32_t a = win_abs + r * RB + i;
          const uint32_t v = ES == 1 ? lds_u32(a & ~3u) >> (8u * (a & 3u)) : ES == 2 ? lds_u16(a) : lds_u32(a);
          stg_elem<ES>(grow + i, v);
        }
      }
      __syncwarp();
      if (more)
        for (uint32_t i = lane * 16u; i < kStripWindow; i += 512u) sts_v4(win_abs + i, fill4);
    }
  }
  if (STAGED) {
    if (sp >= sp_limit) bad |= ANS_STATUS_BAD_LENGTH;
    idx = (sp - stage_abs) >> 2;
  }
  // What is left of the lane lies inside the run of the entry it stopped at: zero-bit states,
  // the dominant symbol already in place.  Walk them one by one to reach the final state.
  uint32_t s = (st - tab_lane) >> stride_log;
  for (uint32_t left = count - z; left != 0 && left <= uint32_t(kMaxRun); --left) s = lds_u16(succ_abs + s * 2u);
  if (count - z > uint32_t(kMaxRun)) bad |= ANS_STATUS_BAD_FINAL_STATE;
  if (s != 0) bad |= ANS_STATUS_BAD_FINAL_STATE;
  // the lane must have used exactly its bits
  const uint32_t used = (idx - 3u) * 32u + bitpos - bit0;
  if (used != len) bad |= ANS_STATUS_BAD_LENGTH;
  return bad;
}

__global__ void __launch_bounds__(kStripWarps * 32) ans_decode_strips_kernel(const __grid_constant__ StripArgs args) {
  extern __shared__ __align__(16) uint8_t sm[];
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  // dynamic shared memory: [table, in copies][successors][windows][stages], each 16-byte aligned
  const uint32_t sm_abs = smem_u32(sm);
  const uint32_t tab_abs = sm_abs;
  const uint32_t succ_abs = tab_abs + args.table_bytes;
  const uint32_t win_abs = succ_abs + args.succ_bytes + warp * kStripWindow;
  const uint32_t stage_abs = succ_abs + args.succ_bytes + kStripWarps * kStripWindow + warp * args.stage_bytes;

  // let the next launch of the stream get its CTAs in place while this one runs (it waits, as this
  // one does below, before it touches memory)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // the layer of this CTA: its first CTA is the last one at or before blockIdx.x
  int lo = 0;
  if (args.ctas <= kStripCtaTable) {
    lo = args.cta_layer[blockIdx.x];
  } else {
    int hi = args.n_layers;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (args.cta_begin[mid] <= blockIdx.x) lo = mid; else hi = mid;
    }
  }
  const StripLayer& L = args.layer[lo];
  const uint32_t zero_point = L.packed & 0xFFu, R = (L.packed >> 8) & 15u, bitwidth = (L.packed >> 12) & 15u;
  const int dtype = static_cast<int>((L.packed >> 16) & 3u);
  const uint32_t G = (L.packed >> 18) & 127u, piece = L.packed >> 25;
  const uint32_t es = dtype == ANS_U8 ? 1u : dtype == ANS_F32 ? 4u : 2u;
  const uint32_t sub = (blockIdx.x - args.cta_begin[lo]) * kStripWarps + warp;
  const bool have = sub < L.n_sub;

  // whatever an earlier launch of the stream wrote is visible from here on (unless the caller has
  // stated that the inputs were settled before that launch: then the wait comes after the table
  // and the bytes have been fetched, before anything is written)
  if (!args.early) asm volatile("griddepcontrol.wait;" ::: "memory");
  // everything the CTA needs from memory is requested before any of it is used: the
  // sub-stream's offsets, the table's header and its entries (the first batch)
  uint64_t off0 = 0, off1 = 0;
  if (have) {
    off0 = __ldg(L.sub_offsets + sub);
    off1 = __ldg(L.sub_offsets + sub + 1);
  }
  const TableHeader* hdr = reinterpret_cast<const TableHeader*>(L.blob);
  const uint32_t* g_single = reinterpret_cast<const uint32_t*>(L.blob + single_offset());
  const uint32_t* g_multi = reinterpret_cast<const uint32_t*>(L.blob + multi_offset(static_cast<int>(R)));
  const uint32_t h_magic = __ldg(&hdr->magic), h_log = __ldg(&hdr->table_log), h_alphabet = __ldg(&hdr->alphabet),
                 h_dominant = __ldg(&hdr->dominant);
  const uint32_t n_states = 1u << R;
  uint32_t gm[kStripBatch], gs[kStripBatch];
  auto request_entries = [&](uint32_t b0) {
#pragma unroll
    for (uint32_t k = 0; k < kStripBatch; ++k) {
      const uint32_t i = b0 + k * blockDim.x + threadIdx.x;
      gm[k] = i < n_states ? __ldg(g_multi + i) : 0u;
      gs[k] = i < n_states ? __ldg(g_single + i) : 0u;
    }
  };
  request_entries(0);

  // the sub-stream's bytes: asynchronous 16-byte copies into shared memory, started as soon as its
  // offsets are here, so that they travel while the table is being staged.  Both ends on 16-byte
  // boundaries, inside the stream.
  uint32_t bad = 0;
  uint64_t extent = 0;
  if (have) {
    extent = off1 - off0;
    if (off1 < off0 || off1 > L.stream_bytes || ((off0 | off1) & 15u) || extent > 0xFFFFFFF0ull) {
      extent = 0;
      off0 = 0;
      bad |= ANS_STATUS_BAD_LENGTH;
    }
  }
  const bool staged = extent > 0 && extent + kStripPad <= args.stage_bytes;
  if (staged) {
    const uint8_t* src = L.stream + off0;
    for (uint32_t o = lane * 16u; o < static_cast<uint32_t>(extent); o += 512u)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(stage_abs + o), "l"(src + o) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (uint32_t i = lane; i < kStripPad / 4u; i += 32u)
      asm volatile("st.shared.u32 [%0], %1;" :: "r"(stage_abs + static_cast<uint32_t>(extent) + i * 4u), "r"(0u) : "memory");
  }

  // stage the table: copies interleaved entry by entry (entry i of copy c at slot i * copies + c;
  // lane l reads copy l mod copies), the dequantised value folded into every entry
  // (a table smaller than the launch's largest uses the room for more copies, up to one per lane)
  const bool short_entries = R <= 8u && es != 4u;
  const uint32_t entry_log = short_entries ? 2u : 3u;
  const uint32_t rep_log = min(short_entries ? 5u : 4u, 31u - static_cast<uint32_t>(__clz(args.table_bytes >> (R + entry_log))));
  const uint32_t reps = 1u << rep_log;
  const uint32_t stride_log = entry_log + rep_log;
  const uint32_t tab_lane = tab_abs + ((lane & (reps - 1u)) << entry_log);
  uint32_t most_bits = 0;
  for (uint32_t b0 = 0; b0 < n_states; b0 += blockDim.x * kStripBatch) {
    if (b0 != 0) request_entries(b0);
#pragma unroll
    for (uint32_t k = 0; k < kStripBatch; ++k) {
      const uint32_t i = b0 + k * blockDim.x + threadIdx.x;
      if (i < n_states) {
        const uint32_t val = dequant_bits(static_cast<int>(entry_sym(gm[k])), static_cast<int>(zero_point), L.scale, dtype);
        const uint2 e = to_strip_entry(gm[k], val, es != 4u);
        const uint32_t e1 = to_strip_entry_short(gm[k], val);
        const uint32_t slot = tab_abs + (i << stride_log);
        if (stride_log >= 4u) {
          // the entry's copies lie side by side: written 16 bytes at a time, every lane starting
          // at another 16 bytes so that the stores of a warp spread over the banks
          const uint4 v = short_entries ? make_uint4(e1, e1, e1, e1) : make_uint4(e.x, e.y, e.x, e.y);
          const uint32_t pieces = 1u << (stride_log - 4u), turn = lane & (pieces - 1u);
#pragma unroll
          for (uint32_t p = 0; p < 8u; ++p)
            if (p < pieces) sts_v4(slot + ((p ^ turn) << 4), v);
        } else {
          for (uint32_t c = 0; c < reps; ++c) {
            const uint32_t a = slot + (c << entry_log);
            if (short_entries) asm volatile("st.shared.u32 [%0], %1;" :: "r"(a), "r"(e1) : "memory");
            else asm volatile("st.shared.v2.u32 [%0], {%1, %2};" :: "r"(a), "r"(e.x), "r"(e.y) : "memory");
          }
        }
        asm volatile("st.shared.u16 [%0], %1;" :: "r"(succ_abs + i * 2u), "r"(entry_newx(gs[k])) : "memory");
        most_bits = max(most_bits, entry_nb(gm[k]));
      }
    }
  }
  if (threadIdx.x == 0 && (h_magic != kTableMagic || h_log != R || h_alphabet > (1u << bitwidth))) bad |= ANS_STATUS_BAD_SYMBOL;
  // four look-ups share one 32-bit extract only if no state takes more than 8 bits
  const bool wide_steps = __syncthreads_or(most_bits > 8u) == 0;

  if (have) {
    // the warp's window starts out holding the dominant symbol's value (the symbol of every
    // zero-bit state; without one no look-up skips a position and the fill is never seen)
    const uint32_t dom = dequant_bits(static_cast<int>(h_dominant < 256u ? h_dominant : 0u), static_cast<int>(zero_point), L.scale, dtype);
    const uint32_t fill = es == 4u ? dom : es == 2u ? (dom & 0xFFFFu) * 0x10001u : (dom & 0xFFu) * 0x01010101u;
    const uint4 fill4 = make_uint4(fill, fill, fill, fill);
    for (uint32_t i = lane * 16u; i < kStripWindow; i += 512u) sts_v4(win_abs + i, fill4);

    // the place of this sub-stream in the output
    const uint64_t chunk = sub / G;
    const uint32_t g = sub - static_cast<uint32_t>(chunk) * G;
    const uint64_t c0 = chunk * L.chunk_symbols;
    const uint32_t nc = static_cast<uint32_t>(min(uint64_t(L.chunk_symbols), L.n_symbols - c0));
    StripGeom geo;
    uint8_t* out_strip;
    uint32_t ns;                                           // symbols of the sub-stream
    if (piece) {
      // channels: lanes 32 g .. 32 g + 31 of a chunk dealt in pieces; every lane owns nc / W symbols
      const uint32_t W = 32u * G;
      geo.count = nc / W;
      geo.E = piece;
      geo.rows = geo.count / piece;
      geo.last_row_bytes = 32u * piece * es;
      geo.row_stride = W * piece * es;
      ns = 32u * geo.count;
      out_strip = L.out + (c0 + uint64_t(32u * g) * piece) * es;
    } else {
      // strips: a contiguous part of the chunk dealt round-robin
      const uint32_t S = L.chunk_symbols / (32u * G);
      const uint32_t sfirst = g * 32u * S;                 // (inside the chunk: below 2^32)
      ns = nc > sfirst ? min(nc - sfirst, 32u * S) : 0u;
      geo.count = lane_symbols(ns, 32u, lane);
      geo.E = 1u;
      geo.rows = (ns + 31u) >> 5;
      geo.last_row_bytes = (ns - (geo.rows ? (geo.rows - 1u) * 32u : 0u)) * es;
      geo.row_stride = 32u * es;
      out_strip = L.out + (c0 + sfirst) * es;
    }
    const uint32_t ext_words = static_cast<uint32_t>(extent >> 2);
    const uint32_t* words = reinterpret_cast<const uint32_t*>(L.stream + off0);

    if (staged) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncwarp();
    }
    if (extent == 0) {
      // unusable offsets (flagged above): nothing is read; an empty strip needs nothing either
      if (ns != 0) bad |= ANS_STATUS_BAD_LENGTH;
    } else {
#define ANSB_SCALL(ES_, ST_, SH_)                                                                     \
  bad |= piece > 1u ? decode_strip<ES_, ST_, SH_, true>(tab_lane, stride_log, succ_abs, win_abs, stage_abs, words, ext_words, \
                                                        R, geo.count, geo.rows, geo.E, geo.last_row_bytes, geo.row_stride, \
                                                        out_strip, fill, wide_steps, args.unit, lane | (args.early << 8)) \
                    : decode_strip<ES_, ST_, SH_, false>(tab_lane, stride_log, succ_abs, win_abs, stage_abs, words, ext_words, \
                                                         R, geo.count, geo.rows, geo.E, geo.last_row_bytes, geo.row_stride, \
                                                         out_strip, fill, wide_steps, args.unit, lane | (args.early << 8))
      if (short_entries) {
        if (staged) { if (es == 1u) ANSB_SCALL(1, true, true); else ANSB_SCALL(2, true, true); }
        else { if (es == 1u) ANSB_SCALL(1, false, true); else ANSB_SCALL(2, false, true); }
      } else if (staged) {
        if (es == 1u) ANSB_SCALL(1, true, false); else if (es == 2u) ANSB_SCALL(2, true, false); else ANSB_SCALL(4, true, false);
      } else {
        if (es == 1u) ANSB_SCALL(1, false, false); else if (es == 2u) ANSB_SCALL(2, false, false); else ANSB_SCALL(4, false, false);
      }
#undef ANSB_SCALL
    }
  }
  bad = __reduce_or_sync(kFull, bad);
  if (args.early && bad) asm volatile("griddepcontrol.wait;" ::: "memory");   // (a warp that wrote nothing has not waited yet)
  if (lane == 0 && bad && args.d_status) atomicOr(args.d_status, bad);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
struct StripFacts { int sms = 0; int smem_sm = 0; int smem_block = 0; size_t smem_set = 0; };
static StripFacts g_strip_facts[64];     // per device; racing writers store equal values

int launch_strips(const ans_layer_desc* h_descs, int n_layers, uint8_t* d_symbols_override, uint32_t* d_status,
                  cudaStream_t st) {
  int dev = 0;
  ANSB_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return ANS_ERR_UNSUPPORTED;
  StripFacts& facts = g_strip_facts[dev];
  if (!facts.sms) {
    int sms = 0, per_sm = 0, per_block = 0;
    ANSB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ANSB_CUDA(cudaDeviceGetAttribute(&per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev));
    ANSB_CUDA(cudaDeviceGetAttribute(&per_block, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    ANSB_CUDA(cudaFuncSetAttribute(ans_decode_strips_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                   cudaSharedmemCarveoutMaxShared));
    facts.smem_sm = per_sm;
    facts.smem_block = per_block;
    facts.sms = sms;
  }
  for (int l0 = 0; l0 < n_layers; l0 += kStripParamLayers) {
    const int cnt = (n_layers - l0) < kStripParamLayers ? (n_layers - l0) : kStripParamLayers;
    StripArgs a{};
    a.n_layers = 0;
    a.d_status = d_status;
    a.unit = 1u;
    a.early = 1u;
    bool idle = true;
    int max_log = 1;
    uint64_t ctas = 0;
    size_t max_avg_sub = 0, one_table = 0;
    for (int i = 0; i < cnt; ++i) {
      const ans_layer_desc& d = h_descs[l0 + i];
      if (d.work_count == 0) continue;
      const uint64_t n_sub = subs_of(d);
      if (n_sub > 0xFFFFFFFFull) return ANS_ERR_UNSUPPORTED;
      if (!(d.flags & ANS_DESC_INPUTS_SETTLED)) a.early = 0u;
      if (!(d.flags & ANS_DESC_OUTPUT_IDLE)) idle = false;
      StripLayer& L = a.layer[a.n_layers];
      L.blob = static_cast<const uint8_t*>(d.d_table);
      L.stream = d.d_stream;
      L.sub_offsets = d.d_sub_offsets;
      L.out = d_symbols_override ? d_symbols_override : static_cast<uint8_t*>(d.d_out);
      L.stream_bytes = d.stream_bytes;
      L.n_symbols = d.n_symbols;
      L.chunk_symbols = d.chunk_symbols;
      L.n_sub = static_cast<uint32_t>(n_sub);
      L.scale = d.scale;
      const uint32_t dtype = d_symbols_override ? ANS_U8 : static_cast<uint32_t>(d.out_dtype);
      L.packed = static_cast<uint32_t>(d.zero_point) | (static_cast<uint32_t>(d.table_log) << 8) |
                 (static_cast<uint32_t>(d.bitwidth) << 12) | (dtype << 16) | ((d.lanes / 32u) << 18) |
                 ((d.layout == ANS_LAYOUT_CHANNELS ? d.piece_symbols : 0u) << 25);
      if (d.layout == ANS_LAYOUT_CHANNELS && d.piece_symbols * (dtype == ANS_U8 ? 1u : dtype == ANS_F32 ? 4u : 2u) > 128u)
        return ANS_ERR_UNSUPPORTED;
      a.cta_begin[a.n_layers] = static_cast<uint32_t>(ctas);
      ctas += d.work_count;
      ++a.n_layers;
      if (d.table_log > max_log) max_log = d.table_log;
      const size_t tb = size_t((d.table_log <= 8 && dtype != ANS_F32) ? 4 : 8) << d.table_log;   // one copy, in its entry form
      if (tb > one_table) one_table = tb;
      const size_t avg = d.stream_bytes / n_sub;
      if (avg > max_avg_sub) max_avg_sub = avg;
    }
    if (a.n_layers == 0) continue;
    if (a.early && idle) a.early = 2u;
    if (ctas > 0x7FFFFFFFull) return ANS_ERR_UNSUPPORTED;
    a.cta_begin[a.n_layers] = static_cast<uint32_t>(ctas);
    a.max_log = static_cast<uint32_t>(max_log);
    a.ctas = static_cast<uint32_t>(ctas);
    if (ctas <= kStripCtaTable)
      for (int l = 0; l < a.n_layers; ++l)
        for (uint32_t c = a.cta_begin[l]; c < a.cta_begin[l + 1]; ++c) a.cta_layer[c] = static_cast<uint8_t>(l);

    // shared memory of a CTA: table copies, successors, barriers, four windows, four staging buffers.
    // A staging buffer holds the largest layer-average sub-stream plus a margin (a longer one is read
    // from global memory).  What room is left under the share of an SM that one wave of CTAs
    // leaves to each goes to more copies of the table (fewer bank conflicts on the look-ups).
    size_t want = max_avg_sub + max_avg_sub / 8 + 256 + kStripPad;
    want = (want + 127) & ~size_t(127);
    const size_t succ = ((size_t(2) << max_log) + 15) & ~size_t(15);
    const size_t fixed = succ + size_t(kStripWarps) * kStripWindow;
    const size_t block_max = static_cast<size_t>(facts.smem_block);
    if (fixed + one_table + kStripWarps * 1024 > block_max) return ANS_ERR_UNSUPPORTED;
    size_t stage = want;
    if (fixed + one_table + kStripWarps * stage > block_max) stage = ((block_max - fixed - one_table) / kStripWarps) & ~size_t(127);
    uint64_t per_sm = (ctas + facts.sms - 1) / facts.sms;
    if (per_sm > 8) per_sm = 8;
    if (per_sm < 1) per_sm = 1;
    // a launch that never waits for the one before it shares the SMs with that launch's CTAs for
    // as long as both run: room for as many CTAs as the registers allow (eight) is then worth
    // more than copies.  (A launch that waits before its first write gains nothing from it: 14.8
    // against 12 us per launch on the ResNet-50 workload.)
    if (a.early == 2u) per_sm = 8;
    size_t cap = static_cast<size_t>(facts.smem_sm) / per_sm;
    cap = cap > 2048 ? cap - 1024 : cap;                   // the system's share per CTA
    if (cap > block_max) cap = block_max;
    size_t smem = fixed + one_table + kStripWarps * stage;
    uint32_t rep_log = 0;
    while (rep_log < 5 && smem + (one_table << rep_log) <= cap) {
      smem += one_table << rep_log;
      ++rep_log;
    }
    a.succ_bytes = static_cast<uint32_t>(succ);
    a.table_bytes = static_cast<uint32_t>(one_table << rep_log);
    a.stage_bytes = static_cast<uint32_t>(stage);
    if (smem > facts.smem_set) {
      ANSB_CUDA(cudaFuncSetAttribute(ans_decode_strips_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(smem)));
      facts.smem_set = smem;
    }
    // launched so that it may take its place on the device while the launch before it on the
    // stream is still running; the kernel waits for that launch before it reads memory
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(ctas));
    cfg.blockDim = dim3(kStripWarps * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ANSB_CUDA(cudaLaunchKernelEx(&cfg, ans_decode_strips_kernel, a));
  }
  return ANS_OK;
}

}  // namespace ansb
