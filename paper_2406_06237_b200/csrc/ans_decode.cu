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
#include "ans_decode_common.cuh"
#include "ans_walk_interleaved.cuh"
#include "ans_walk_lockstep.cuh"
#include "ans_walk_prewalk.cuh"
#include "ans_walk_quads.cuh"

namespace ansb {

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
  __shared__ uint32_t s_dom, s_maxadv, s_maxnb;
  uint32_t parity = 0;
  // let the next launch of the stream take its place as this one's CTAs leave; this launch waits
  // for the work before it either here, before it reads anything, or (inputs settled before that
  // work began, as the descriptors' flags say) only before its first write to device memory
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!args.early) asm volatile("griddepcontrol.wait;" ::: "memory");
  bool waited = args.early != 1u;

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
    // quads with 1-byte outputs: one-word entries, so twice the copies (up to 32) in the same room;
    // quads with 2-byte outputs and 2^10 to 2^12 states likewise (smaller tables already have a
    // conflict-free copy per lane pair in the two-word form, larger ones do not fit one word)
    const bool short_entries = kQuads && (args.d_symbols_override || L.out_dtype == ANS_U8 ||
                                          (L.out_dtype == ANS_BF16 && R >= 10 && R <= 12));
    const uint32_t rep_two = min(4u, args.rep_log + (args.max_log - static_cast<uint32_t>(R)));
    const uint32_t rep_log = (kPrivate && !lock) ? args.rep_log : short_entries ? rep_two + 1u : rep_two;
    const uint32_t reps = 1u << rep_log;
    const uint32_t stride_log = (short_entries ? 2u : 3u) + rep_log;
    const uint32_t tab_lane = tab_abs + (lane & (reps - 1u)) * (short_entries ? 4u : 8u);
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
          uint64_t pol;                                   // (the bytes are read once: they need not stay in L2)
          asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
          asm volatile(
              "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
              :: "r"(stage_abs), "l"(L.d_stream + it.off0), "r"(bytes), "r"(bar), "l"(pol) : "memory");
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
    // (a warp whose wait on a copy ran out takes no further work: it only keeps the CTA's
    // barriers company, so that nothing is issued on a barrier whose phase never completed)
    const bool have_first = !gave_up && warp_sub(cursor, first_sub);
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
          s_maxnb = 0u;
          if (h_magic != kTableMagic || h_log != uint32_t(R) || h_alphabet > (1u << L.bitwidth))
            bad |= ANS_STATUS_BAD_SYMBOL;
        }
        __syncthreads();
      }
      uint32_t longest = 0, most_bits = 0;
#pragma unroll
      for (uint32_t k = 0; k < kStageBatch; ++k) {
        const uint32_t i = b0 + k * blockDim.x + threadIdx.x;
        if (i < n_states) {
          const uint2 e = kQuads ? to_quads_entry(g[k], vals[entry_sym(g[k])], es != 4)
                                 : to_smem_entry(g[k], vals[entry_sym(g[k])], 32u * static_cast<uint32_t>(es));
          // every lane starts at another copy: the stores of a warp spread over the banks
          if (short_entries) {
            const uint32_t qq = entry_newx(g[k]) >> entry_nb(g[k]);
            const uint32_t e1 = es == 2 ? entry_nb(g[k]) | (qq << 4) | (vals[entry_sym(g[k])] << 16)
                                        : entry_nb(g[k]) | (qq << 8) | (vals[entry_sym(g[k])] << 24);
            for (uint32_t c = 0; c < reps; ++c)
              reinterpret_cast<uint32_t*>(tab)[(i << rep_log) + ((c + lane) & (reps - 1u))] = e1;
          } else {
            for (uint32_t c = 0; c < reps; ++c) tab[(i << rep_log) + ((c + lane) & (reps - 1u))] = e;
          }
          if (kPrivate && !lock) succ[i] = static_cast<uint16_t>(entry_newx(g1[k]));
          longest = max(longest, entry_run(g[k]) + 1u);
          most_bits = max(most_bits, entry_nb(g[k]));
        }
      }
      longest = __reduce_max_sync(kFull, longest);
      if (lane == 0 && longest > 1u) atomicMax(&s_maxadv, longest);
      // the lockstep walks share one 32-bit extract among four look-ups when no state of this
      // table takes more than 8 bits (a table of 2^12 states over a handful of symbols does not)
      most_bits = __reduce_max_sync(kFull, most_bits);
      if (lane == 0) atomicMax(&s_maxnb, most_bits);
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
        if (!__all_sync(kFull, ok)) {                     // the copy never landed: stop this warp's work
          bad |= wbad | kStatusTimeout;
          gave_up = true;
          continue;
        }
        parity ^= 1u;
        __syncwarp();
      }
      if (!waited) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
      }
      if (kPrivate) {
        const uint32_t* words = reinterpret_cast<const uint32_t*>(g_bytes);
#define ANSB_CALL(ES_, ST_)                                                                              \
  wbad |= decode_private<ES_, ST_>(tab_lane, stride_log, succ_abs, ring_abs, stage_abs, park_abs, ring, dom, words, \
                                   ext_words, wbeg, wend, lane == 31, state, my_count, rows, min_count, \
                                   out_row0, rsb, lane, s_maxadv)
#define ANSB_LCALL(ES_, ST_)                                                                             \
  wbad |= decode_lockstep<ES_, ST_>(tab_lane, stride_log, stage_abs, words, ext_words, wbeg, wend, lane == 31, \
                                    state, my_count, rows, min_count, out_row0, W / 32u, lane, s_maxnb <= 8u, args.unit)
#define ANSB_QCALL(ES_, ST_, SH_)                                                                        \
  wbad |= decode_quads<ES_, ST_, SH_>(tab_lane, stride_log, stage_abs, words, ext_words, wbeg, wend, lane == 31, \
                                      state, my_count, min_count, out_row0 + size_t(lane) * 4u * ES_, W / 32u, \
                                      s_maxnb <= 8u, args.unit)
        if constexpr (kQuads) {                           // (1-byte outputs: one-word entries, see above)
          if (staged) {
            if (es == 1) ANSB_QCALL(1, true, true);
            else if (es == 2) { if (short_entries) ANSB_QCALL(2, true, true); else ANSB_QCALL(2, true, false); }
            else ANSB_QCALL(4, true, false);
          } else {
            if (es == 1) ANSB_QCALL(1, false, true);
            else if (es == 2) { if (short_entries) ANSB_QCALL(2, false, true); else ANSB_QCALL(2, false, false); }
            else ANSB_QCALL(4, false, false);
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
  if (args.early && bad) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (lane == 0 && bad && args.d_status) atomicOr(args.d_status, bad);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
constexpr int kMaxDevices = 64;
struct LaunchShape { size_t smem = 0; int warps = 0; int per_sm = 0; };
struct DeviceFacts { int sms = 0; int smem_max = 0; LaunchShape shape[8]; };
static DeviceFacts g_facts[kMaxDevices];    // remembered per device; racing writers store equal values

int launch_strips(const ans_layer_desc* h_descs, int n_layers, uint8_t* d_symbols_override, uint32_t* d_status,
                  cudaStream_t st);                       // ans_decode_strips.cu

static int launch(const ans_layer_desc* d_descs, const ans_layer_desc* h_descs, int n_layers,
                  uint8_t* d_symbols_override, uint32_t* d_status, cudaStream_t st) {
  int max_log = 1, busy_layers = 0;
  uint32_t flags_all = ~0u;                               // flags every layer with work carries
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
      flags_all &= h_descs[l].flags;
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
  if (layout == ANS_LAYOUT_STRIPS || layout == ANS_LAYOUT_CHANNELS)
    return launch_strips(h_descs, n_layers, d_symbols_override, d_status, st);

  LaunchArgs a{};
  a.d_descs = d_descs;
  if (!d_descs) a.one = h_descs[0];
  a.n_layers = n_layers;
  a.total_work = static_cast<uint32_t>(total);
  a.d_status = d_status;
  a.d_symbols_override = d_symbols_override;
  a.unit = 1u;
  a.early = !(flags_all & ANS_DESC_INPUTS_SETTLED) ? 0u : (flags_all & ANS_DESC_OUTPUT_IDLE) ? 2u : 1u;
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
  // launched so that it may take its place on the device while the work before it on the stream
  // is still running; the kernel waits for that work before it reads (or, with the descriptors'
  // flags, before it writes) anything
  const void* fns[8] = {
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_QUADS, true, false>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_QUADS, true, true>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, true, false>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, true, true>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, false, false>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_PRIVATE, false, false>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_INTERLEAVED, true, false>),
      reinterpret_cast<const void*>(&ans_decode_kernel<ANS_LAYOUT_INTERLEAVED, true, true>)};
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(static_cast<unsigned>(warps) * 32u);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  void* kargs[1] = {&a};
  ANSB_CUDA(cudaLaunchKernelExC(&cfg, fns[launch_which & 7], kargs));
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
  ApiRange range("ans_decode_layer");
  if (!h_desc || !d_status) return ANS_ERR_INVALID_ARG;
  if (!d_symbols_out && h_desc->n_symbols) return ANS_ERR_INVALID_ARG;
  ans_layer_desc d = *h_desc;
  d.flags &= ~ANS_DESC_OUTPUT_IDLE;                        // (that flag speaks of d_out, which this call does not write)
  const int rc = ans_plan_batch(&d, 1, nullptr);
  if (rc != ANS_OK) return rc;
  if (d.n_symbols == 0) return validate_desc(d, false);
  return launch(nullptr, &d, 1, d_symbols_out, d_status, static_cast<cudaStream_t>(stream));
}

ANS_EXPORT int ans_decode_dequant(const ans_layer_desc* h_desc, uint32_t* d_status, void* stream) {
  ApiRange range("ans_decode_dequant");
  if (!h_desc || !d_status) return ANS_ERR_INVALID_ARG;
  ans_layer_desc d = *h_desc;
  const int rc = ans_plan_batch(&d, 1, nullptr);
  if (rc != ANS_OK) return rc;
  return launch(nullptr, &d, 1, nullptr, d_status, static_cast<cudaStream_t>(stream));
}

ANS_EXPORT int ans_decode_dequant_batch(const ans_layer_desc* d_descs, const ans_layer_desc* h_descs,
                                        int n_layers, uint32_t* d_status, void* stream) {
  ApiRange range("ans_decode_dequant_batch");
  if (n_layers < 0 || !d_status) return ANS_ERR_INVALID_ARG;
  if (n_layers == 0) return ANS_OK;
  if (!h_descs || (!d_descs && lane_meta_size(h_descs[0].layout))) return ANS_ERR_INVALID_ARG;
  return launch(d_descs, h_descs, n_layers, nullptr, d_status, static_cast<cudaStream_t>(stream));
}
