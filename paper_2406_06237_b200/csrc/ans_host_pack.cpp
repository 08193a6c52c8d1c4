// Host-side packer: histogram normalisation and tANS encoding into the containers the
// decode kernels read.  CPU only, off the inference path (the paper compresses offline,
// Section III-A).  The encoder is table driven: per symbol a threshold decides how many bits a
// state sheds (Section II-A: "following a state transition ... and concatenating the binary
// string that labels the transition"), per (symbol, reduced state) a table gives the next state.
#include <algorithm>
#include <cstring>
#include <thread>
#include <vector>

#include "ans_b200.h"

#define ANS_EXPORT extern "C" __attribute__((visibility("default")))

namespace {

struct EncTable {
  int R = 0;
  uint32_t L = 0;
  uint32_t freq[256] = {};
  uint32_t first[257] = {};          // first[s]: slots handed out before symbol s
  uint32_t max_bits[256] = {};       // bits shed by the large states of s
  uint32_t split[256] = {};          // states below split[s] shed one bit less
  std::vector<uint16_t> next_index;  // [first[s] + reduced - freq[s]] -> state index
  bool ok = false;
};

inline uint32_t reverse_bits(uint32_t v, int R) {
  v = ((v >> 1) & 0x55555555u) | ((v & 0x55555555u) << 1);
  v = ((v >> 2) & 0x33333333u) | ((v & 0x33333333u) << 2);
  v = ((v >> 4) & 0x0F0F0F0Fu) | ((v & 0x0F0F0F0Fu) << 4);
  v = ((v >> 8) & 0x00FF00FFu) | ((v & 0x00FF00FFu) << 8);
  v = (v >> 16) | (v << 16);
  return v >> (32 - R);
}

bool make_enc_table(const uint32_t* freqs, int A, int R, EncTable& T) {
  T.R = R;
  T.L = 1u << R;
  uint64_t acc = 0;
  for (int s = 0; s < 256; ++s) {
    T.freq[s] = s < A ? freqs[s] : 0;
    T.first[s] = static_cast<uint32_t>(acc);
    acc += T.freq[s];
  }
  T.first[256] = static_cast<uint32_t>(acc);
  if (acc != T.L) return false;
  for (int s = 0; s < 256; ++s) {
    const uint32_t f = T.freq[s];
    if (!f) continue;
    const int hb = 31 - __builtin_clz(f);
    T.max_bits[s] = static_cast<uint32_t>(R - hb);
    T.split[s] = f << T.max_bits[s];
  }
  // walk the table positions upwards; position i was the bitrev(i)-th slot handed out, which
  // tells whose it is; the visit order numbers that symbol's states upwards
  std::vector<uint8_t> owner(T.L);
  for (int s = 0; s < 256; ++s)
    for (uint32_t j = T.first[s]; j < T.first[s + 1]; ++j) owner[j] = static_cast<uint8_t>(s);
  T.next_index.assign(T.L, 0);
  uint32_t seen[256] = {};
  for (uint32_t i = 0; i < T.L; ++i) {
    const int s = owner[reverse_bits(i, R)];
    T.next_index[T.first[s] + seen[s]++] = static_cast<uint16_t>(i);
  }
  T.ok = true;
  return true;
}

// Encode one lane backwards from state index 0; labels are stored in decode order.
// Returns the initial decode state, or -1 if a symbol has no state.
inline int encode_lane(const EncTable& T, const uint8_t* sym, size_t count, size_t stride,
                       uint8_t* nb_out, uint16_t* val_out) {
  uint32_t x = T.L;                                  // state index 0
  for (size_t t = count; t-- > 0;) {
    const uint32_t s = sym[t * stride];
    const uint32_t f = T.freq[s];
    if (!f) return -1;
    const uint32_t k = T.max_bits[s] - (x < T.split[s] ? 1u : 0u);
    nb_out[t] = static_cast<uint8_t>(k);
    val_out[t] = static_cast<uint16_t>(x & ((1u << k) - 1u));
    x = T.L + T.next_index[T.first[s] + (x >> k) - f];
  }
  return static_cast<int>(x - T.L);
}

struct BitWriter {
  std::vector<uint8_t>& out;
  uint64_t acc = 0;
  int fill = 0;
  explicit BitWriter(std::vector<uint8_t>& o) : out(o) {}
  void put(uint32_t v, int n) {
    acc |= static_cast<uint64_t>(v) << fill;
    fill += n;
    while (fill >= 8) { out.push_back(static_cast<uint8_t>(acc)); acc >>= 8; fill -= 8; }
  }
  void finish(size_t align) {
    if (fill > 0) { out.push_back(static_cast<uint8_t>(acc)); acc = 0; fill = 0; }
    while (out.size() % align) out.push_back(0);
  }
};

inline size_t lane_count(size_t nc, size_t W, size_t lambda) { return nc > lambda ? (nc - lambda + W - 1) / W : 0; }

// Bits from the top of 32-bit words down, a field's high bit first; words go out little-endian.
struct TopBitWriter {
  std::vector<uint8_t>& out;
  uint64_t acc = 0;      // pending bits, left-aligned in the low `fill` positions counted from bit 63
  int fill = 0;
  explicit TopBitWriter(std::vector<uint8_t>& o) : out(o) {}
  void word(uint32_t w) { for (int b = 0; b < 4; ++b) out.push_back(static_cast<uint8_t>(w >> (8 * b))); }
  void put(uint32_t v, int n) {
    if (n == 0) return;
    acc |= static_cast<uint64_t>(v) << (64 - fill - n);
    fill += n;
    if (fill >= 32) { word(static_cast<uint32_t>(acc >> 32)); acc <<= 32; fill -= 32; }
  }
  void finish() { if (fill > 0) { word(static_cast<uint32_t>(acc >> 32)); acc = 0; fill = 0; } }
};

// quads container: symbols a lane owns, and where its t-th symbol sits in the chunk
inline size_t quad_lane_count(size_t nc, size_t W, size_t lambda) {
  const size_t full = nc / 4, rem = nc % 4;
  return 4 * (full > lambda ? (full - lambda + W - 1) / W : 0) + ((rem && full % W == lambda) ? rem : 0);
}
inline size_t quad_position(size_t W, size_t lambda, size_t t) { return ((t / 4) * W + lambda) * 4 + t % 4; }

// One sub-stream of the strips container: `strip` holds its ns symbols (a contiguous part of the
// chunk), dealt to the 32 lanes round-robin.  Appended to `bytes`: the lanes' bit lengths, then
// their strings (state in R bits, then the fields) back to back from the top bit of 32-bit words.
bool pack_strip(const EncTable& T, const uint8_t* strip, size_t ns, std::vector<uint8_t>& bytes,
                std::vector<uint8_t>& nb, std::vector<uint16_t>& val) {
  const size_t base = bytes.size();
  bytes.resize(base + 64, 0);
  const size_t max_lane = (ns + 31) / 32 + 1;
  nb.resize(max_lane);
  val.resize(max_lane);
  TopBitWriter bw(bytes);
  for (size_t k = 0; k < 32; ++k) {
    const size_t cnt = lane_count(ns, 32, k);
    uint64_t len = 0;
    if (cnt) {
      const int init = encode_lane(T, strip + k, cnt, 32, nb.data(), val.data());
      if (init < 0) return false;
      bw.put(static_cast<uint32_t>(init), T.R);
      len = static_cast<uint64_t>(T.R);
      for (size_t t = 0; t < cnt; ++t) { bw.put(val[t], nb[t]); len += nb[t]; }
    }
    if (len > 0xFFFF) return false;
    bytes[base + 2 * k] = static_cast<uint8_t>(len & 0xFF);        // (the writer only appends, so the header stays put)
    bytes[base + 2 * k + 1] = static_cast<uint8_t>(len >> 8);
  }
  bw.finish();
  while ((bytes.size() - base) % 16) bytes.push_back(0);
  return true;
}

// One sub-stream of the channels container: lanes 32 g .. 32 g + 31 of a chunk whose symbols come
// in pieces of E, piece j belonging to lane j mod W; every lane owns cnt symbols.  Bytes as for strips.
bool pack_channels_sub(const EncTable& T, const uint8_t* chunk, size_t cnt, size_t W, size_t E, size_t g,
                       std::vector<uint8_t>& bytes, std::vector<uint8_t>& nb, std::vector<uint16_t>& val,
                       std::vector<uint8_t>& mine) {
  const size_t base = bytes.size();
  bytes.resize(base + 64, 0);
  nb.resize(cnt + 1);
  val.resize(cnt + 1);
  mine.resize(cnt + 1);
  TopBitWriter bw(bytes);
  for (size_t k = 0; k < 32; ++k) {
    uint64_t len = 0;
    if (cnt) {
      const size_t lambda = 32 * g + k;
      for (size_t t = 0; t < cnt; ++t) mine[t] = chunk[((t / E) * W + lambda) * E + t % E];
      const int init = encode_lane(T, mine.data(), cnt, 1, nb.data(), val.data());
      if (init < 0) return false;
      bw.put(static_cast<uint32_t>(init), T.R);
      len = static_cast<uint64_t>(T.R);
      for (size_t t = 0; t < cnt; ++t) { bw.put(val[t], nb[t]); len += nb[t]; }
    }
    if (len > 0xFFFF) return false;
    bytes[base + 2 * k] = static_cast<uint8_t>(len & 0xFF);
    bytes[base + 2 * k + 1] = static_cast<uint8_t>(len >> 8);
  }
  bw.finish();
  while ((bytes.size() - base) % 16) bytes.push_back(0);
  return true;
}

// One sub-stream (32 lanes) into `bytes` (appended) and meta (32 entries).
bool pack_sub(const EncTable& T, const uint8_t* chunk, size_t nc, size_t W, size_t g, int layout,
              std::vector<uint8_t>& bytes, void* meta32, std::vector<uint8_t>& nb, std::vector<uint16_t>& val,
              std::vector<uint8_t>& lane_bytes) {
  const bool quads = layout == ANS_LAYOUT_QUADS;
  const size_t max_lane = quads ? 4 * ((nc / 4 + W - 1) / W) + 4 : lane_count(nc, W, 32 * g);
  nb.resize(32 * max_lane + 1);
  val.resize(32 * max_lane + 1);
  size_t cnt[32];
  int init[32];
  for (size_t k = 0; k < 32; ++k) {
    const size_t lambda = 32 * g + k;
    if (quads) {
      cnt[k] = quad_lane_count(nc, W, lambda);
      lane_bytes.resize(max_lane);                    // the lane's symbols, gathered
      for (size_t t = 0; t < cnt[k]; ++t) lane_bytes[t] = chunk[quad_position(W, lambda, t)];
      init[k] = encode_lane(T, lane_bytes.data(), cnt[k], 1, nb.data() + k * max_lane, val.data() + k * max_lane);
    } else {
      cnt[k] = lane_count(nc, W, lambda);
      init[k] = encode_lane(T, chunk + lambda, cnt[k], W, nb.data() + k * max_lane, val.data() + k * max_lane);
    }
    if (init[k] < 0) return false;
  }
  const size_t base = bytes.size();
  if (quads) {
    uint32_t* meta = static_cast<uint32_t*>(meta32);
    for (size_t k = 0; k < 32; ++k) {
      const size_t word0 = (bytes.size() - base) / 4;
      if (word0 > 0xFFFF) return false;
      meta[k] = static_cast<uint32_t>(init[k]) | (static_cast<uint32_t>(word0) << 16);
      TopBitWriter bw(bytes);
      for (size_t t = 0; t < cnt[k]; ++t) bw.put(val[k * max_lane + t], nb[k * max_lane + t]);
      bw.finish();
    }
  } else if (layout == ANS_LAYOUT_PRIVATE) {
    uint32_t* meta = static_cast<uint32_t*>(meta32);
    for (size_t k = 0; k < 32; ++k) {
      const size_t word0 = (bytes.size() - base) / 4;
      if (word0 > 0xFFFF) return false;
      meta[k] = static_cast<uint32_t>(init[k]) | (static_cast<uint32_t>(word0) << 16);
      BitWriter bw(bytes);
      for (size_t t = 0; t < cnt[k]; ++t) bw.put(val[k * max_lane + t], nb[k * max_lane + t]);
      bw.finish(4);
    }
  } else {
    uint16_t* meta = static_cast<uint16_t*>(meta32);
    // each lane's own bit string first, as 16-bit units ...
    const size_t lane_cap = max_lane * 2 + 8;
    lane_bytes.assign(32 * lane_cap, 0);
    for (size_t k = 0; k < 32; ++k) {
      meta[k] = static_cast<uint16_t>(init[k]);
      uint64_t acc = 0; int fill = 0; size_t w = k * lane_cap;
      for (size_t t = 0; t < cnt[k]; ++t) {
        acc |= static_cast<uint64_t>(val[k * max_lane + t]) << fill;
        fill += nb[k * max_lane + t];
        while (fill >= 8) { lane_bytes[w++] = static_cast<uint8_t>(acc); acc >>= 8; fill -= 8; }
      }
      if (fill > 0) lane_bytes[w++] = static_cast<uint8_t>(acc);
    }
    // ... then the order in which a decoder will ask for them: before a round, lanes that
    // still decode and hold < 16 bits take one unit each, lowest lane first
    int held[32] = {};
    size_t taken[32] = {};
    for (size_t r = 0; r < max_lane; ++r) {
      for (size_t k = 0; k < 32; ++k) {
        if (r < cnt[k] && held[k] < 16) {
          const uint8_t* src = lane_bytes.data() + k * lane_cap + 2 * taken[k]++;
          bytes.push_back(src[0]);
          bytes.push_back(src[1]);
          held[k] += 16;
        }
      }
      for (size_t k = 0; k < 32; ++k)
        if (r < cnt[k]) held[k] -= nb[k * max_lane + r];
    }
  }
  while ((bytes.size() - base) % 16) bytes.push_back(0);
  return true;
}

}  // namespace

ANS_EXPORT int ans_host_normalize_freqs(const uint64_t* h_counts, int alphabet, int table_log,
                                        uint32_t* h_freqs_out) {
  if (!h_counts || !h_freqs_out || alphabet < 1 || alphabet > ANS_MAX_ALPHABET) return ANS_ERR_INVALID_ARG;
  if (table_log < 1 || table_log > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
  const uint64_t L = 1ull << table_log;
  uint64_t total = 0, present = 0;
  for (int s = 0; s < alphabet; ++s) { total += h_counts[s]; present += h_counts[s] != 0; }
  std::fill(h_freqs_out, h_freqs_out + 256, 0u);
  if (total == 0 || present > L) return ANS_ERR_BAD_FREQS;
  // floor share (at least one state for a symbol that occurs), then settle the difference:
  // short -> +1 to the largest remainders; over -> -1 from the largest shares
  std::vector<std::pair<uint64_t, int>> rem;
  int64_t given = 0;
  for (int s = 0; s < alphabet; ++s) {
    if (!h_counts[s]) continue;
    const unsigned __int128 scaled = static_cast<unsigned __int128>(h_counts[s]) * L;
    const uint64_t q = static_cast<uint64_t>(scaled / total);
    rem.emplace_back(static_cast<uint64_t>(scaled % total), s);
    h_freqs_out[s] = static_cast<uint32_t>(std::max<uint64_t>(q, 1));
    given += h_freqs_out[s];
  }
  int64_t diff = static_cast<int64_t>(L) - given;
  if (diff > 0) {
    std::stable_sort(rem.begin(), rem.end(),
                     [](const auto& a, const auto& b) { return a.first > b.first; });   // ties keep symbol order
    for (int64_t i = 0; i < diff; ++i) h_freqs_out[rem[static_cast<size_t>(i) % rem.size()].second] += 1;
  }
  while (diff < 0) {
    int best = -1;
    for (int s = 0; s < alphabet; ++s)
      if (h_freqs_out[s] > 1 && (best < 0 || h_freqs_out[s] > h_freqs_out[best])) best = s;
    if (best < 0) return ANS_ERR_BAD_FREQS;
    h_freqs_out[best] -= 1;
    ++diff;
  }
  return ANS_OK;
}

ANS_EXPORT int ans_host_pack_bound(uint64_t n_symbols, uint32_t chunk_symbols, uint32_t lanes, int layout,
                                   uint64_t* h_bytes_out) {
  if (!h_bytes_out || chunk_symbols == 0 || lanes == 0 || lanes % 32) return ANS_ERR_INVALID_ARG;
  if (layout < ANS_LAYOUT_INTERLEAVED || layout > ANS_LAYOUT_CHANNELS) return ANS_ERR_UNSUPPORTED;
  const uint64_t chunks = n_symbols ? (n_symbols + chunk_symbols - 1) / chunk_symbols : 0;
  const uint64_t subs = chunks * (lanes / 32);
  // <= 14 bits per symbol, plus per lane a last unit/word (strips: a length and a state), plus
  // per sub-stream 16 bytes of pad
  *h_bytes_out = n_symbols * 2 + subs * (32 * 4 + 16) + 16;
  return ANS_OK;
}

static int pack_any(const uint8_t* h_symbols, uint64_t n_symbols, const uint32_t* h_freqs,
                    int alphabet, int table_log, uint32_t chunk_symbols, uint32_t lanes,
                    int layout, uint32_t piece, uint8_t* h_stream_out, uint64_t stream_cap,
                    uint64_t* h_stream_bytes_out, uint64_t* h_sub_offsets_out,
                    void* h_lane_meta_out, int n_threads);

ANS_EXPORT int ans_host_pack_layer(const uint8_t* h_symbols, uint64_t n_symbols, const uint32_t* h_freqs,
                                   int alphabet, int table_log, uint32_t chunk_symbols, uint32_t lanes,
                                   int layout, uint8_t* h_stream_out, uint64_t stream_cap,
                                   uint64_t* h_stream_bytes_out, uint64_t* h_sub_offsets_out,
                                   void* h_lane_meta_out, int n_threads) {
  if (layout == ANS_LAYOUT_CHANNELS) return ANS_ERR_UNSUPPORTED;     // needs the piece size: ans_host_pack_channels
  return pack_any(h_symbols, n_symbols, h_freqs, alphabet, table_log, chunk_symbols, lanes, layout, 1, h_stream_out,
                  stream_cap, h_stream_bytes_out, h_sub_offsets_out, h_lane_meta_out, n_threads);
}

ANS_EXPORT int ans_host_pack_channels(const uint8_t* h_symbols, uint64_t n_symbols, const uint32_t* h_freqs,
                                      int alphabet, int table_log, uint32_t chunk_symbols, uint32_t lanes,
                                      uint32_t piece_symbols, uint8_t* h_stream_out, uint64_t stream_cap,
                                      uint64_t* h_stream_bytes_out, uint64_t* h_sub_offsets_out, int n_threads) {
  return pack_any(h_symbols, n_symbols, h_freqs, alphabet, table_log, chunk_symbols, lanes, ANS_LAYOUT_CHANNELS,
                  piece_symbols, h_stream_out, stream_cap, h_stream_bytes_out, h_sub_offsets_out, nullptr, n_threads);
}

static int pack_any(const uint8_t* h_symbols, uint64_t n_symbols, const uint32_t* h_freqs,
                    int alphabet, int table_log, uint32_t chunk_symbols, uint32_t lanes,
                    int layout, uint32_t piece, uint8_t* h_stream_out, uint64_t stream_cap,
                    uint64_t* h_stream_bytes_out, uint64_t* h_sub_offsets_out,
                    void* h_lane_meta_out, int n_threads) {
  if (!h_freqs || !h_stream_bytes_out || !h_sub_offsets_out) return ANS_ERR_INVALID_ARG;
  if (alphabet < 1 || alphabet > ANS_MAX_ALPHABET || chunk_symbols == 0) return ANS_ERR_INVALID_ARG;
  if (table_log < 1 || table_log > ANS_MAX_TABLE_LOG) return ANS_ERR_UNSUPPORTED;
  if (lanes < 32 || lanes > ANS_MAX_LANES || lanes % 32) return ANS_ERR_UNSUPPORTED;
  if (layout < ANS_LAYOUT_INTERLEAVED || layout > ANS_LAYOUT_CHANNELS) return ANS_ERR_UNSUPPORTED;
  const bool channels = layout == ANS_LAYOUT_CHANNELS;
  if (channels) {
    if (piece < 1 || piece > ANS_MAX_PIECE_SYMBOLS) return ANS_ERR_UNSUPPORTED;
    const uint64_t unit = uint64_t(lanes) * piece;
    if (chunk_symbols % unit || n_symbols % unit || chunk_symbols / lanes > ANS_MAX_CHANNEL_LANE_SYMBOLS)
      return ANS_ERR_UNSUPPORTED;
  }
  const bool strips = layout == ANS_LAYOUT_STRIPS;
  if (strips && (chunk_symbols % lanes || chunk_symbols / lanes > ANS_MAX_STRIP_LANE_SYMBOLS))
    return ANS_ERR_UNSUPPORTED;
  if (n_symbols && (!h_symbols || !h_stream_out || (!h_lane_meta_out && !strips && !channels))) return ANS_ERR_INVALID_ARG;
  EncTable T;
  if (!make_enc_table(h_freqs, alphabet, table_log, T)) return ANS_ERR_BAD_FREQS;

  const size_t C = chunk_symbols, W = lanes, G = lanes / 32;
  const size_t chunks = n_symbols ? (n_symbols + C - 1) / C : 0;
  const size_t meta_es = layout == ANS_LAYOUT_INTERLEAVED ? 2 : 4;
  unsigned nt = n_threads > 0 ? static_cast<unsigned>(n_threads) : std::thread::hardware_concurrency();
  nt = std::max(1u, std::min<unsigned>(nt, static_cast<unsigned>(std::max<size_t>(chunks, 1))));

  // pass 1: every thread packs a contiguous range of chunks into its own buffer
  std::vector<std::vector<uint8_t>> part(nt);
  std::vector<std::vector<uint64_t>> part_offs(nt);   // sub-stream starts inside part[i]
  std::vector<int> part_rc(nt, ANS_OK);
  const size_t per = (chunks + nt - 1) / std::max(1u, nt);
  auto work = [&](unsigned ti) {
    std::vector<uint8_t> nb, lane_bytes;
    std::vector<uint16_t> val;
    const size_t c0 = std::min(chunks, ti * per), c1 = std::min(chunks, c0 + per);
    part[ti].reserve((c1 - c0) * C / 4 + 64);
    for (size_t c = c0; c < c1; ++c) {
      const size_t nc = std::min<uint64_t>(C, n_symbols - c * C);
      for (size_t g = 0; g < G; ++g) {
        part_offs[ti].push_back(part[ti].size());
        if (channels) {
          if (!pack_channels_sub(T, h_symbols + c * C, nc / W, W, piece, g, part[ti], nb, val, lane_bytes)) {
            part_rc[ti] = ANS_ERR_BAD_FREQS;
            return;
          }
          continue;
        }
        if (strips) {
          const size_t first = g * 32 * (C / W);
          const size_t ns = nc > first ? std::min(nc - first, 32 * (C / W)) : 0;
          if (!pack_strip(T, h_symbols + c * C + first, ns, part[ti], nb, val)) {
            part_rc[ti] = ANS_ERR_BAD_FREQS;
            return;
          }
          continue;
        }
        void* meta = static_cast<uint8_t*>(h_lane_meta_out) + (c * G + g) * 32 * meta_es;
        if (!pack_sub(T, h_symbols + c * C, nc, W, g, layout, part[ti], meta, nb, val, lane_bytes)) {
          part_rc[ti] = ANS_ERR_BAD_FREQS;
          return;
        }
      }
    }
  };
  if (nt == 1) work(0);
  else {
    std::vector<std::thread> th;
    for (unsigned ti = 0; ti < nt; ++ti) th.emplace_back(work, ti);
    for (auto& t : th) t.join();
  }
  for (int rc : part_rc) if (rc != ANS_OK) return rc;

  // pass 2: lay the parts end to end
  uint64_t total = 0;
  for (unsigned ti = 0; ti < nt; ++ti) total += part[ti].size();
  if (total > stream_cap) return ANS_ERR_BUFFER_TOO_SMALL;
  uint64_t off = 0, sub = 0;
  for (unsigned ti = 0; ti < nt; ++ti) {
    for (uint64_t o : part_offs[ti]) h_sub_offsets_out[sub++] = off + o;
    if (!part[ti].empty()) memcpy(h_stream_out + off, part[ti].data(), part[ti].size());
    off += part[ti].size();
  }
  h_sub_offsets_out[sub] = off;
  *h_stream_bytes_out = off;
  return ANS_OK;
}
