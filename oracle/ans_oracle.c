/*
 * CPU oracle for tabled-ANS (tANS) weight coding and zero-point dequantisation.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference the CUDA
 * library is checked against.  It shares no code with the CUDA library and the
 * library never calls it.  Everything is written for legibility: one symbol at
 * a time, no blocking, no fusion, no tables beyond the ones the paper names.
 *
 * What the paper fixes (Section II-A, Fig. 2, Section III-B):
 *   - the coder is tabled ANS, a finite automaton with l = 2^R states;
 *   - the decoder is a look-up table giving, per state, the decoded symbol, a
 *     number of bits nb_bits to take from the stream and a transition integer
 *     newX; the next state is newX plus the bits taken;
 *   - several streams are decoded at once with ONE table and a VECTOR of states
 *     (one state per stream), each stream of n weights costing n look-ups and
 *     n small additions;
 *   - transitions that take zero bits exist; they are what carries the rate
 *     under 1 bit per symbol;
 *   - the quantiser is uniform with a zero-point (Section II-B), so the inverse
 *     is w = step * (q - zero_point).
 * What the paper leaves open and this oracle fixes (each reading is listed in
 * the design notes of the repository):
 *   - symbol spread over the states: bit-reversal order;
 *   - numbering of a symbol's states: ascending;
 *   - bit order: fields packed least-significant-bit first;
 *   - every lane starts ENCODING at state index 0, so a decoder must END at 0;
 *   - the containers that carry many lanes:
 *       "interleaved": 32 lanes share one sequence of 16-bit units, ordered by
 *                      the decoder's refill schedule;
 *       "private":     each lane owns a contiguous run of 32-bit words;
 *       "quads":       private lanes that take four consecutive symbols per
 *                      turn and fill their words most significant bit first.
 *       "strips":      a sub-stream owns a contiguous strip of the chunk, dealt
 *                      round-robin to its lanes; a lane's bits begin with its
 *                      initial state; a sub-stream carries its lanes' bit
 *                      lengths and their strings back to back.
 *       "channels":    the paper's grouping: pieces of H*W symbols dealt to the
 *                      lanes, so that a lane is an input channel of a layer
 *                      stored O x I x H x W; bytes laid out as in "strips".
 *   - frequency normalisation (largest-remainder, every present symbol >= 1).
 *
 * Pins (see tests): hand-enumerated state traces, table tiling invariants,
 * the closed-form bit count for power-of-two frequencies, exhaustive round
 * trips on tiny alphabets, the cross-entropy bound, and library conversions
 * for the dequantiser.  Exact megabyte figures of the paper's Tables II/III
 * need the trained networks: parity unpinned for those.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ANSO_MAX_R 14
#define ANSO_MAX_A 256

enum {
  ANSO_OK = 0,
  ANSO_ERR_ARG = -1,      /* bad argument */
  ANSO_ERR_FREQ = -2,     /* frequencies do not sum to 2^R, or symbol has f = 0 */
  ANSO_ERR_SPACE = -3,    /* output buffer too small */
  ANSO_ERR_CORRUPT = -4   /* decoder did not end in state 0 / length mismatch */
};

typedef struct {
  int R;                       /* table_log, l = 2^R states (Section II-A)     */
  int A;                       /* alphabet size                                */
  uint32_t f[ANSO_MAX_A];      /* normalised frequencies, sum = 2^R            */
  uint32_t cum[ANSO_MAX_A + 1];
  uint8_t  sym[1 << ANSO_MAX_R];   /* decoded symbol of state index i          */
  uint8_t  nb[1 << ANSO_MAX_R];    /* nb_bits of state index i                 */
  uint16_t newx[1 << ANSO_MAX_R];  /* transition integer newX of state index i */
  uint16_t idx_of[1 << ANSO_MAX_R];/* encoder: cum[s] + (x_s - f_s) -> index i */
} anso_table;

size_t anso_table_sizeof(void) { return sizeof(anso_table); }

/* Reverse the low R bits of j. */
static uint32_t bitrev(uint32_t j, int R) {
  uint32_t r = 0;
  for (int b = 0; b < R; ++b)
    if (j & (1u << b)) r |= 1u << (R - 1 - b);
  return r;
}

static int floor_log2(uint32_t x) {
  int k = -1;
  while (x) { x >>= 1; ++k; }
  return k;
}

/*
 * Spread + decode table (Section II-A: "the table outputs the decoded symbol,
 * a number of bits nb_bits and a transition integer newX").
 * State index i in [0, l) stands for the ANS state x = l + i.
 */
int anso_build_table(const uint32_t* freqs, int A, int R, anso_table* T) {
  if (!freqs || !T || A < 1 || A > ANSO_MAX_A || R < 1 || R > ANSO_MAX_R) return ANSO_ERR_ARG;
  const uint32_t L = 1u << R;
  uint64_t total = 0;
  for (int s = 0; s < A; ++s) total += freqs[s];
  if (total != L) return ANSO_ERR_FREQ;

  memset(T, 0, sizeof(*T));
  T->R = R; T->A = A;
  T->cum[0] = 0;
  for (int s = 0; s < A; ++s) { T->f[s] = freqs[s]; T->cum[s + 1] = T->cum[s] + freqs[s]; }

  /* 1. spread: the j-th slot handed out (symbols in ascending order, f_s slots
   *    each) lands at index bitrev_R(j). */
  uint32_t j = 0;
  for (int s = 0; s < A; ++s)
    for (uint32_t c = 0; c < freqs[s]; ++c, ++j)
      T->sym[bitrev(j, R)] = (uint8_t)s;

  /* 2. number each symbol's states in ascending index order:
   *    x_s = f_s, f_s + 1, ..., 2 f_s - 1.  Decoding state i yields symbol s and
   *    the reduced state x_s; nb bits bring it back into [l, 2l). */
  uint32_t next[ANSO_MAX_A];
  for (int s = 0; s < A; ++s) next[s] = freqs[s];
  for (uint32_t i = 0; i < L; ++i) {
    int s = T->sym[i];
    uint32_t xs = next[s]++;
    int nb = R - floor_log2(xs);
    T->nb[i] = (uint8_t)nb;
    T->newx[i] = (uint16_t)((xs << nb) - L);
    T->idx_of[T->cum[s] + (xs - freqs[s])] = (uint16_t)i;
  }
  return ANSO_OK;
}

/* Field accessors so a Python test can read the table without knowing the layout. */
int anso_table_entry(const anso_table* T, int i, int* sym, int* nb, int* newx) {
  if (!T || i < 0 || i >= (1 << T->R)) return ANSO_ERR_ARG;
  *sym = T->sym[i]; *nb = T->nb[i]; *newx = T->newx[i];
  return ANSO_OK;
}

/*
 * Encode one lane (Section II-A: "following a state transition in the automaton
 * and concatenating the binary string that labels the transition").
 * Symbols m[0], m[stride], ..., n of them.  Encoding runs from the LAST symbol
 * to the first, starting at state index 0, so that the decoder, which runs
 * forwards, ends at index 0.
 *   field_nb[t], field_val[t] : label of the transition that decodes symbol t
 *   returns the initial decode state index, or a negative error.
 */
int anso_encode_lane(const anso_table* T, const uint8_t* m, int64_t n, int64_t stride,
                     uint8_t* field_nb, uint16_t* field_val) {
  const uint32_t L = 1u << T->R;
  uint32_t i = 0;
  for (int64_t t = n - 1; t >= 0; --t) {
    int s = m[t * stride];
    if (s >= T->A || T->f[s] == 0) return ANSO_ERR_FREQ;
    uint32_t x = L + i;
    int k = 0;
    while ((x >> k) >= 2 * T->f[s]) ++k;          /* smallest k with x>>k < 2 f_s */
    field_nb[t] = (uint8_t)k;
    field_val[t] = (uint16_t)(x & ((1u << k) - 1));
    i = T->idx_of[T->cum[s] + ((x >> k) - T->f[s])];
  }
  return (int)i;
}

/* Append `nb` low bits of `val` at bit position *pos of a zero-initialised
 * little-endian byte string (least significant bit first). */
static void put_bits(uint8_t* bytes, uint64_t* pos, uint32_t val, int nb) {
  for (int b = 0; b < nb; ++b, ++*pos)
    if (val & (1u << b)) bytes[*pos >> 3] |= (uint8_t)(1u << (*pos & 7));
}

static uint32_t get_bits(const uint8_t* bytes, uint64_t nbytes, uint64_t pos, int nb) {
  uint32_t v = 0;
  for (int b = 0; b < nb; ++b, ++pos)
    if ((pos >> 3) < nbytes && (bytes[pos >> 3] >> (pos & 7)) & 1) v |= 1u << b;
  return v;
}

/*
 * Plain single-lane coder: the lane's bit string is field_0, field_1, ...
 * concatenated LSB first.  `bytes` must be zeroed and hold (n*R+7)/8 bytes.
 */
int anso_encode_plain(const anso_table* T, const uint8_t* m, int64_t n,
                      uint8_t* bytes, uint64_t cap_bytes, uint64_t* nbits_out) {
  uint8_t* fnb = (uint8_t*)malloc((size_t)(n > 0 ? n : 1));
  uint16_t* fval = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)(n > 0 ? n : 1));
  int init = anso_encode_lane(T, m, n, 1, fnb, fval);
  uint64_t pos = 0;
  if (init >= 0) {
    uint64_t total = 0;
    for (int64_t t = 0; t < n; ++t) total += fnb[t];
    if ((total + 7) / 8 > cap_bytes) init = ANSO_ERR_SPACE;
    else for (int64_t t = 0; t < n; ++t) put_bits(bytes, &pos, fval[t], fnb[t]);
  }
  if (nbits_out) *nbits_out = pos;
  free(fnb); free(fval);
  return init;
}

/*
 * Plain single-lane decoder (Section II-A / Fig. 2): state -> (symbol, nb_bits,
 * newX); take nb_bits from the stream; next state = newX + bits.
 * trace (optional) receives the n visited state indices.
 */
int anso_decode_plain(const anso_table* T, const uint8_t* bytes, uint64_t nbytes, int init,
                      int64_t n, uint8_t* out, int32_t* trace, uint64_t* nbits_used) {
  uint32_t i = (uint32_t)init;
  uint64_t pos = 0;
  for (int64_t t = 0; t < n; ++t) {
    if (trace) trace[t] = (int32_t)i;
    out[t] = T->sym[i];
    int nb = T->nb[i];
    uint32_t v = get_bits(bytes, nbytes, pos, nb);
    pos += (uint64_t)nb;
    i = T->newx[i] + v;
  }
  if (nbits_used) *nbits_used = pos;
  return i == 0 ? ANSO_OK : ANSO_ERR_CORRUPT;
}

/* ------------------------------------------------------------------------- *
 * Containers.  A layer of n symbols is cut into chunks of C consecutive
 * symbols.  Inside a chunk, W = 32*G lanes take the symbols round-robin:
 * chunk-relative symbol q is the (q div W)-th symbol of lane q mod W.  Lane
 * lambda is lane k = lambda mod 32 of sub-stream g = lambda div 32.  Every lane
 * has its own state: the states of all streams kept side by side, as in Section III-B.
 * Sub-streams are numbered chunk-major: sub = chunk*G + g.
 * ------------------------------------------------------------------------- */

static int64_t lane_count(int64_t n_chunk, int W, int lambda) {
  /* number of symbols lane lambda owns in a chunk of n_chunk symbols */
  return n_chunk > lambda ? (n_chunk - lambda + W - 1) / W : 0;
}

/*
 * Interleaved container: the 32 lanes of a sub-stream share one sequence of
 * little-endian 16-bit units.  The order of the units is the order in which
 * the decoder asks for them: before round r, every active lane (one that still
 * has a symbol in round r) whose bit buffer holds fewer than 16 bits takes the
 * next unit, lanes in ascending order; then every active lane decodes one
 * symbol.  Each sub-stream is zero-padded to a multiple of 16 bytes.
 *
 *   stream        : out, capacity cap_bytes
 *   sub_offsets   : out, [n_sub + 1] byte offsets into stream
 *   init_states   : out, [n_sub][32]
 * returns total bytes, or negative error.
 */
int64_t anso_pack_interleaved(const anso_table* T, const uint8_t* symbols, int64_t n,
                              int64_t C, int G, uint8_t* stream, uint64_t cap_bytes,
                              uint64_t* sub_offsets, uint16_t* init_states) {
  if (!T || C < 1 || G < 1 || n < 0) return ANSO_ERR_ARG;
  const int W = 32 * G;
  const int64_t n_chunks = (n + C - 1) / C;
  const int64_t max_lane = (C + W - 1) / W;
  uint8_t* fnb = (uint8_t*)malloc((size_t)(32 * max_lane + 1));
  uint16_t* fval = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)(32 * max_lane + 1));
  uint8_t* lane_bits = (uint8_t*)malloc((size_t)(32 * (max_lane * 2 + 4)));
  const int64_t lane_bytes_cap = max_lane * 2 + 4;   /* R <= 14 < 16 bits per symbol */
  uint64_t off = 0;
  int64_t rc = ANSO_OK;

  for (int64_t c = 0; c < n_chunks && rc >= 0; ++c) {
    const uint8_t* cs = symbols + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G && rc >= 0; ++g) {
      const int64_t sub = c * G + g;
      sub_offsets[sub] = off;
      int64_t cnt_k[32];
      /* encode each lane and lay out its own bit string */
      memset(lane_bits, 0, (size_t)(32 * lane_bytes_cap));
      for (int k = 0; k < 32; ++k) {
        const int lambda = 32 * g + k;
        cnt_k[k] = lane_count(nc, W, lambda);
        int init = anso_encode_lane(T, cs + lambda, cnt_k[k], W, fnb + k * max_lane, fval + k * max_lane);
        if (init < 0) { rc = init; break; }
        init_states[sub * 32 + k] = (uint16_t)init;
        uint64_t pos = 0;
        for (int64_t t = 0; t < cnt_k[k]; ++t)
          put_bits(lane_bits + k * lane_bytes_cap, &pos, fval[k * max_lane + t], fnb[k * max_lane + t]);
      }
      if (rc < 0) break;
      /* replay the decoder's refill schedule to order the units */
      int bits_in_buf[32]; int64_t unit_of[32];
      for (int k = 0; k < 32; ++k) { bits_in_buf[k] = 0; unit_of[k] = 0; }
      const int64_t rounds = cnt_k[0];                /* lane 0 owns the most symbols */
      for (int64_t r = 0; r < rounds; ++r) {
        for (int k = 0; k < 32; ++k) {
          if (r >= cnt_k[k] || bits_in_buf[k] >= 16) continue;
          if (off + 2 > cap_bytes) { rc = ANSO_ERR_SPACE; break; }
          const uint8_t* lb = lane_bits + k * lane_bytes_cap + 2 * unit_of[k];
          stream[off] = lb[0]; stream[off + 1] = lb[1];
          off += 2; unit_of[k] += 1; bits_in_buf[k] += 16;
        }
        if (rc < 0) break;
        for (int k = 0; k < 32; ++k)
          if (r < cnt_k[k]) bits_in_buf[k] -= fnb[k * max_lane + r];
      }
      while (off % 16) { if (off >= cap_bytes) { rc = ANSO_ERR_SPACE; break; } stream[off++] = 0; }
    }
  }
  if (rc >= 0) sub_offsets[n_chunks * G] = off;
  free(fnb); free(fval); free(lane_bits);
  return rc < 0 ? rc : (int64_t)off;
}

/*
 * Decode the interleaved container for chunks [chunk_begin, chunk_end).
 * Every lane keeps (state, 32-bit buffer, bit count): the decode step is the
 * paper's, the refill rule is the container's.
 * Returns ANSO_OK, or ANSO_ERR_CORRUPT if a lane does not end in state 0 or a
 * sub-stream's unit count disagrees with its byte extent.
 */
int anso_unpack_interleaved(const anso_table* T, const uint8_t* stream, const uint64_t* sub_offsets,
                            const uint16_t* init_states, int64_t n, int64_t C, int G,
                            int64_t chunk_begin, int64_t chunk_end, uint8_t* out) {
  const int W = 32 * G;
  int rc = ANSO_OK;
  for (int64_t c = chunk_begin; c < chunk_end; ++c) {
    uint8_t* co = out + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G; ++g) {
      const int64_t sub = c * G + g;
      const uint8_t* p = stream + sub_offsets[sub];
      const uint64_t extent = sub_offsets[sub + 1] - sub_offsets[sub];
      uint64_t used = 0;
      uint32_t state[32], buf[32]; int cnt[32]; int64_t cnt_k[32];
      for (int k = 0; k < 32; ++k) {
        state[k] = init_states[sub * 32 + k]; buf[k] = 0; cnt[k] = 0;
        cnt_k[k] = lane_count(nc, W, 32 * g + k);
      }
      for (int64_t r = 0; r < cnt_k[0]; ++r) {
        for (int k = 0; k < 32; ++k) {
          if (r >= cnt_k[k] || cnt[k] >= 16) continue;
          uint32_t unit = 0;
          if (used + 2 <= extent) unit = (uint32_t)p[used] | ((uint32_t)p[used + 1] << 8);
          else rc = ANSO_ERR_CORRUPT;
          used += 2;
          buf[k] |= unit << cnt[k]; cnt[k] += 16;
        }
        for (int k = 0; k < 32; ++k) {
          if (r >= cnt_k[k]) continue;
          const uint32_t i = state[k];
          co[r * W + 32 * g + k] = T->sym[i];
          const int nb = T->nb[i];
          const uint32_t v = buf[k] & ((1u << nb) - 1);
          buf[k] >>= nb; cnt[k] -= nb;
          state[k] = T->newx[i] + v;
        }
      }
      for (int k = 0; k < 32; ++k) if (state[k] != 0) rc = ANSO_ERR_CORRUPT;
      if (((used + 15) / 16) * 16 != extent) rc = ANSO_ERR_CORRUPT;
    }
  }
  return rc;
}

/*
 * Private container: each lane's own bit string, zero-padded to whole 32-bit
 * little-endian words, the 32 lanes of a sub-stream laid one after the other
 * in ascending lane order; the sub-stream is zero-padded to a multiple of 16
 * bytes.
 *   lane_meta[sub][k] = init_state | (first word of lane k, counted from the
 *                       sub-stream's start) << 16
 */
int64_t anso_pack_private(const anso_table* T, const uint8_t* symbols, int64_t n,
                          int64_t C, int G, uint8_t* stream, uint64_t cap_bytes,
                          uint64_t* sub_offsets, uint32_t* lane_meta) {
  if (!T || C < 1 || G < 1 || n < 0) return ANSO_ERR_ARG;
  const int W = 32 * G;
  const int64_t n_chunks = (n + C - 1) / C;
  const int64_t max_lane = (C + W - 1) / W;
  uint8_t* fnb = (uint8_t*)malloc((size_t)(max_lane + 1));
  uint16_t* fval = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)(max_lane + 1));
  uint64_t off = 0;
  int64_t rc = ANSO_OK;
  for (int64_t c = 0; c < n_chunks && rc >= 0; ++c) {
    const uint8_t* cs = symbols + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G && rc >= 0; ++g) {
      const int64_t sub = c * G + g;
      sub_offsets[sub] = off;
      const uint64_t base = off;
      for (int k = 0; k < 32; ++k) {
        const int lambda = 32 * g + k;
        const int64_t cnt = lane_count(nc, W, lambda);
        int init = anso_encode_lane(T, cs + lambda, cnt, W, fnb, fval);
        if (init < 0) { rc = init; break; }
        uint64_t nbits = 0;
        for (int64_t t = 0; t < cnt; ++t) nbits += fnb[t];
        const uint64_t nbytes = ((nbits + 31) / 32) * 4;
        const uint64_t word0 = (off - base) / 4;
        if (word0 > 0xFFFF) { rc = ANSO_ERR_ARG; break; }
        if (off + nbytes > cap_bytes) { rc = ANSO_ERR_SPACE; break; }
        lane_meta[sub * 32 + k] = (uint32_t)init | ((uint32_t)word0 << 16);
        memset(stream + off, 0, (size_t)nbytes);
        uint64_t pos = 0;
        for (int64_t t = 0; t < cnt; ++t) put_bits(stream + off, &pos, fval[t], fnb[t]);
        off += nbytes;
      }
      while (rc >= 0 && off % 16) { if (off >= cap_bytes) { rc = ANSO_ERR_SPACE; break; } stream[off++] = 0; }
    }
  }
  if (rc >= 0) sub_offsets[n_chunks * G] = off;
  free(fnb); free(fval);
  return rc < 0 ? rc : (int64_t)off;
}

int anso_unpack_private(const anso_table* T, const uint8_t* stream, const uint64_t* sub_offsets,
                        const uint32_t* lane_meta, int64_t n, int64_t C, int G,
                        int64_t chunk_begin, int64_t chunk_end, uint8_t* out) {
  const int W = 32 * G;
  int rc = ANSO_OK;
  for (int64_t c = chunk_begin; c < chunk_end; ++c) {
    uint8_t* co = out + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G; ++g) {
      const int64_t sub = c * G + g;
      const uint8_t* p = stream + sub_offsets[sub];
      const uint64_t extent = sub_offsets[sub + 1] - sub_offsets[sub];
      for (int k = 0; k < 32; ++k) {
        const int lambda = 32 * g + k;
        const int64_t cnt = lane_count(nc, W, lambda);
        const uint32_t meta = lane_meta[sub * 32 + k];
        const uint64_t begin = (uint64_t)(meta >> 16) * 4;
        const uint64_t end = (k < 31) ? (uint64_t)(lane_meta[sub * 32 + k + 1] >> 16) * 4 : extent;
        if (begin > end || end > extent) { rc = ANSO_ERR_CORRUPT; continue; }
        uint32_t i = meta & 0xFFFF;
        uint64_t pos = 0;
        for (int64_t t = 0; t < cnt; ++t) {
          co[t * W + lambda] = T->sym[i];
          const int nb = T->nb[i];
          const uint32_t v = get_bits(p + begin, end - begin, pos, nb);
          pos += (uint64_t)nb;
          i = T->newx[i] + v;
        }
        if (i != 0) rc = ANSO_ERR_CORRUPT;
        /* the lane's words must be exactly what its bits need (last lane: up to the pad) */
        const uint64_t need = ((pos + 31) / 32) * 4;
        if (k < 31 ? (need != end - begin) : (need > end - begin || end - begin - need >= 16)) rc = ANSO_ERR_CORRUPT;
      }
    }
  }
  return rc;
}

/*
 * Quads container: private lanes as above, with two differences that the paper
 * leaves open just the same (Section II-A fixes neither the order of bits in a
 * stream word nor which symbols a stream owns):
 *   - lanes take the chunk's symbols FOUR AT A TIME: chunk-relative symbol q
 *     sits in quad j = q div 4; quad j belongs to lane j mod W, as that lane's
 *     (j div W)-th quad; inside the lane the quad's symbols keep their order.
 *     (A chunk's last quad may hold fewer than four symbols.)
 *   - a lane's bit string fills its 32-bit words from the MOST significant bit
 *     down, and a field's most significant bit comes first.  Words are stored
 *     little-endian, zero-padded as in the private container.
 * lane_meta and the sub-stream order are those of the private container.
 */
static int64_t quad_lane_count(int64_t n_chunk, int W, int lambda) {
  /* symbols lane lambda owns: 4 per full quad, plus the short last quad if it is the lane's */
  const int64_t full = n_chunk / 4, rem = n_chunk % 4;
  int64_t cnt = 4 * (full > lambda ? (full - lambda + W - 1) / W : 0);
  if (rem && full % W == lambda) cnt += rem;
  return cnt;
}

/* chunk-relative position of lane lambda's t-th symbol */
static int64_t quad_position(int W, int lambda, int64_t t) {
  return ((t / 4) * W + lambda) * 4 + t % 4;
}

/* Append `nb` bits of `val`, most significant first; bit position p of the string is bit
 * 31 - p%32 of 32-bit little-endian word p/32. */
static void put_bits_msb(uint8_t* bytes, uint64_t* pos, uint32_t val, int nb) {
  for (int b = nb - 1; b >= 0; --b, ++*pos) {
    const int bit_in_word = 31 - (int)(*pos % 32);
    if (val & (1u << b)) bytes[(*pos / 32) * 4 + bit_in_word / 8] |= (uint8_t)(1u << (bit_in_word % 8));
  }
}

static uint32_t get_bits_msb(const uint8_t* bytes, uint64_t nbytes, uint64_t pos, int nb) {
  uint32_t v = 0;
  for (int b = 0; b < nb; ++b, ++pos) {
    const int bit_in_word = 31 - (int)(pos % 32);
    const uint64_t byte = (pos / 32) * 4 + (uint64_t)(bit_in_word / 8);
    v <<= 1;
    if (byte < nbytes && (bytes[byte] >> (bit_in_word % 8)) & 1) v |= 1u;
  }
  return v;
}

int64_t anso_pack_quads(const anso_table* T, const uint8_t* symbols, int64_t n,
                        int64_t C, int G, uint8_t* stream, uint64_t cap_bytes,
                        uint64_t* sub_offsets, uint32_t* lane_meta) {
  if (!T || C < 1 || G < 1 || n < 0) return ANSO_ERR_ARG;
  const int W = 32 * G;
  const int64_t n_chunks = (n + C - 1) / C;
  const int64_t max_lane = 4 * ((C / 4 + W - 1) / W) + 4;
  uint8_t* mine = (uint8_t*)malloc((size_t)max_lane);
  uint8_t* fnb = (uint8_t*)malloc((size_t)max_lane);
  uint16_t* fval = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)max_lane);
  uint64_t off = 0;
  int64_t rc = ANSO_OK;
  for (int64_t c = 0; c < n_chunks && rc >= 0; ++c) {
    const uint8_t* cs = symbols + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G && rc >= 0; ++g) {
      const int64_t sub = c * G + g;
      sub_offsets[sub] = off;
      const uint64_t base = off;
      for (int k = 0; k < 32; ++k) {
        const int lambda = 32 * g + k;
        const int64_t cnt = quad_lane_count(nc, W, lambda);
        for (int64_t t = 0; t < cnt; ++t) mine[t] = cs[quad_position(W, lambda, t)];
        int init = anso_encode_lane(T, mine, cnt, 1, fnb, fval);
        if (init < 0) { rc = init; break; }
        uint64_t nbits = 0;
        for (int64_t t = 0; t < cnt; ++t) nbits += fnb[t];
        const uint64_t nbytes = ((nbits + 31) / 32) * 4;
        const uint64_t word0 = (off - base) / 4;
        if (word0 > 0xFFFF) { rc = ANSO_ERR_ARG; break; }
        if (off + nbytes > cap_bytes) { rc = ANSO_ERR_SPACE; break; }
        lane_meta[sub * 32 + k] = (uint32_t)init | ((uint32_t)word0 << 16);
        memset(stream + off, 0, (size_t)nbytes);
        uint64_t pos = 0;
        for (int64_t t = 0; t < cnt; ++t) put_bits_msb(stream + off, &pos, fval[t], fnb[t]);
        off += nbytes;
      }
      while (rc >= 0 && off % 16) { if (off >= cap_bytes) { rc = ANSO_ERR_SPACE; break; } stream[off++] = 0; }
    }
  }
  if (rc >= 0) sub_offsets[n_chunks * G] = off;
  free(mine); free(fnb); free(fval);
  return rc < 0 ? rc : (int64_t)off;
}

int anso_unpack_quads(const anso_table* T, const uint8_t* stream, const uint64_t* sub_offsets,
                      const uint32_t* lane_meta, int64_t n, int64_t C, int G,
                      int64_t chunk_begin, int64_t chunk_end, uint8_t* out) {
  const int W = 32 * G;
  int rc = ANSO_OK;
  for (int64_t c = chunk_begin; c < chunk_end; ++c) {
    uint8_t* co = out + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G; ++g) {
      const int64_t sub = c * G + g;
      const uint8_t* p = stream + sub_offsets[sub];
      const uint64_t extent = sub_offsets[sub + 1] - sub_offsets[sub];
      for (int k = 0; k < 32; ++k) {
        const int lambda = 32 * g + k;
        const int64_t cnt = quad_lane_count(nc, W, lambda);
        const uint32_t meta = lane_meta[sub * 32 + k];
        const uint64_t begin = (uint64_t)(meta >> 16) * 4;
        const uint64_t end = (k < 31) ? (uint64_t)(lane_meta[sub * 32 + k + 1] >> 16) * 4 : extent;
        if (begin > end || end > extent) { rc = ANSO_ERR_CORRUPT; continue; }
        uint32_t i = meta & 0xFFFF;
        uint64_t pos = 0;
        for (int64_t t = 0; t < cnt; ++t) {
          co[quad_position(W, lambda, t)] = T->sym[i];
          const int nb = T->nb[i];
          const uint32_t v = get_bits_msb(p + begin, end - begin, pos, nb);
          pos += (uint64_t)nb;
          i = T->newx[i] + v;
        }
        if (i != 0) rc = ANSO_ERR_CORRUPT;
        const uint64_t need = ((pos + 31) / 32) * 4;
        if (k < 31 ? (need != end - begin) : (need > end - begin || end - begin - need >= 16)) rc = ANSO_ERR_CORRUPT;
      }
    }
  }
  return rc;
}

/*
 * Strips container.  The paper leaves open which symbols a stream owns and how
 * a stream is laid out (Section III-B only fixes one state per stream and a
 * shared table); this container keeps a sub-stream's symbols in one contiguous
 * strip of the chunk and the per-lane overhead down to the state and one
 * 16-bit length:
 *   - C must be a multiple of W = 32*G; S = C / W <= 4096 is the number of
 *     symbols a lane owns in a full chunk.
 *   - Sub-stream g of a chunk owns the chunk-relative symbols
 *     [g*32*S, min((g+1)*32*S, n_chunk)): its strip, which may be short or
 *     empty in the layer's last chunk.
 *   - Inside the strip the 32 lanes take the symbols round-robin: strip-relative
 *     symbol q is the (q div 32)-th symbol of lane q mod 32.
 *   - A lane that owns at least one symbol has the bit string
 *         initial decode state index (R bits), field_0, field_1, ...
 *     every item most significant bit first; a lane without symbols has the
 *     empty string.
 *   - The sub-stream's bytes: 32 little-endian uint16 = the bit lengths of
 *     its lanes' strings; then the 32 strings back to back, without gaps, in
 *     lane order, filling 32-bit little-endian words from the most significant
 *     bit down (the bit order of the quads container); zero-padded to a
 *     multiple of 16 bytes.  There is no lane_meta array.
 * Sub-streams are numbered chunk-major as in the other containers.
 */
#define ANSO_STRIP_HEADER 64   /* bytes: 32 lanes x uint16 bit length */
#define ANSO_STRIP_MAX_S 4096

static int64_t strip_symbols(int64_t n_chunk, int64_t S, int g) {
  int64_t ns = n_chunk - (int64_t)g * 32 * S;
  if (ns > 32 * S) ns = 32 * S;
  return ns < 0 ? 0 : ns;
}

int64_t anso_pack_strips(const anso_table* T, const uint8_t* symbols, int64_t n,
                         int64_t C, int G, uint8_t* stream, uint64_t cap_bytes,
                         uint64_t* sub_offsets) {
  if (!T || C < 1 || G < 1 || n < 0) return ANSO_ERR_ARG;
  const int W = 32 * G;
  if (C % W) return ANSO_ERR_ARG;
  const int64_t S = C / W;
  if (S > ANSO_STRIP_MAX_S) return ANSO_ERR_ARG;
  const int64_t n_chunks = (n + C - 1) / C;
  uint8_t* fnb = (uint8_t*)malloc((size_t)S);
  uint16_t* fval = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)S);
  uint64_t off = 0;
  int64_t rc = ANSO_OK;
  for (int64_t c = 0; c < n_chunks && rc >= 0; ++c) {
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G && rc >= 0; ++g) {
      const int64_t sub = c * G + g;
      const uint8_t* strip = symbols + c * C + (int64_t)g * 32 * S;
      const int64_t ns = strip_symbols(nc, S, g);
      sub_offsets[sub] = off;
      /* worst case: header + 32 lanes of R + S*R bits, + padding */
      const uint64_t worst = ANSO_STRIP_HEADER + (uint64_t)(32 * (S + 1) * T->R + 7) / 8 + 20;
      if (off + worst > cap_bytes) { rc = ANSO_ERR_SPACE; break; }
      memset(stream + off, 0, (size_t)worst);
      uint8_t* body = stream + off + ANSO_STRIP_HEADER;
      uint64_t pos = 0;                                /* bit position in the body */
      for (int k = 0; k < 32; ++k) {
        const int64_t cnt = lane_count(ns, 32, k);
        const uint64_t pos0 = pos;
        if (cnt > 0) {
          int init = anso_encode_lane(T, strip + k, cnt, 32, fnb, fval);
          if (init < 0) { rc = init; break; }
          put_bits_msb(body, &pos, (uint32_t)init, T->R);
          for (int64_t t = 0; t < cnt; ++t) put_bits_msb(body, &pos, fval[t], fnb[t]);
        }
        const uint64_t len = pos - pos0;
        stream[off + 2 * k] = (uint8_t)(len & 0xFF);
        stream[off + 2 * k + 1] = (uint8_t)(len >> 8);
      }
      if (rc < 0) break;
      off += ANSO_STRIP_HEADER + ((pos + 31) / 32) * 4;
      while (off % 16) ++off;                          /* already zero */
    }
  }
  if (rc >= 0) sub_offsets[n_chunks * G] = off;
  free(fnb); free(fval);
  return rc < 0 ? rc : (int64_t)off;
}

int anso_unpack_strips(const anso_table* T, const uint8_t* stream, const uint64_t* sub_offsets,
                       int64_t n, int64_t C, int G,
                       int64_t chunk_begin, int64_t chunk_end, uint8_t* out) {
  const int W = 32 * G;
  if (C % W) return ANSO_ERR_ARG;
  const int64_t S = C / W;
  int rc = ANSO_OK;
  for (int64_t c = chunk_begin; c < chunk_end; ++c) {
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    for (int g = 0; g < G; ++g) {
      const int64_t sub = c * G + g;
      uint8_t* so = out + c * C + (int64_t)g * 32 * S;      /* the strip's place in the output */
      const int64_t ns = strip_symbols(nc, S, g);
      const uint8_t* p = stream + sub_offsets[sub];
      const uint64_t extent = sub_offsets[sub + 1] - sub_offsets[sub];
      if (extent < ANSO_STRIP_HEADER) { rc = ANSO_ERR_CORRUPT; continue; }
      const uint8_t* body = p + ANSO_STRIP_HEADER;
      const uint64_t body_bytes = extent - ANSO_STRIP_HEADER;
      uint64_t start = 0;                              /* bit position of lane k's string */
      for (int k = 0; k < 32; ++k) {
        const int64_t cnt = lane_count(ns, 32, k);
        const uint64_t len = (uint64_t)p[2 * k] | ((uint64_t)p[2 * k + 1] << 8);
        uint64_t pos = start;
        if (cnt > 0) {
          uint32_t i = get_bits_msb(body, body_bytes, pos, T->R);
          pos += (uint64_t)T->R;
          for (int64_t t = 0; t < cnt; ++t) {
            so[t * 32 + k] = T->sym[i];
            const int nb = T->nb[i];
            const uint32_t v = get_bits_msb(body, body_bytes, pos, nb);
            pos += (uint64_t)nb;
            i = T->newx[i] + v;
          }
          if (i != 0) rc = ANSO_ERR_CORRUPT;
        }
        if (pos - start != len) rc = ANSO_ERR_CORRUPT;   /* the lane used exactly its bits */
        start += len;
      }
      /* the sub-stream holds exactly the header, the words its bits need, and the pad */
      uint64_t want = ANSO_STRIP_HEADER + ((start + 31) / 32) * 4;
      want = (want + 15) / 16 * 16;
      if (want != extent) rc = ANSO_ERR_CORRUPT;
    }
  }
  return rc;
}

/*
 * Channels container: the paper's own grouping (Section III-B: the weights of a
 * layer are split into streams by INPUT CHANNEL, so that the streams feed the
 * input-channel-parallel multipliers side by side).  For a convolution tensor
 * stored output-channel major, O x I x H x W, the weights of input channel c are
 * O pieces of E = H*W consecutive symbols, one piece every I*E symbols.  Hence:
 *   - a chunk's symbols come in pieces of E consecutive symbols; piece j of the
 *     chunk belongs to lane j mod W (W = 32*G lanes) as that lane's
 *     (j div W)-th piece.  With one chunk per layer and W = I, lane c is input
 *     channel c.  C and n must be multiples of W*E, so every lane of a chunk
 *     owns the same number of whole pieces.
 *   - sub-stream g holds lanes 32g .. 32g+31; its bytes are laid out exactly as
 *     in the strips container (32 lengths, then the strings, each headed by its
 *     initial state, most significant bit first).
 */
static int64_t channels_position(int W, int E, int lambda, int64_t t) {
  return ((t / E) * W + lambda) * E + t % E;    /* chunk-relative place of lane lambda's t-th symbol */
}

int64_t anso_pack_channels(const anso_table* T, const uint8_t* symbols, int64_t n,
                           int64_t C, int G, int E, uint8_t* stream, uint64_t cap_bytes,
                           uint64_t* sub_offsets) {
  if (!T || C < 1 || G < 1 || E < 1 || n < 0) return ANSO_ERR_ARG;
  const int W = 32 * G;
  if (C % ((int64_t)W * E) || n % ((int64_t)W * E)) return ANSO_ERR_ARG;
  const int64_t n_chunks = (n + C - 1) / C;
  const int64_t max_lane = C / W;
  uint8_t* mine = (uint8_t*)malloc((size_t)max_lane);
  uint8_t* fnb = (uint8_t*)malloc((size_t)max_lane);
  uint16_t* fval = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)max_lane);
  uint64_t off = 0;
  int64_t rc = ANSO_OK;
  for (int64_t c = 0; c < n_chunks && rc >= 0; ++c) {
    const uint8_t* cs = symbols + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    const int64_t cnt = nc / W;                        /* symbols of every lane of this chunk */
    for (int g = 0; g < G && rc >= 0; ++g) {
      const int64_t sub = c * G + g;
      sub_offsets[sub] = off;
      const uint64_t worst = ANSO_STRIP_HEADER + (uint64_t)(32 * (cnt + 1) * T->R + 7) / 8 + 20;
      if (off + worst > cap_bytes) { rc = ANSO_ERR_SPACE; break; }
      memset(stream + off, 0, (size_t)worst);
      uint8_t* body = stream + off + ANSO_STRIP_HEADER;
      uint64_t pos = 0;
      for (int k = 0; k < 32; ++k) {
        const uint64_t pos0 = pos;
        if (cnt > 0) {
          for (int64_t t = 0; t < cnt; ++t) mine[t] = cs[channels_position(W, E, 32 * g + k, t)];
          int init = anso_encode_lane(T, mine, cnt, 1, fnb, fval);
          if (init < 0) { rc = init; break; }
          put_bits_msb(body, &pos, (uint32_t)init, T->R);
          for (int64_t t = 0; t < cnt; ++t) put_bits_msb(body, &pos, fval[t], fnb[t]);
        }
        const uint64_t len = pos - pos0;
        if (len > 0xFFFF) { rc = ANSO_ERR_ARG; break; }   /* a lane's length must fit its 16-bit field */
        stream[off + 2 * k] = (uint8_t)(len & 0xFF);
        stream[off + 2 * k + 1] = (uint8_t)(len >> 8);
      }
      if (rc < 0) break;
      off += ANSO_STRIP_HEADER + ((pos + 31) / 32) * 4;
      while (off % 16) ++off;
    }
  }
  if (rc >= 0) sub_offsets[n_chunks * G] = off;
  free(mine); free(fnb); free(fval);
  return rc < 0 ? rc : (int64_t)off;
}

int anso_unpack_channels(const anso_table* T, const uint8_t* stream, const uint64_t* sub_offsets,
                         int64_t n, int64_t C, int G, int E,
                         int64_t chunk_begin, int64_t chunk_end, uint8_t* out) {
  const int W = 32 * G;
  if (E < 1 || C % ((int64_t)W * E) || n % ((int64_t)W * E)) return ANSO_ERR_ARG;
  int rc = ANSO_OK;
  for (int64_t c = chunk_begin; c < chunk_end; ++c) {
    uint8_t* co = out + c * C;
    const int64_t nc = (n - c * C) < C ? (n - c * C) : C;
    const int64_t cnt = nc / W;
    for (int g = 0; g < G; ++g) {
      const int64_t sub = c * G + g;
      const uint8_t* p = stream + sub_offsets[sub];
      const uint64_t extent = sub_offsets[sub + 1] - sub_offsets[sub];
      if (extent < ANSO_STRIP_HEADER) { rc = ANSO_ERR_CORRUPT; continue; }
      const uint8_t* body = p + ANSO_STRIP_HEADER;
      const uint64_t body_bytes = extent - ANSO_STRIP_HEADER;
      uint64_t start = 0;
      for (int k = 0; k < 32; ++k) {
        const uint64_t len = (uint64_t)p[2 * k] | ((uint64_t)p[2 * k + 1] << 8);
        uint64_t pos = start;
        if (cnt > 0) {
          uint32_t i = get_bits_msb(body, body_bytes, pos, T->R);
          pos += (uint64_t)T->R;
          for (int64_t t = 0; t < cnt; ++t) {
            co[channels_position(W, E, 32 * g + k, t)] = T->sym[i];
            const int nb = T->nb[i];
            const uint32_t v = get_bits_msb(body, body_bytes, pos, nb);
            pos += (uint64_t)nb;
            i = T->newx[i] + v;
          }
          if (i != 0) rc = ANSO_ERR_CORRUPT;
        }
        if (pos - start != len) rc = ANSO_ERR_CORRUPT;
        start += len;
      }
      uint64_t want = ANSO_STRIP_HEADER + ((start + 31) / 32) * 4;
      want = (want + 15) / 16 * 16;
      if (want != extent) rc = ANSO_ERR_CORRUPT;
    }
  }
  return rc;
}

/* ------------------------------------------------------------------------- *
 * Dequantisation: uniform quantiser with a zero-point (Section II-B), so
 * w = (q - zero_point) * step, one IEEE single-precision multiply.
 * bf16 is the upper half of that fp32 after round-to-nearest-even.
 * ------------------------------------------------------------------------- */
void anso_dequant_f32(const uint8_t* sym, int64_t n, int zero_point, float scale, float* out) {
  for (int64_t t = 0; t < n; ++t) {
    const float d = (float)((int)sym[t] - zero_point);
    out[t] = d * scale;
  }
}

static uint16_t f32_to_bf16_rne(float x) {
  uint32_t u; memcpy(&u, &x, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x0040u); /* NaN */
  const uint32_t kept_lsb = (u >> 16) & 1u;
  const uint32_t dropped = u & 0xFFFFu;
  uint32_t hi = u >> 16;
  if (dropped > 0x8000u || (dropped == 0x8000u && kept_lsb)) hi += 1;
  return (uint16_t)hi;
}

void anso_dequant_bf16(const uint8_t* sym, int64_t n, int zero_point, float scale, uint16_t* out) {
  for (int64_t t = 0; t < n; ++t) {
    const float d = (float)((int)sym[t] - zero_point);
    out[t] = f32_to_bf16_rne(d * scale);
  }
}

/* ------------------------------------------------------------------------- *
 * Frequency normalisation (the paper codes "each layer using a 256 states
 * tANS coder", Section III-A, without saying how the histogram is cut into l
 * slots).  Every present symbol gets at least one slot; the floor allocation
 * is corrected by largest remainder (ties to the lower symbol) or, when it
 * overshoots, by taking from the largest frequency (ties to the lower symbol).
 * ------------------------------------------------------------------------- */
int anso_normalize_freqs(const uint64_t* counts, int A, int R, uint32_t* freqs) {
  if (!counts || !freqs || A < 1 || A > ANSO_MAX_A || R < 1 || R > ANSO_MAX_R) return ANSO_ERR_ARG;
  const uint64_t L = 1ull << R;
  uint64_t n = 0; int present = 0;
  for (int s = 0; s < A; ++s) { n += counts[s]; present += counts[s] > 0; }
  if (n == 0) { for (int s = 0; s < A; ++s) freqs[s] = 0; return ANSO_ERR_FREQ; }
  if ((uint64_t)present > L) return ANSO_ERR_FREQ;
  uint64_t rem[ANSO_MAX_A]; int64_t sum = 0;
  for (int s = 0; s < A; ++s) {
    if (!counts[s]) { freqs[s] = 0; rem[s] = 0; continue; }
    unsigned __int128 prod = (unsigned __int128)counts[s] * L;
    uint64_t q = (uint64_t)(prod / n);
    rem[s] = (uint64_t)(prod % n);
    freqs[s] = (uint32_t)(q ? q : 1);
    sum += freqs[s];
  }
  int64_t D = (int64_t)L - sum;
  /* D > 0: the floors fell short by fewer than one slot per present symbol, so
   * one pass of +1 by descending remainder is enough. */
  uint8_t served[ANSO_MAX_A];
  memset(served, 0, sizeof(served));
  while (D > 0) {
    int best = -1;
    for (int s = 0; s < A; ++s)
      if (counts[s] && !served[s] && (best < 0 || rem[s] > rem[best])) best = s;
    if (best < 0) return ANSO_ERR_FREQ;
    freqs[best] += 1; served[best] = 1; --D;
  }
  while (D < 0) {                      /* take from the largest frequency */
    int best = -1;
    for (int s = 0; s < A; ++s)
      if (freqs[s] > 1 && (best < 0 || freqs[s] > freqs[best])) best = s;
    if (best < 0) return ANSO_ERR_FREQ;
    freqs[best] -= 1; ++D;
  }
  return ANSO_OK;
}

void anso_histogram(const uint8_t* sym, int64_t n, uint64_t* counts256) {
  memset(counts256, 0, 256 * sizeof(uint64_t));
  for (int64_t t = 0; t < n; ++t) counts256[sym[t]] += 1;
}
