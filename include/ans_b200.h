/*
 * ans_b200 -- inference-time decoding of tabled-ANS (tANS) coded, zero-point quantised
 * neural-network weights on NVIDIA B200 (sm_100a).
 *
 * The operation is the decoder of "Efficient Neural Compression with Inference-time
 * Decoding" (Metz, Bichler, Dupret; ISCAS 2024):
 *   - Section II-A, Fig. 2: a look-up table gives, for the current state, the decoded
 *     symbol, a number of bits nb_bits to take from the compressed stream and a
 *     transition integer newX; the next state is newX + the bits taken.  Transitions
 *     that take no bits are what lets the rate fall under 1 bit per weight.
 *   - Section III-B: many streams are decoded at once with ONE table per layer and a
 *     VECTOR of states, one state per stream.
 *   - Section II-B: weights come from a uniform quantiser with a zero-point, so a
 *     decoded symbol q becomes the weight  w = scale * (q - zero_point).
 *
 * C ABI, plain pointers and sizes.  Pointer names say where the memory lives:
 *   h_*  host memory,  d_*  device memory of the CURRENT CUDA device.
 * The caller owns every buffer.  Unless a function says otherwise the library
 * allocates nothing, keeps no state except the last CUDA error code, enqueues its
 * device work on the caller's stream (`stream` is a cudaStream_t passed as void*;
 * NULL is the default stream) and returns without waiting for it.
 * Every function returns ANS_OK (0) or a negative ANS_ERR_* code; none throws, aborts
 * or prints.
 *
 * Containers (how one layer's symbols are cut into independently decodable pieces;
 * the paper fixes only that every stream has a state of its own):
 *   A layer of n symbols (the tensor flattened in memory order) is cut into chunks of
 *   `chunk_symbols` consecutive symbols.  Inside a chunk, `lanes` = 32*G lanes take the
 *   symbols round-robin (chunk-relative symbol q is the (q / lanes)-th symbol of lane
 *   q % lanes); every lane is its own tANS stream with its own state, all lanes of a
 *   layer share the layer's table.  Lane 32*g + k is lane k of sub-stream g; sub-streams
 *   are numbered chunk-major: sub = chunk*G + g.  Every sub-stream's bytes start at a
 *   16-byte aligned offset of d_stream, given by d_sub_offsets[sub] (n_sub + 1 entries, each
 *   a multiple of 16; a sub-stream whose begin or end is not, or lies outside the stream, is
 *   flagged ANS_STATUS_BAD_LENGTH and not read).
 *   (With one chunk per layer and as many lanes as a conv layer has input channels, over
 *   weights stored channels-last, lane c is the stream of input channel c: the paper's own
 *   grouping, Section III-B.)
 *   Bits are packed least-significant first; a lane's encoder starts from state index 0,
 *   so a sound stream makes its decoder END in state index 0.
 *     ANS_LAYOUT_INTERLEAVED: the 32 lanes of a sub-stream share ONE sequence of
 *       little-endian 16-bit units.  Before each round every lane that still has a
 *       symbol to decode and holds fewer than 16 buffered bits takes the next unit
 *       (lanes in ascending order); then each such lane decodes one symbol.
 *       d_lane_meta is uint16_t[n_sub][32]: initial state index per lane.
 *     ANS_LAYOUT_PRIVATE: every lane owns a contiguous run of little-endian 32-bit
 *       words inside its sub-stream, lanes in ascending order.
 *       d_lane_meta is uint32_t[n_sub][32]: initial state | (first word, counted from
 *       the sub-stream's start) << 16.
 *     ANS_LAYOUT_QUADS: private lanes with two differences.  Lanes take the chunk's symbols
 *       four at a time: chunk-relative symbol q sits in quad j = q / 4, quad j is the
 *       (j / lanes)-th quad of lane j % lanes (the chunk's last quad may be short), so a
 *       lane writes 4 adjacent outputs per turn.  And a lane's bits fill its 32-bit words
 *       from the most significant bit down, each field most significant bit first (the
 *       words themselves are stored little-endian).  d_lane_meta as for ANS_LAYOUT_PRIVATE.
 *     ANS_LAYOUT_STRIPS: made for layers in which one symbol owns most of the states, so that
 *       many transitions take no bits (Section II-A) and a look-up can stand for a run of that
 *       symbol plus one more.  chunk_symbols must be a multiple of lanes, with
 *       S = chunk_symbols / lanes <= 4096.  Sub-stream g of a chunk owns the chunk's symbols
 *       [g * 32 * S, (g + 1) * 32 * S): a contiguous strip (short or empty at the layer's end).
 *       Inside the strip its 32 lanes take the symbols round-robin (strip-relative symbol q is
 *       the (q / 32)-th symbol of lane q % 32).  A lane that owns symbols has the bit string: initial state (table_log
 *       bits), then its fields, every item most significant bit first.  The sub-stream's bytes
 *       are 32 little-endian uint16 (the lanes' bit lengths), then the 32 strings back to back
 *       without gaps, filling 32-bit little-endian words from the most significant bit down,
 *       zero-padded to a multiple of 16 bytes.  There is no per-lane array: d_lane_meta is
 *       ignored and may be NULL.
 *     ANS_LAYOUT_CHANNELS: the paper's own grouping (Section III-B: a layer's weights are split
 *       into streams by input channel).  A chunk's symbols come in pieces of `piece_symbols`
 *       consecutive symbols; piece j of the chunk is the (j / lanes)-th piece of lane j % lanes.
 *       For a convolution tensor stored O x I x H x W, with piece_symbols = H * W, lanes = I
 *       and one chunk per layer (chunk_symbols = n_symbols), lane c carries input channel c and
 *       the decoded tensor comes out in its own O x I x H x W order.  chunk_symbols and
 *       n_symbols must be multiples of lanes * piece_symbols; a lane owns at most 32768
 *       symbols per chunk and its string at most 65535 bits; piece_symbols * element size of
 *       the output at most 128 bytes (an 8 x 8 kernel in bf16).  Sub-stream g holds lanes
 *       32 g .. 32 g + 31; its bytes are laid out as for ANS_LAYOUT_STRIPS; no d_lane_meta.
 */
#ifndef ANS_B200_H
#define ANS_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ANS_OK                    0
#define ANS_ERR_INVALID_ARG      -1   /* null pointer, size out of range, misaligned buffer      */
#define ANS_ERR_BAD_FREQS        -2   /* frequencies do not sum to 2^table_log / unusable symbol */
#define ANS_ERR_UNSUPPORTED      -3   /* table_log outside [1,14], lanes not 32*G, unknown dtype */
#define ANS_ERR_BUFFER_TOO_SMALL -4
#define ANS_ERR_CUDA             -5   /* a CUDA call failed; raw code from ans_last_cuda_error() */
#define ANS_ERR_CORRUPT          -6   /* device status word: a stream did not decode soundly     */

#define ANS_U8   0   /* decoded symbols, one byte each             */
#define ANS_F32  1   /* dequantised weights, IEEE single           */
#define ANS_BF16 2   /* dequantised weights, bfloat16 (RNE of F32) */

#define ANS_LAYOUT_INTERLEAVED 0
#define ANS_LAYOUT_PRIVATE     1
#define ANS_LAYOUT_QUADS       2
#define ANS_LAYOUT_STRIPS      3
#define ANS_LAYOUT_CHANNELS    4

#define ANS_MAX_TABLE_LOG 14
#define ANS_MAX_LANES     2048   /* lanes per chunk: any multiple of 32 up to this */
#define ANS_MAX_ALPHABET  256
#define ANS_MAX_STRIP_LANE_SYMBOLS 4096   /* ANS_LAYOUT_STRIPS: chunk_symbols / lanes at most */
#define ANS_MAX_CHANNEL_LANE_SYMBOLS 32768 /* ANS_LAYOUT_CHANNELS: chunk_symbols / lanes at most */
#define ANS_MAX_PIECE_SYMBOLS 127         /* ANS_LAYOUT_CHANNELS: piece_symbols at most */

/* bits of the device status word (0 = every stream sound) */
#define ANS_STATUS_BAD_FINAL_STATE 1u   /* a lane did not end in state index 0          */
#define ANS_STATUS_BAD_LENGTH      2u   /* a sub-stream consumed more or fewer bytes than it holds */
#define ANS_STATUS_BAD_SYMBOL      4u   /* a decoded symbol does not fit `bitwidth` bits  */
#define ANS_STATUS_COPY_TIMEOUT    8u   /* an asynchronous copy of compressed bytes into shared memory
                                           did not complete within the kernel's bounded wait; the
                                           warp that waited decoded nothing further            */

/*
 * One layer of a decode call.  For the *_batch call an array of these lives in device
 * memory (with a host copy for validation); all pointers inside are device pointers.
 */
typedef struct ans_layer_desc {
  const void*     d_table;        /* this layer's table, written by ans_build_decode_tables  */
  const uint8_t*  d_stream;       /* compressed bytes of all the layer's sub-streams, 16-byte aligned */
  const uint64_t* d_sub_offsets;  /* [n_sub + 1] byte offsets into d_stream, each a multiple of 16 */
  const void*     d_lane_meta;    /* per-lane initial state (and first word): see the layouts above;
                                     unused (may be NULL) for ANS_LAYOUT_STRIPS                */
  void*           d_out;          /* n_symbols elements of out_dtype, 16-byte aligned       */
  uint64_t        stream_bytes;   /* bytes readable at d_stream (offsets beyond it are flagged) */
  uint64_t        n_symbols;      /* weights in the layer; may be 0                          */
  uint32_t        chunk_symbols;  /* symbols per chunk (last chunk may be shorter), >= 1    */
  uint32_t        lanes;          /* 32*G, G in 1..64 (the kernels' fast paths: G in {1,2,4,8}) */
  int32_t         table_log;      /* R: the table has 2^R states (paper: l = 64..256; here 1..14) */
  int32_t         bitwidth;       /* b in [1,8]: symbols must be < 2^b (checked on the device) */
  int32_t         zero_point;     /* symbol that dequantises to 0 (Section II-B)            */
  float           scale;          /* quantisation step                                      */
  int32_t         out_dtype;      /* ANS_U8 | ANS_F32 | ANS_BF16                            */
  int32_t         layout;         /* ANS_LAYOUT_*                                           */
  uint32_t        work_begin;     /* written by ans_plan_batch: first work item of the layer */
  uint32_t        work_count;     /* written by ans_plan_batch: the layer's work items (a work
                                     item is a group of up to 4 consecutive sub-streams)     */
  uint32_t        piece_symbols;  /* ANS_LAYOUT_CHANNELS: symbols of a piece (H * W of the conv
                                     kernel), 1 .. 127; ignored by the other layouts           */
  uint32_t        flags;          /* ANS_DESC_* bits, 0 by default                           */
} ans_layer_desc;

/* ans_layer_desc.flags.
 *
 * The decode kernels are launched so that they may take their place on the device while the
 * work before them on the stream is still running (programmatic dependent launch).  By default
 * a kernel waits for that work before it reads anything.
 *
 * ANS_DESC_INPUTS_SETTLED: the caller states that this layer's table, stream, offsets and lane
 * metadata (and, for the *_batch call, the descriptor array in device memory) were complete
 * before the work that precedes this call on the stream began: weights loaded and tables built
 * once, decoded many times, the usual case at inference time.  With the bit set on every layer
 * of a launch the kernel reads its inputs, stages its table and begins to decode into shared
 * memory while the preceding work drains, and waits for it only before its first write to
 * device memory (outputs, status word).
 *
 * ANS_DESC_OUTPUT_IDLE (only together with ANS_DESC_INPUTS_SETTLED): the caller also states that
 * the work that precedes this call on the stream neither reads nor writes this layer's d_out (a
 * decode into one buffer while the layer before it is still being consumed from another).  The
 * kernel then does not wait for the preceding work at all, except before it sets a bit in
 * *d_status.  Work that follows the call on the stream is ordered after it as always.
 *
 * ans_decode_layer, which writes d_symbols_out and not d_out, honours the first flag only.
 * The host-buffer calls (ans_decode_dequant_host, ans_decode_dequant_host_noalloc) copy their
 * inputs in on the same stream and ignore the flags; so do the encoder and ans_decode_gemm_bf16. */
#define ANS_DESC_INPUTS_SETTLED 1u
#define ANS_DESC_OUTPUT_IDLE 2u

/* Library version (major*100 + minor). */
int ans_version(void);

/* Text for an ANS_* code; never NULL. */
const char* ans_strerror(int code);

/* The cudaError_t of the most recent failed CUDA call made by this library (0 if none). */
int ans_last_cuda_error(void);

/*
 * Bytes one layer's device table takes for a given table_log (a multiple of 256).
 * Section II-A sizes the paper's table at 3 bytes per state; this library stores 32-bit
 * entries plus a pre-walked copy for chains of zero-bit transitions.
 */
int ans_table_bytes(int table_log, size_t* h_bytes_out);

/*
 * Build the decode tables of n_layers layers on the device (Section II-A: per state the
 * symbol, nb_bits and newX).  States are handed to symbols in bit-reversal order and a
 * symbol's states are numbered upwards, the same rule an encoder must use.
 *   h_norm_freqs   [n_layers][256]  normalised frequencies; row l sums to 1 << h_table_log[l]
 *   h_alphabet     [n_layers]       symbols in use (frequencies at or beyond it must be 0)
 *   h_table_log    [n_layers]       R per layer, 1..14
 *   d_tables       device buffer, 256-byte aligned, d_tables_bytes long; layer l's table
 *                  is written at byte offset h_table_offsets_out[l]
 *   h_table_offsets_out [n_layers]  filled on return
 * The host arrays are read before the call returns.  Asynchronous on `stream`.
 * Errors: INVALID_ARG, UNSUPPORTED (R), BAD_FREQS, BUFFER_TOO_SMALL, CUDA.
 */
int ans_build_decode_tables(const uint32_t* h_norm_freqs, const int32_t* h_alphabet,
                            const int32_t* h_table_log, int n_layers,
                            void* d_tables, size_t d_tables_bytes,
                            uint64_t* h_table_offsets_out, void* stream);

/*
 * Fill work_begin / work_count of every descriptor (one work item per group of up to 4
 * consecutive sub-streams of a layer) so that a batch can run as ONE launch.  Call it on the host array before copying it to the
 * device.  h_total_work_out receives the number of work items.  Host only.
 */
int ans_plan_batch(ans_layer_desc* h_descs, int n_layers, uint64_t* h_total_work_out);

/*
 * Decode one layer to symbols (Section II-A decode rule over the layer's vector of states,
 * Section III-B): d_symbols_out receives h_desc->n_symbols bytes; d_out/out_dtype/scale are
 * ignored.  d_status (one uint32 in device memory, zeroed by the caller or by an earlier
 * ans_read_status) receives ANS_STATUS_* bits by atomic OR.  Asynchronous on `stream`.
 */
int ans_decode_layer(const ans_layer_desc* h_desc, uint8_t* d_symbols_out,
                     uint32_t* d_status, void* stream);

/*
 * Decode one layer and dequantise it in the same kernel (Section II-B):
 * d_out[i] = (float)(q_i - zero_point) * scale, one IEEE single-precision multiply, then
 * for ANS_BF16 a round-to-nearest-even to bfloat16; ANS_U8 stores q_i itself.
 */
int ans_decode_dequant(const ans_layer_desc* h_desc, uint32_t* d_status, void* stream);

/*
 * The same for n_layers layers in one kernel launch.  d_descs is the device copy of
 * h_descs (after ans_plan_batch); the host copy is only used for validation and sizing.
 * All layers of one call share `layout`; out_dtype, table_log and every other field may
 * differ from layer to layer.
 */
int ans_decode_dequant_batch(const ans_layer_desc* d_descs, const ans_layer_desc* h_descs,
                             int n_layers, uint32_t* d_status, void* stream);

/*
 * Wait for `stream`, copy the status word to *h_status_out, clear it on the device.
 * Returns ANS_ERR_CORRUPT if any bit was set, ANS_OK otherwise.
 */
int ans_read_status(uint32_t* d_status, void* stream, uint32_t* h_status_out);

/*
 * End-to-end helper with HOST buffers: copies the layer's stream, offsets and lane
 * metadata to the device scratch the caller provides, decodes + dequantises, copies the
 * result back to h_out and waits.  h_desc's d_stream/d_sub_offsets/d_lane_meta/d_out are
 * IGNORED; the host pointers given here are used instead.  d_table must already be on the
 * device.  d_scratch must hold ans_host_scratch_bytes(...) bytes, 256-byte aligned.
 * Synchronous: returns after h_out is complete; returns ANS_ERR_CORRUPT on a bad stream.
 */
int ans_host_scratch_bytes(const ans_layer_desc* h_desc, uint64_t stream_bytes, size_t* h_bytes_out);
int ans_decode_dequant_host(const ans_layer_desc* h_desc,
                            const uint8_t* h_stream, uint64_t stream_bytes,
                            const uint64_t* h_sub_offsets, const void* h_lane_meta,
                            void* h_out, void* d_scratch, size_t d_scratch_bytes, void* stream);

/*
 * (No counterpart in the paper: this is a deployment convenience.)
 * The host-buffer decode call for callers that cannot allocate device memory at all: code that
 * runs where cudaMalloc is forbidden or unavailable (a plug-in inside a host application that
 * owns the memory budget, a real-time loop that may not enter the allocator, a process started
 * with a device memory pool it may not grow).  The call takes ONLY host buffers: the layer's
 * normalised frequencies, its compressed stream, offsets and lane metadata, and the host
 * output.  The table is built and everything is staged inside a fixed 8 MiB working area that
 * belongs to the library image (each GPU that loads the library holds that area until the
 * process exits; ans_noalloc_max_bytes reports its size).  h_desc's d_* pointers are ignored.
 *   - A layer whose table + stream + offsets + lane metadata + output (each rounded up to 256
 *     bytes, plus 256) exceed the area is refused with ANS_ERR_BUFFER_TOO_SMALL.
 *   - The first call on each device looks up the area's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one area, which keeps the last call's bytes: two calls
 *     that overlap on the GPU (different streams or host threads) race.  The call itself is
 *     synchronous: it returns after h_out is complete.
 *   - No cudaMalloc / cudaFree or other device allocation is made.
 * Returns ANS_OK, ANS_ERR_CORRUPT for an unsound stream, or another ANS_ERR_* code.
 */
int ans_noalloc_max_bytes(size_t* h_bytes_out);
int ans_decode_dequant_host_noalloc(const ans_layer_desc* h_desc, const uint32_t* h_norm_freqs,
                                    int alphabet, const uint8_t* h_stream, uint64_t stream_bytes,
                                    const uint64_t* h_sub_offsets, const void* h_lane_meta,
                                    void* h_out, void* stream);

/* ------------------------------------------------------------------------------------
 * Host-side packer: makes the streams the decoder reads.  Runs on the CPU, off the
 * inference path (the paper compresses offline, Section III-A); it is here so that a
 * user can produce containers without any other tool.
 * ------------------------------------------------------------------------------------ */

/*
 * Histogram -> normalised frequencies summing to 1 << table_log; every symbol that occurs
 * keeps at least one state.  h_counts[alphabet], h_freqs_out[256] (entries >= alphabet = 0).
 */
int ans_host_normalize_freqs(const uint64_t* h_counts, int alphabet, int table_log,
                             uint32_t* h_freqs_out);

/* Upper bound of the stream bytes ans_host_pack_layer / ans_host_pack_channels can produce. */
int ans_host_pack_bound(uint64_t n_symbols, uint32_t chunk_symbols, uint32_t lanes,
                        int layout, uint64_t* h_bytes_out);

/*
 * Encode one layer (Section II-A: follow the automaton's transition for each symbol and
 * append its label bits) into the chosen container.
 *   h_symbols[n_symbols]; h_freqs[256] as given to ans_build_decode_tables
 *   h_stream_out (capacity stream_cap), h_sub_offsets_out[n_sub + 1],
 *   h_lane_meta_out: uint16_t[n_sub][32] (interleaved) or uint32_t[n_sub][32] (private, quads);
 *                    unused (may be NULL) for the strips layout
 *   n_threads: host threads to use (<= 0: all)
 * *h_stream_bytes_out receives the bytes written.
 */
int ans_host_pack_layer(const uint8_t* h_symbols, uint64_t n_symbols,
                        const uint32_t* h_freqs, int alphabet, int table_log,
                        uint32_t chunk_symbols, uint32_t lanes, int layout,
                        uint8_t* h_stream_out, uint64_t stream_cap, uint64_t* h_stream_bytes_out,
                        uint64_t* h_sub_offsets_out, void* h_lane_meta_out, int n_threads);

/*
 * The same for ANS_LAYOUT_CHANNELS (Section III-B: one stream per input channel), which needs
 * the piece size: h_symbols is the tensor as stored (O x I x H x W), piece_symbols = H * W,
 * lanes = I, chunk_symbols = n_symbols for one chunk per layer.  No lane metadata is written.
 */
int ans_host_pack_channels(const uint8_t* h_symbols, uint64_t n_symbols,
                           const uint32_t* h_freqs, int alphabet, int table_log,
                           uint32_t chunk_symbols, uint32_t lanes, uint32_t piece_symbols,
                           uint8_t* h_stream_out, uint64_t stream_cap, uint64_t* h_stream_bytes_out,
                           uint64_t* h_sub_offsets_out, int n_threads);

/* ------------------------------------------------------------------------------------
 * The compress side on the device.  Off the inference path (the paper compresses offline,
 * Section III-A); it serves training-time use, where the entropy of the quantised weights is
 * wanted at every step (Section II-C, Eq. 3 regularises the entropy H_W of the weights) and
 * the weights are already on the device.  All asynchronous on `stream`; every d_* buffer is
 * the caller's.
 * ------------------------------------------------------------------------------------ */

/* Histogram of n_symbols bytes: d_counts[256] (zeroed by the call, then counted). */
int ans_histogram_device(const uint8_t* d_symbols, uint64_t n_symbols, uint64_t* d_counts, void* stream);

/*
 * Entropy of a histogram over its first `alphabet` entries, in double precision:
 * d_entropy_out[0] = -sum_s p_s log2 p_s (bits per symbol, p_s = count_s / total; 0 for an empty
 * histogram), d_entropy_out[1] = that times the total (bits for the layer): the H_W of Eq. 3.
 */
int ans_entropy_device(const uint64_t* d_counts, int alphabet, double* d_entropy_out, void* stream);

/*
 * Histogram -> frequencies summing to 1 << table_log, the rule of ans_host_normalize_freqs
 * (floor share, at least one state per symbol that occurs, largest remainders up, largest
 * shares down, ties to the lower symbol), in integer arithmetic: d_freqs_out[256].
 * Bit 1 of *d_status (optional, OR-ed) is set if the histogram is empty, has more symbols than
 * states or more than 2^50 counts.
 */
int ans_normalize_freqs_device(const uint64_t* d_counts, int alphabet, int table_log, uint32_t* d_freqs_out,
                               uint32_t* d_status, void* stream);

/*
 * Encode one layer on the device into the strips container (Section II-A: encoding follows a
 * transition of the automaton and appends the bits that label it), byte for byte what
 * ans_host_pack_layer writes for ANS_LAYOUT_STRIPS (the only layout this call takes).
 *   d_symbols[n_symbols]; d_table: the layer's table from ans_build_decode_tables (it carries
 *   the frequencies the encoder needs); d_stream_out: stream_cap bytes, 16-byte aligned, zeroed
 *   and filled by the call (ans_host_pack_bound gives a sufficient stream_cap);
 *   d_sub_offsets_out[n_sub + 1]: byte offsets, the last one the stream's size;
 *   d_scratch: ans_encode_scratch_bytes(...) bytes, 256-byte aligned.
 * *d_status (OR-ed): bit 2 = the stream did not fit stream_cap (what did not fit is not
 * written), bit 4 = a symbol without a state in the table, or a lane longer than 65535 bits.
 */
int ans_encode_scratch_bytes(uint64_t n_symbols, uint32_t chunk_symbols, uint32_t lanes, size_t* h_bytes_out);
/* The same for the channels container (Section III-B: one stream per input channel of a tensor
 * stored O x I x H x W): byte for byte what ans_host_pack_channels writes; sizes as there
 * (piece_symbols = H * W in 1 .. ANS_MAX_PIECE_SYMBOLS, lanes = I, chunk_symbols and n_symbols
 * multiples of lanes * piece_symbols); buffers, scratch and status as for ans_encode_layer_device. */
int ans_encode_channels_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                               uint32_t chunk_symbols, uint32_t lanes, uint32_t piece_symbols,
                               uint8_t* d_stream_out, uint64_t stream_cap, uint64_t* d_sub_offsets_out,
                               void* d_scratch, size_t d_scratch_bytes, uint32_t* d_status, void* stream);
/* The same for the quads container: byte for byte what ans_host_pack_layer writes for
 * ANS_LAYOUT_QUADS, d_lane_meta_out[n_sub][32] included (initial state | first word << 16).  Any
 * chunk_symbols >= 1; bit 4 of *d_status also if a sub-stream is longer than 65535 words. */
int ans_encode_quads_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                            uint32_t chunk_symbols, uint32_t lanes, uint8_t* d_stream_out, uint64_t stream_cap,
                            uint64_t* d_sub_offsets_out, uint32_t* d_lane_meta_out, void* d_scratch,
                            size_t d_scratch_bytes, uint32_t* d_status, void* stream);
int ans_encode_layer_device(const uint8_t* d_symbols, uint64_t n_symbols, const void* d_table, int table_log,
                            uint32_t chunk_symbols, uint32_t lanes, int layout, uint8_t* d_stream_out,
                            uint64_t stream_cap, uint64_t* d_sub_offsets_out, void* d_scratch,
                            size_t d_scratch_bytes, uint32_t* d_status, void* stream);

/* ------------------------------------------------------------------------------------
 * Decode fused into its consumer (Section I, Section III-C: the weights are decompressed just
 * before the computation that uses them and the decoded weights never travel through DRAM):
 *   Y[M x N] = X[M x K] * W^T,  W[N x K] read in compressed form,
 * X bfloat16 row-major, Y float row-major, the product on the tensor cores with fp32
 * accumulation (the order of the K-direction sums is the hardware's).  W is dequantised to
 * bfloat16 exactly as ans_decode_dequant would (Section II-B).
 *   h_desc: W's layer: ANS_LAYOUT_STRIPS, chunk_symbols = 4096, lanes = 32, table_log <= 12,
 *           n_symbols = N * K, the symbols being W in blocks of 64 x 64: block (n / 64, k / 64)
 *           holds 4096 consecutive symbols, blocks ordered [N / 64][K / 64].  Inside a block
 *           element (r, c) (r: output feature, c: input feature, both modulo 64) is symbol
 *             (r / 8) * 512 + (r % 8) * 64 + ((c / 8) ^ (r % 8)) * 8 + c % 8
 *           (the order in which the tensor core reads a 128-byte-swizzled K-major tile, so
 *           that a decoded block is an operand as it lies).  d_out / out_dtype are ignored.
 *   1 <= M <= 128; N and K multiples of 64; d_x and d_y 16-byte aligned.
 * d_status as for the decode calls.  Asynchronous on `stream`.
 * ------------------------------------------------------------------------------------ */
int ans_decode_gemm_bf16(const ans_layer_desc* h_desc, const void* d_x, int M, int N, int K, float* d_y,
                         uint32_t* d_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ANS_B200_H */
