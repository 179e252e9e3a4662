/*
 * tq -- fused dictionary-decode + GEMV/GEMM for Tiny-QMoE-format weights on B200 (sm_100a).
 *
 * C ABI.  Every call returns an int status (TQ_OK = 0, negative = error); nothing throws or
 * aborts across this boundary.  Pointers are marked HOST or DEVICE.  The library never calls
 * cudaMalloc on behalf of the caller: all device memory is caller-owned (a tq_ddict / tq_dmat
 * only remembers addresses inside the caller's buffer, so the buffer must outlive the handle).
 * Streams are passed as void* (a cudaStream_t); device calls are asynchronous on that stream
 * unless stated otherwise.  Handles are opaque, library-owned host objects released with the
 * matching *_free call.
 *
 * The data format is the paper's (Section 4, Listings 2-4): 8-bit weight levels, a table of the
 * K <= 65534 most frequent windows of 4 consecutive levels (code = rank + 1), and per matrix a
 * uint16 token stream in which every aligned group of 4 levels is either its code or the marker
 * 0xFFFF followed by the 4 levels, each widened to 16 bits.
 */
#ifndef TQ_H_
#define TQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TQ_OK 0
#define TQ_ERR_INVALID_ARG (-1)
#define TQ_ERR_CORRUPT_STREAM (-2)
#define TQ_ERR_BUFFER_TOO_SMALL (-3)
#define TQ_ERR_UNSUPPORTED_SHAPE (-4)
#define TQ_ERR_CUDA (-5)
#define TQ_ERR_TIMEOUT (-6)
#define TQ_ERR_NOMEM (-7)

#define TQ_ESCAPE 0xFFFFu
#define TQ_MAX_ENTRIES 65534u

/* Device status bits (tq_device_status). */
#define TQ_STATUS_BAD_CODE 1u      /* a code of 0 or > K was met; it decoded as four zero bytes */
#define TQ_STATUS_BAD_ROW 2u       /* a row segment did not hold exactly cols/4 groups          */
#define TQ_STATUS_WAIT_EXPIRED 4u  /* a bounded wait inside a kernel ran out                    */

typedef struct tq_dict tq_dict;   /* HOST: the compression table                                */
typedef struct tq_ddict tq_ddict; /* handle of a table resident in DEVICE memory                */
typedef struct tq_dmat tq_dmat;   /* handle of one compressed matrix resident in DEVICE memory  */

/* Human-readable text for a status code (static storage). */
const char* tq_strerror(int status);

/* Text of the calling thread's most recent CUDA failure behind a TQ_ERR_CUDA (static storage,
 * empty if none). */
const char* tq_last_cuda_error(void);

/* Worker threads used by the host calls below (0 = hardware concurrency).  Returns the value in
 * effect. */
int tq_set_num_threads(int n);

/* ------------------------------------------------------------------------------------------
 * Host side: quantize, build the table, encode.
 * ---------------------------------------------------------------------------------------- */

/* Per-tensor min-max quantizer at 8 bits (Listing 1): scale = (max-min)/255,
 * zero = round(-min/scale), q = clamp(round(x/scale) + zero, 0, 255); fp32, round half to even.
 * x, q: HOST, n elements.  Fails with TQ_ERR_INVALID_ARG when max == min. */
int tq_quantize_tensor(const float* x, uint64_t n, uint8_t* q, float* scale, float* zero);

/* The same quantizer at another bit count (Listing 1's configure step: maxq = 2^bits - 1; Section 3
 * reports 2, 4, 6 and 8 bits): levels 0..maxq, still one byte per level, so every later step of the
 * path (table, tokens, decode, products) takes them unchanged.  bits: integer 1..8, anything else
 * (the listing's ternary setting included, which makes no integer level) is TQ_ERR_INVALID_ARG. */
int tq_quantize_tensor_bits(const float* x, uint64_t n, int bits, uint8_t* q, float* scale, float* zero);

/* Per-output-row symmetric int8 quantizer used by the benchmark workloads (not in the paper;
 * it produces the same kind of 8-bit level Listing 1 does, W ~ scale_r * q):
 * scale_r = max_c |w[r][c]| / 127 (1 for an all-zero row), q = clamp(round(w/scale_r), -127, 127).
 * w: HOST [rows][cols] row-major; q: HOST [rows][cols]; scale: HOST [rows]. */
int tq_quantize_rows(const float* w, uint32_t rows, uint32_t cols, int8_t* q, float* scale);

/* Same computation on the GPU, bit-identical results.  d_w, d_q, d_scale: DEVICE. */
int tq_quantize_rows_device(const float* d_w, uint32_t rows, uint32_t cols, int8_t* d_q,
                            float* d_scale, void* cuda_stream);

/* Frequent-sequence table (Listing 2).  Counts every window of 4 consecutive bytes (stride 1) of
 * each flattened matrix -- windows never span two matrices -- and keeps the top_k most frequent
 * in descending count order; equal counts keep first-seen order (matrix order, then position);
 * code = rank + 1.  Code 65535 is the escape marker, so at most 65534 entries are kept
 * (top_k > 65534 is clamped).  mats: HOST array of n_mats HOST pointers; n_elems: HOST, bytes
 * per matrix.  The total window count must be < 2^32.  *out is owned by the library. */
int tq_build_dictionary(const uint8_t* const* mats, const uint64_t* n_elems, int n_mats,
                        uint32_t top_k, tq_dict** out);

/* tq_build_dictionary for matrices that are on the DEVICE (d_mats: HOST array of n_mats DEVICE
 * pointers, 4-byte aligned): the windows are counted on the GPU (keys, radix sort and run lengths
 * per matrix, a hash table over all matrices) and only the candidates for the table (count at
 * least that of rank top_k, every tie included) come back to the host, where they are ranked by
 * the same rule -- the result is the table tq_build_dictionary builds.  d_workspace: DEVICE,
 * 256-byte aligned, tq_build_dictionary_device_size bytes (about 28 bytes per byte of the largest
 * matrix plus up to 2.6 GB).  TQ_ERR_BUFFER_TOO_SMALL if the data has more distinct windows than
 * the hash table holds (2^28 at most), TQ_ERR_UNSUPPORTED_SHAPE if more than 2^24 windows tie at
 * the cut: use tq_build_dictionary then.  Synchronises cuda_stream. */
int tq_build_dictionary_device_size(const uint64_t* n_elems, int n_mats, uint64_t* workspace_bytes);
int tq_build_dictionary_device(const uint8_t* const* d_mats, const uint64_t* n_elems, int n_mats,
                               uint32_t top_k, void* d_workspace, uint64_t workspace_bytes,
                               void* cuda_stream, tq_dict** out);

/* A table from an explicit entry list (K x 4 bytes, rank order, HOST). */
int tq_dict_from_entries(const uint8_t* entries, uint32_t K, tq_dict** out);

/* Borrow the table: *K entries, *entries -> K x 4 bytes in rank order (HOST, valid until
 * tq_dict_free).  counts (may be NULL) -> K occurrence counts (zeros for tq_dict_from_entries). */
int tq_dict_entries(const tq_dict* d, uint32_t* K, const uint8_t** entries,
                    const uint64_t** counts);

/* Token stream of one matrix (Listing 3): aligned groups of 4 bytes; a group found in the table
 * is written as its code, any other as 0xFFFF followed by its 4 bytes widened to uint16; a tail of
 * n mod 4 bytes is written as 0xFFFF followed by those bytes.  codes: HOST, n bytes.  out: HOST,
 * room for out_cap uint16; out == NULL only queries the size.  *out_len receives the stream length
 * in uint16 units; n_hits / n_miss (may be NULL) the number of coded / escaped groups.
 * TQ_ERR_BUFFER_TOO_SMALL if out_cap is short. */
int tq_encode(const tq_dict* d, const uint8_t* codes, uint64_t n, uint16_t* out, uint64_t out_cap,
              uint64_t* out_len, uint64_t* n_hits, uint64_t* n_miss);

void tq_dict_free(tq_dict* d);

/* ------------------------------------------------------------------------------------------
 * Device side: upload, decompress, fused products.
 * ---------------------------------------------------------------------------------------- */

/* Bytes of DEVICE memory a table needs: the full 16-bit index range (256 KB: words past the last
 * entry are zero, so a kernel may index the table with any token) and a 2 MB map from 4-byte
 * windows to codes for the device-side encoder. */
int tq_dict_upload_size(const tq_dict* d, uint64_t* device_bytes);

/* Copy the table into the caller's DEVICE buffer d_buf (256-byte aligned, d_buf_bytes long) and
 * return a handle.  Synchronises cuda_stream before returning. */
int tq_dict_upload(const tq_dict* d, void* d_buf, uint64_t d_buf_bytes, void* cuda_stream,
                   tq_ddict** out);
void tq_ddict_free(tq_ddict* d); /* host handle only */

/* Device layouts of a compressed matrix. */
#define TQ_LAYOUT_STREAM 0 /* the paper's token stream, byte for byte, cut into per-row segments */
#define TQ_LAYOUT_PLANES 1 /* the same tokens re-tiled without loss: one 16-bit token per group in a
                              fixed-stride plane (code, or 0xFFFF), and the 4 bytes that followed each
                              0xFFFF packed into one word of a second, compact plane.  2 + 4*miss_rate
                              bytes per group instead of 2 + 8*miss_rate, and no sequential parse. */

#define TQ_LAYOUT_TILES 2  /* the PLANES content ordered for the integer tensor-core GEMV: tokens in 1 KB
                              tiles of 16 rows x 32 groups laid out in the register order of an 8-bit
                              mma (so a looked-up word is an operand as it stands), raw words in one
                              stream, each addressed by the token that replaces its marker.  Same bytes per group as
                              PLANES.  tq_decompress and tq_fused_gemv accept it; tq_fused_gemm does not.
                              Requires cols <= TQ_TILES_MAX_COLS.  The kernels hold the table they index in shared
                              memory, which has room for TQ_TILES_TABLE_WORDS words: a group whose code is
                              beyond that is stored as Listing 3 stores a group that is not in the table
                              (marker + its 4 bytes), i.e. the image is the stream Listing 3 produces with
                              top_k = TQ_TILES_TABLE_WORDS - 1.  Same decoded bytes, 4 more bytes per such
                              group (tq_dmat_info.n_raw_words counts them). */
#define TQ_TILES_TABLE_WORDS 33024u
#define TQ_TILES_MAX_COLS 65536u /* 32-bit integer accumulators; rows of more than 8448 columns go through the
                                    column-panel kernel, whose shared memory need does not grow with the row */
#define TQ_TILES_RING_WORDS 1024u /* a miss token of the image is 0xFC00 + (index of its raw word mod 1024) */

/* Bytes of DEVICE memory the layout of this stream needs.  stream: HOST.  Requires cols % 4 == 0
 * (no aligned group straddles two rows; true of every LLaMA shape), else TQ_ERR_UNSUPPORTED_SHAPE. */
int tq_upload_size(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                   int layout, uint64_t* device_bytes);

/* Validate a token stream (Listing 4's walk must yield exactly rows*cols bytes, every code must be
 * in 1..K, every raw slot <= 255) and place it in the caller's DEVICE buffer in the given layout,
 * together with the per-row scale and zero point of the dequantisation scale_r * (q - zero_r)
 * (Listing 1).  row_zero may be NULL (all zero).  levels_signed != 0: the decoded byte is an int8
 * bit pattern (per-row symmetric quantizer); 0: an unsigned level 0..255 (Listing 1).
 * stream, row_scale, row_zero: HOST.  d_buf: DEVICE, 256-byte aligned.  Synchronises cuda_stream
 * before returning.  A corrupt stream is rejected with TQ_ERR_CORRUPT_STREAM and nothing is
 * uploaded. */
int tq_upload(const tq_ddict* dict, const uint16_t* stream, uint64_t stream_len, uint32_t rows,
              uint32_t cols, const float* row_scale, const float* row_zero, int levels_signed,
              int layout, void* d_buf, uint64_t d_buf_bytes, void* cuda_stream, tq_dmat** out);

/* The TQ_LAYOUT_TILES image exactly as tq_upload would place it in device memory, built in HOST
 * memory instead (for inspection, or to prepare images ahead of time).  out == NULL only queries
 * *out_bytes.  offsets[5] receives the byte offsets of: row scales, row zero points, the tile_raw
 * index (tiles + 1 uint32), the token tiles (1 KB each), the raw words; dims[2] receives tiles per
 * row block and row blocks.  Tile layout: see TQ_LAYOUT_TILES; inside a tile, lane l = 4*g + t
 * holds at byte h*512 + l*16 the 8 tokens of row 16*row_block + g + 8*h, groups
 * 32*step + 8*t .. + 7. */
int tq_tiles_image_host(const tq_dict* d, const uint16_t* stream, uint64_t stream_len, uint32_t rows,
                        uint32_t cols, const float* row_scale, const float* row_zero, uint8_t* out,
                        uint64_t out_cap, uint64_t* out_bytes, uint64_t* offsets, uint32_t* dims);

/* tq_upload for 8-bit levels that are already on the device (for instance the output of
 * tq_quantize_rows_device): Listing 3's decision for every aligned group (in the table: its code;
 * else the marker and its 4 bytes) is taken on the GPU and written straight into the
 * TQ_LAYOUT_TILES image, which is byte for byte the image tq_upload builds from the host stream.
 * d_levels: DEVICE, rows x cols bytes, row-major, 16-byte aligned; d_row_scale / d_row_zero: DEVICE
 * [rows] (zero may be NULL).  d_buf: DEVICE, 256-byte aligned, tq_upload_device_size bytes (sized
 * for the worst case of no group in the table; tq_dmat_info.device_bytes reports what the image
 * uses, the rest may be released by a caller who can shrink its buffer).  Requires cols % 4 == 0.
 * The dictionary must have been uploaded with tq_dict_upload.  Synchronises cuda_stream. */
int tq_upload_device_size(uint32_t rows, uint32_t cols, uint64_t* device_bytes);
int tq_upload_device(const tq_ddict* dict, const uint8_t* d_levels, uint32_t rows, uint32_t cols,
                     const float* d_row_scale, const float* d_row_zero, int levels_signed, void* d_buf,
                     uint64_t d_buf_bytes, void* cuda_stream, tq_dmat** out);

/* Row shard (for a model split by output rows over several GPUs, one process each: every GPU holds
 * the whole table and the whole activation, decodes and multiplies its own rows, and the outputs are
 * concatenated; the product needs no reduction because a row's sum never leaves its GPU).  Rows
 * row_begin .. row_end-1 of the rows x cols matrix at d_levels become a compressed matrix of their
 * own, exactly as tq_upload_device would make it from those rows alone: Listing 3 takes its decision
 * per aligned group, and with cols % 4 == 0 no group spans two rows, so the shard's tokens are the
 * tokens those rows have in the unsharded stream.  d_row_scale / d_row_zero: the full [rows] arrays.
 * The first row of the shard must start on a 16-byte boundary (TQ_ERR_INVALID_ARG otherwise).
 * d_buf: tq_upload_device_size(row_end - row_begin, cols) bytes. */
int tq_upload_device_rows(const tq_ddict* dict, const uint8_t* d_levels, uint32_t rows, uint32_t cols,
                          uint32_t row_begin, uint32_t row_end, const float* d_row_scale,
                          const float* d_row_zero, int levels_signed, void* d_buf, uint64_t d_buf_bytes,
                          void* cuda_stream, tq_dmat** out);

typedef struct tq_dmat_info {
  uint32_t rows, cols, K;
  int32_t layout, levels_signed;
  uint64_t n_hits, n_miss;   /* coded / escaped groups                                        */
  uint64_t stream_bytes;     /* the paper's stream: 2 * (n_hits + 5 * n_miss)                  */
  uint64_t payload_bytes;    /* bytes a kernel reads per pass: token segments with their
                                padding + per-row index + scales                              */
  uint64_t device_bytes;     /* whole footprint in the caller's buffer                         */
  uint64_t n_raw_words;      /* 4-byte raw words in the device layout: n_miss, plus for
                                TQ_LAYOUT_TILES the groups coded beyond TQ_TILES_TABLE_WORDS     */
} tq_dmat_info;
int tq_dmat_get_info(const tq_dmat* m, tq_dmat_info* info);

/* Decompress (Listing 4): write the rows*cols decoded bytes, row-major, to d_codes (DEVICE). */
int tq_decompress(const tq_dmat* m, uint8_t* d_codes, void* cuda_stream);

/* Compressed linear layer for small batches (Section 2.3: weights are expanded layer by layer,
 * then used as an ordinary linear layer; here the expansion, Listing 1's scale*(q-zero) and the
 * product are one kernel and the weights never reach memory):
 *   y[b][r] = scale_r * sum_c (q[r][c] - zero_r) * x[b][c].
 * d_x_bf16: DEVICE [B][cols] bf16, 16-byte aligned; B in 1..32; d_y: DEVICE [B][rows] fp32.
 *
 * Arithmetic and its domain.  TQ_LAYOUT_STREAM / TQ_LAYOUT_PLANES: exact int8 x bf16 products,
 * fp32 accumulation.  TQ_LAYOUT_TILES: each vector x[b] is put on a fixed-point grid 30 bits below
 * the power of two above its largest magnitude (X = round(x * 2^(30-e)), max |x[b]| < 2^e) and the
 * sums are exact integers, so the result does not depend on how the work is split and
 *   |y[b][r] - exact| <= scale_r * 2^(e-31) * sum_c |q[r][c] - zero_r|   (+ one fp32 rounding of y).
 * An element keeps every bit of its bf16 value while it is at most 2^22 times smaller than the
 * largest element of its vector; smaller ones are rounded to the grid.  Against max_r |y[b][r]| this
 * is far inside 2e-3 unless the row sums rest on elements more than about 2^20 times smaller than one
 * that meets (near-)zero weights.  Subnormal and smallest-normal bf16 inputs are exact.  A vector with
 * an Inf or NaN element yields NaN for all of its outputs (other vectors are unaffected); the status
 * word is not touched.
 *
 * TQ_LAYOUT_TILES with more than two vectors (or rows too long for the one-vector kernel) stages
 * digit planes of the activations in a scratch area inside the matrix's own device image: calls
 * on the same matrix must not overlap on the GPU (calls on one stream never do). */
int tq_fused_gemv(const tq_dmat* m, const void* d_x_bf16, int B, float* d_y, void* cuda_stream);

/* The same call with HOST operands: copies x to the DEVICE staging buffer d_x_stage ([B][cols]
 * bf16), runs the kernel, copies y back from d_y_stage ([B][rows] fp32), all on cuda_stream, and
 * does not synchronise.  h_x_bf16 / h_y should be pinned for the copies to be asynchronous. */
int tq_fused_gemv_host(const tq_dmat* m, const void* h_x_bf16, int B, float* h_y, void* d_x_stage,
                       float* d_y_stage, void* cuda_stream);

/* tq_fused_gemv_host for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a convenience of the library).  Such callers exist: code running inside a stream
 * capture or a latency-critical serving loop where cudaMalloc would synchronise the device, a
 * plug-in handed a fixed memory budget by its host application, a process that only receives
 * device pointers from elsewhere.  The staging copies of x and y live in a fixed 1.5 MiB array
 * that is part of the library image (every GPU that loads the library keeps it until the process
 * exits), so the call is limited to B * cols <= 262144 and B * rows <= 262144 and returns
 * TQ_ERR_UNSUPPORTED_SHAPE (text in tq_last_cuda_error) beyond that.  No cudaMalloc, cudaFree or
 * other allocating routine is called.  The first call on each device looks up the array's device
 * address with that device current; make that first call outside any stream capture.  All calls
 * on a device share the one array: nothing in it has to start at zero (x is overwritten by the
 * copy, y by the kernel, before either is read), but two calls whose GPU work overlaps (different
 * streams, or different threads) race on it -- serialise them.  The array that is used is the
 * current device's, so the device the matrix lives on must be current: TQ_ERR_INVALID_ARG otherwise.
 * h_x_bf16, h_y: HOST, as for tq_fused_gemv_host; asynchronous on cuda_stream. */
int tq_fused_gemv_host_static(const tq_dmat* m, const void* h_x_bf16, int B, float* h_y,
                              void* cuda_stream);

/* Same product for prefill-sized batches (M tokens): decoded weight tiles are converted to bf16
 * (exact: |level| <= 255) in shared memory and fed to tcgen05 tensor-core MMAs with fp32
 * accumulation; scale and zero point are applied in fp32 afterwards.
 * d_X_bf16: DEVICE [M][cols] bf16, 16-byte aligned; d_Y: DEVICE [M][rows] fp32. */
int tq_fused_gemm(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, void* cuda_stream);

/* The prefill-sized product for a TQ_LAYOUT_TILES matrix, in two phases on cuda_stream that share a
 * caller-provided DEVICE workspace (256-byte aligned, tq_gemm_workspace_size bytes = the matrix as
 * bf16, padded to whole tiles): the layer is decompressed once into the workspace as bf16
 * (level - zero point: exact when every zero point is an integer no further than 256 from any level,
 * which holds for Listing 1's zero points of tensors that straddle 0; TQ_ERR_UNSUPPORTED_SHAPE for
 * other zero points, here and in tq_fused_gemm), then a persistent tcgen05 GEMM reads both
 * operands by TMA and applies the row scale in fp32.  Same result definition, argument layout and
 * alignment as tq_fused_gemm; the workspace may be reused by the next call on the same stream. */
int tq_gemm_workspace_size(const tq_dmat* m, uint64_t* bytes);
int tq_fused_gemm_ws(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, void* d_workspace,
                     uint64_t workspace_bytes, void* cuda_stream);
/* The two phases on their own: a layer's weights do not depend on the activations, so phase 1 may run
 * ahead of time, and tq_decode_bf16_stack (declared with the stack calls below) runs it for every
 * matrix of a stack in one launch.  tq_gemm_bf16_ws multiplies by a workspace that one of them
 * filled for this matrix. */
int tq_decode_bf16(const tq_dmat* m, void* d_workspace, uint64_t workspace_bytes, void* cuda_stream);
int tq_gemm_bf16_ws(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, const void* d_workspace,
                    void* cuda_stream);

/* A stack: several TQ_LAYOUT_TILES matrices that share one table (for instance every linear layer
 * of a decoder, Section 2.3: the weights are expanded layer by layer), bound to their operands and
 * executed by ONE persistent launch in which every SM loads the table into shared memory once and
 * then streams its share of the row blocks of all the matrices.  The products are independent of
 * one another: a caller whose layers feed each other makes one stack per group of layers that can
 * run together (q/k/v; gate/up; ...).  d_x[i]: DEVICE bf16 [B][cols_i], 16-byte aligned; d_y[i]:
 * DEVICE fp32 [B][rows_i]; B in 1..32.  One vector (two where the digits of two fit beside the
 * table for every matrix) runs the kernel whose decoding warps multiply on the spot; more vectors,
 * and matrices whose rows are too long for that kernel, run ONE pass of the tcgen05 kernel for all
 * vectors, preceded by a small launch that turns the activations into digit planes
 * (tq_stack_launches tells how many launches a call makes).  mats, d_x, d_y: HOST arrays of n_mats
 * entries.  The work split, the operand addresses and the scratch of the digit planes are written
 * to the caller's DEVICE buffer d_buf (256-byte aligned, tq_stack_size bytes for these matrices and
 * this B; B = 0 for a stack without operands), which must outlive the handle, as must the matrices.
 * TQ_ERR_UNSUPPORTED_SHAPE if the matrices do not share table, level type and layout.
 * tq_stack_create synchronises cuda_stream; tq_fused_gemv_stack is asynchronous.  Calls on one
 * stack share its scratch: they must not overlap on the GPU. */
typedef struct tq_stack tq_stack;
int tq_stack_size(const tq_dmat* const* mats, int n_mats, int B, uint64_t* device_bytes);
/* The work split tq_stack_create computes, as a host-only call (no device needed): the row blocks
 * (16 rows) of the matrices, in order, are cut into n_ctas consecutive shares of about equal cost
 * (bytes streamed plus a fixed charge per segment); a share is a list of segments (matrix, first
 * row block, one past the last).  steps[i] = ceil(cols_i / 128), row_blocks[i] = ceil(rows_i / 16),
 * rb_raw[i] = HOST array of row_blocks[i] + 1 prefix counts of raw words per row block.  segs
 * receives 3 values per segment (at most n_mats + n_ctas segments), *n_segs their number,
 * cta_seg[n_ctas + 1] the first segment of each share. */
int tq_stack_plan_host(int n_mats, const uint32_t* steps, const uint32_t* row_blocks,
                       const uint32_t* const* rb_raw, uint32_t n_ctas, uint32_t* segs, uint32_t segs_cap,
                       uint32_t* n_segs, uint32_t* cta_seg);
int tq_stack_create(const tq_dmat* const* mats, const void* const* d_x, float* const* d_y, int n_mats,
                    int B, void* d_buf, uint64_t d_buf_bytes, void* cuda_stream, tq_stack** out);
int tq_fused_gemv_stack(const tq_stack* s, void* cuda_stream);
/* The same call with HOST operands, for a stack whose d_x[i] all lie in one DEVICE arena of x_bytes
 * and whose d_y[i] all lie in one DEVICE arena of y_bytes: copies h_x (the arena's image, HOST) in,
 * runs the stack, copies the y arena out to h_y, all on cuda_stream, without synchronising. */
int tq_fused_gemv_stack_host(const tq_stack* s, const void* h_x, void* d_x_arena, uint64_t x_bytes,
                             float* h_y, const float* d_y_arena, uint64_t y_bytes, void* cuda_stream);
int tq_stack_launches(const tq_stack* s); /* kernel launches one tq_fused_gemv_stack call makes */
/* tq_decompress of every matrix of the stack in one persistent launch.  d_out_ptrs: DEVICE array of
 * n_mats DEVICE pointers, each 16-byte aligned with room for rows_i * cols_i bytes.  A stack made
 * with d_x == d_y == NULL (B ignored) serves this call only. */
int tq_decompress_stack(const tq_stack* s, uint8_t* const* d_out_ptrs, void* cuda_stream);
/* Phase 1 of tq_fused_gemm_ws for every matrix of the stack in one persistent launch.
 * d_workspace_ptrs: DEVICE array of n_mats DEVICE pointers (256-byte aligned, tq_gemm_workspace_size
 * bytes each). */
int tq_decode_bf16_stack(const tq_stack* s, void* const* d_workspace_ptrs, void* cuda_stream);

/* Phase 2 of tq_fused_gemm_ws for several matrices and one token count in ONE persistent launch: the
 * output tiles of all products form one sequence (longest rows first) that the CTAs share, so no SM
 * idles at the end of a small matrix.  Y_i[M][rows_i] = scale_i * (W_i as bf16 in d_workspaces[i]) x
 * X_i[M][cols_i]; the workspaces are the ones tq_decode_bf16 / tq_decode_bf16_stack fill.
 * tq_gemm_plan_create binds the operands (HOST arrays of n_mats DEVICE pointers; alignment as for
 * tq_gemm_bf16_ws), writes the tensor maps and the tile index into d_buf (DEVICE, 256-byte aligned,
 * tq_gemm_plan_size bytes, caller-owned, must outlive the plan) on cuda_stream and synchronises it
 * once; tq_gemm_plan_run launches without synchronising and may be called any number of times while
 * the bound buffers are alive.  Matrices must be TQ_LAYOUT_TILES with cols a multiple of 8
 * (TQ_ERR_UNSUPPORTED_SHAPE otherwise).  tq_gemm_plan_status synchronises cuda_stream and returns the
 * plan's own sticky status word (TQ_STATUS_WAIT_EXPIRED if a bounded wait inside the kernel ran out). */
typedef struct tq_gemm_plan tq_gemm_plan;
int tq_gemm_plan_size(int n_mats, uint64_t* device_bytes);
int tq_gemm_plan_create(const tq_dmat* const* mats, const void* const* d_X_bf16, float* const* d_Y,
                        const void* const* d_workspaces, int n_mats, int M, void* d_buf,
                        uint64_t d_buf_bytes, void* cuda_stream, tq_gemm_plan** out);
int tq_gemm_plan_run(const tq_gemm_plan* plan, void* cuda_stream);
int tq_gemm_plan_status(const tq_gemm_plan* plan, void* cuda_stream, uint32_t* status);
void tq_gemm_plan_free(tq_gemm_plan* plan); /* host handle only */
void tq_stack_free(tq_stack* s);

/* Test hook for the bounded waits inside the kernels (no counterpart in the paper).  While on, the
 * one- and two-vector TQ_LAYOUT_TILES GEMV kernel is launched expecting one chunk of the table that is
 * never copied: every wait for the table runs into its limit (about 2 s), the warps give up, the
 * kernel ends normally with undefined y and TQ_STATUS_WAIT_EXPIRED in the matrix's status word, and
 * the context stays usable.  Nothing faults, traps or waits without bound.  Off by default. */
void tq_test_withhold_table_chunk(int on);

/* Read and clear the matrix's device status word (TQ_STATUS_* bits); synchronises cuda_stream. */
int tq_device_status(const tq_dmat* m, void* cuda_stream, uint32_t* status);

void tq_dmat_free(tq_dmat* m); /* host handle only */

#ifdef __cplusplus
}
#endif
#endif /* TQ_H_ */
