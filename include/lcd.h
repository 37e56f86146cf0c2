/*
 * lcd.h - C ABI of the B200 (sm_100a) LUT-based inference matmul of the LCD paper
 *         ("Inference with Table Lookup", Section 4).
 *
 * A linear layer y = x W^T (W is N x K) whose clustered weights are stored as packed 2-, 3- or 4-bit
 * centroid indices idx[n][k] plus a per-output-row fp16 codebook cb[n][w].  Activations are
 * smoothed per input channel, mapped to 4-bit indices a = q + 8 (q in [-8,7]) with one fp32 scale
 * per token, and every output is formed by table lookup and accumulation:
 *
 *      y[m][n] = s_q[m] * sum_k q[m][k] * cb[n][idx[n][k]]          (fp32)
 *
 * Conventions for every function:
 *   - returns an lcd_status; never aborts, traps or throws;
 *   - "host" / "device" in a parameter comment says where the pointer must point;
 *   - the caller owns every buffer; the library keeps no state except lazily set kernel attributes (per device) and
 *     the built-in scratch array of lcd_lut_linear_static with its per-device address;
 *   - device entry points are stream-ordered on `cuda_stream` (a cudaStream_t passed as void*;
 *     NULL = legacy default stream), do not synchronise and do not allocate;
 *   - argument errors are reported before anything is launched; an asynchronous problem (a bounded
 *     wait inside a kernel that expired) is written to `*status_word_dev` when that pointer is given.
 */
#ifndef LCD_H_
#define LCD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LCD_OK = 0,
  LCD_ERR_INVALID_ARG = 1,      /* null pointer, non-positive size, bad alignment, bad enum          */
  LCD_ERR_UNSUPPORTED = 2,      /* valid request this build has no kernel for                       */
  LCD_ERR_BUFFER_TOO_SMALL = 3, /* an output / workspace / scratch buffer is smaller than required  */
  LCD_ERR_INDEX_RANGE = 4,      /* a weight index >= C                                              */
  LCD_ERR_BAD_BLOB = 5,         /* header magic / version / layout / checksum / size mismatch       */
  LCD_ERR_CUDA = 6,             /* a CUDA runtime call or a launch failed (see lcd_last_cuda_error) */
  LCD_ERR_TIMEOUT = 7           /* value written to the status word when a device-side wait expired */
} lcd_status;

/* Which kernel family lcd_lut_linear uses.  Every family computes the same y. */
typedef enum {
  LCD_ALGO_AUTO = 0,        /* M <= 16: SHARED_BUCKET where it applies and the layer is large enough to pay    */
                            /* for its tables, else REGISTER_LUT; DENSE_TC above (17..32 tokens on rows of at   */
                            /* least 8192 columns: REGISTER_LUT in two launches, measured faster there)         */
  LCD_ALGO_REFERENCE = 1,   /* plain per-weight lookup cb[n][idx] and multiply-accumulate; any M, slow        */
  LCD_ALGO_BUCKET_LUT = 2,  /* Section 4.2 centroid-stationary buckets: per output and per centroid w the exact */
                            /* integer sum S_w of the activation levels whose weight index is w (one-hot byte   */
                            /* tables looked up four weights at a time, accumulated by int8 tensor-core MMAs),   */
                            /* then y = s_q * sum_w cb[w] * S_w: 2^bits multiplies per output.  M <= 16.         */
  LCD_ALGO_REGISTER_LUT = 3,/* Section 4.2 lookup with the row codebook held as byte tables in registers        */
                            /* (16-bit fixed point, high and low byte), four weights looked up per instruction,  */
                            /* accumulated by int8 tensor-core MMAs against the activation levels.  M <= 16.     */
  LCD_ALGO_DENSE_TC = 4,    /* batched prefill on tcgen05 tensor cores: the byte tables of REGISTER_LUT decode   */
                            /* the indices into two int8 planes in shared memory, int8 levels arrive by TMA,     */
                            /* kind::i8 MMAs accumulate exact int32 sums in tensor memory.                      */
  LCD_ALGO_DENSE_F16 = 5,   /* the same with fp16 operands: indices decoded through the codebook into fp16     */
                            /* shared-memory tiles, fp32 accumulators (no fixed-point step; slower).            */
  LCD_ALGO_TC_LUT = 6,      /* REGISTER_LUT's tables and sums, the looked-up bytes written to tensor memory as  */
                            /* the A operand of tcgen05 kind::i8 MMAs over a 16-token tile.  M <= 16.            */
  LCD_ALGO_SHARED_BUCKET = 7/* Section 4.2 centroid-stationary buckets with the tables in shared memory: for    */
                            /* every four columns a table indexed by the byte of their four weight indices      */
                            /* holds the four partial bucket sums of the token's levels, so one load looks four */
                            /* weights up for all centroids; exact integer S_w, y = s_q * sum_w cb[w] * S_w.     */
                            /* One token (M = 1), 2-bit indices, 4-bit levels.                                   */
} lcd_algo;

#define LCD_HEADER_BYTES 64
#define LCD_ACT_BITS 4
#define LCD_MAX_BATCH 8   /* problems per grouped call */

const char* lcd_status_string(lcd_status s);
/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* lcd_last_cuda_error(void);

/* ----------------------------------------------------------------------------------------------
 * Offline: index packing (Section 4.2, last paragraph: fewer than 16 centroids per layer allow a
 * compact low-bit index representation; Section 4.1: everything the lookup needs is fixed ahead of
 * time).  Host functions, bit-exact, no CUDA calls.
 *
 * Blob = 64-byte header | zero padding to 256 | index area | codebook area.
 *   header (little endian): u32 magic 'LCDW', u32 version 1, u64 N, u64 K, u64 K_pad, u32 bits, u32 C,
 *     u32 layout (2), u32 checksum (sum of all bytes after the header, mod 2^32), u64 index_offset (256),
 *     u64 codebook_offset.
 *   index area: rows padded to N_pad = 16*ceil(N/16), columns to K_pad = 256*ceil(K/256) with index 0,
 *     cut into items of 16 rows x 256 columns stored row-group major: item (rp, kt) starts at
 *     index_offset + (rp*(K_pad/256) + kt)*2T and is two tiles of T = 512 (2 bit), 768 (3 bit) or 1024 (4 bit) bytes, rows
 *     16rp..16rp+7 then rows 16rp+8..16rp+15.  Inside a tile, lane l = 4*g + t (g = row 0..7, t = quarter
 *     0..3) owns columns 128*h + 32*t .. +31 of row g for both 128-column k-blocks h = 0,1 of the tile:
 *       2 bit: 16 bytes at tile + 16*l; bytes [8h, 8h+8) belong to k-block h; byte p of those holds the
 *              four columns 128h + 32t + 4p + i (i = 0..3, at bits [2i,2i+2)).
 *       3 bit: three 256-byte planes; plane b has, at plane + 8*l + 4*h, word b of the lane's 12-byte
 *              record of k-block h.  A record packs columns 128h + 32t + m: m = 8i+j (i < 3) at bits
 *              [4j, 4j+3) of word i; m = 24+j has bit b of its index at bit 4j+3 of word b.
 *       4 bit: two 512-byte planes, one per k-block h; plane h has the lane's 16 bytes at plane + 16*l, byte p of
 *              which holds the two columns 128h + 32t + 2p + i (i = 0, 1, at bits [4i, 4i+4)).
 *   codebook area: N_pad rows of 2^bits fp16 values; entries >= C and padding rows are zero.
 * -------------------------------------------------------------------------------------------- */

/* Size in bytes of the blob for an N x K layer.  bits in {2,3,4}.  *bytes is written on LCD_OK. */
lcd_status lcd_packed_weights_bytes(int64_t N, int64_t K, int bits, size_t* bytes);

/* idx: host, uint8 [N][K] row-major (ld = K), every value < C else LCD_ERR_INDEX_RANGE
 *      (bad_n/bad_k, if non-NULL, receive the first offending position);
 * codebook_fp16: host, raw IEEE binary16 bits [N][C]; 1 <= C <= 2^bits;
 * out: host buffer of out_bytes >= lcd_packed_weights_bytes(...), written completely.
 * The caller copies the blob to the device (base address aligned to 256 bytes) and keeps the first
 * 64 bytes on the host: device entry points take both. */
lcd_status lcd_pack_weights(const uint8_t* idx, const uint16_t* codebook_fp16, int64_t N, int64_t K,
                            int bits, int C, void* out, size_t out_bytes, int64_t* bad_n, int64_t* bad_k);

/* Exact inverse.  blob: host.  Any of idx / codebook_fp16 may be NULL to only read the sizes; otherwise
 * idx must hold N*K bytes and codebook_fp16 N*C values.  Verifies magic, version, layout, sizes, checksum. */
lcd_status lcd_unpack_weights(const void* blob, size_t blob_bytes, uint8_t* idx, uint16_t* codebook_fp16,
                              int64_t* N, int64_t* K, int* bits, int* C);

/* ----------------------------------------------------------------------------------------------
 * Online step 1: input transformation (Section 4.1, both equations).  Smoothing and uniform symmetric
 * quantisation are one multiply followed by round-to-nearest(-even) and clip to [-8, 7]:
 *     dynamic (static_scale == NULL), per token:  t_k = x_k * inv_smooth_k ; A = max_k |t_k| ;
 *         A == 0: s_q = 1, q = 0 ; else s_q = A / 7, r = 7 / A, q_k = clip(rint(t_k * r)) ;
 *     static (the paper's literal form, scale fixed offline): inv_smooth_k must already hold
 *         1/(s_k * s_q) and *static_scale = s_q;  q_k = clip(rint(x_k * inv_smooth_k)).
 * All arithmetic is IEEE binary32, one rounding per written operation, so the indices are reproducible
 * bit for bit.
 *   x_fp16:      device, binary16 [M][ldx], ldx >= K;
 *   inv_smooth:  device, fp32 [K], or NULL for all ones;
 *   static_scale device, fp32 scalar, or NULL;
 *   act_bits:    4, or 8 (the paper's own b = 8: the same steps with 127 in place of 7 and the clip range
 *                [-128, 127]);
 *   act_idx:     device out.  act_bits = 4: uint8 [M][K_pad/2], K_pad = 256*ceil(K/256): a = q + 8, column k
 *                even in the low nibble; columns K..K_pad-1 are written as a = 8 (q = 0).
 *                act_bits = 8: [M][K_pad] signed bytes q, columns K..K_pad-1 written as 0; 16-byte aligned;
 *   act_scale:   device out, fp32 [M] (s_q).
 * -------------------------------------------------------------------------------------------- */
lcd_status lcd_smooth_quantize_act(const void* x_fp16, int64_t M, int64_t K, int64_t ldx,
                                   const float* inv_smooth, const float* static_scale, int act_bits,
                                   uint8_t* act_idx, float* act_scale, void* cuda_stream);

/* The same transformation for up to LCD_MAX_BATCH independent activation matrices (the inputs of the
 * projections of one decoder layer) in one launch.  Fields as the arguments of lcd_smooth_quantize_act. */
typedef struct {
  const void* x_fp16;        /* device */
  int64_t M, K, ldx;
  const float* inv_smooth;   /* device or NULL */
  const float* static_scale; /* device or NULL */
  uint8_t* act_idx;          /* device out */
  float* act_scale;          /* device out */
} lcd_act_problem;

/* act_bits: 4 or 8, for all problems of the call (8: every act_idx is [M][K_pad] signed bytes). */
lcd_status lcd_smooth_quantize_act_batch(const lcd_act_problem* problems /* host */, int count, int act_bits,
                                         void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * Online steps 2+3: table lookup and accumulation (Section 4.2).
 *   packed_weights_dev: device, the blob, 256-byte aligned;
 *   header_host:        host, the blob's first 64 bytes;
 *   act_idx, act_scale: device, as written by lcd_smooth_quantize_act for the same K;
 *   y:                  device out, fp32 [M][ldy], ldy >= N;
 *   algo:               LCD_ALGO_AUTO: see lcd_algo; a family asked for
 *                       outside its range => LCD_ERR_UNSUPPORTED;
 *   workspace:          device scratch of at least lcd_lut_linear_workspace_bytes(...) bytes, 256-byte
 *                       aligned (may be NULL when that size is 0).  REGISTER_LUT and BUCKET_LUT keep integer
 *                       partial sums and arrival counters there: the caller zero-fills it once before its
 *                       first use, every call that completes leaves it zero-filled again, and two calls that
 *                       may overlap on the device need separate workspaces.  The other families do not care
 *                       about its contents;
 *   status_word_dev:    device int32 or NULL; receives LCD_ERR_TIMEOUT if a bounded device-side wait
 *                       expired (the output is then invalid and the workspace must be zero-filled again);
 *                       never written otherwise.
 * The M <= 16 kernels are launched with programmatic stream serialization: they begin streaming weights
 * while the previous kernel of the stream finishes and wait for it before reading act_idx / act_scale (x_fp16 in the
 * fused call).  The blob and inv_smooth are read before that wait: they must be complete when the call is enqueued,
 * not produced by work that may still be running on the stream (lcd_smoothing_search's output: synchronise, or put
 * another kernel between).  K_pad >= 2^21 (where the exact int32 sums could overflow) gives LCD_ERR_UNSUPPORTED.
 * -------------------------------------------------------------------------------------------- */
lcd_status lcd_lut_linear_workspace_bytes(const void* header_host, int64_t M, lcd_algo algo, size_t* bytes);

lcd_status lcd_lut_linear(const void* packed_weights_dev, const void* header_host, const uint8_t* act_idx,
                          const float* act_scale, int64_t M, float* y, int64_t ldy, lcd_algo algo,
                          void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                          void* cuda_stream);

/* The same lookup and accumulation for 8-bit activation levels (Section 4.1 with b = 8; Section 4.2's tables then
 * have 129 sign-folded rows, here as there never materialised: the weight is looked up, the level multiplies in
 * the integer MMA).  act_q: device, [M][K_pad] signed bytes as written by lcd_smooth_quantize_act with
 * act_bits = 8, 16-byte aligned.  Everything else, the workspace size and its zero-fill contract included, as
 * lcd_lut_linear; algo may be AUTO, REFERENCE, REGISTER_LUT, BUCKET_LUT, TC_LUT or DENSE_TC (DENSE_F16 and
 * K_pad >= 131072, where the int32 sums could overflow, give LCD_ERR_UNSUPPORTED). */
lcd_status lcd_lut_linear_act8(const void* packed_weights_dev, const void* header_host, const int8_t* act_q,
                               const float* act_scale, int64_t M, float* y, int64_t ldy, lcd_algo algo,
                               void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                               void* cuda_stream);

/* Up to LCD_MAX_BATCH independent problems with M <= 16 (e.g. the q/k/v or gate/up projections of a decoder
 * layer, or all projections of a layer when their inputs are independent) in ONE launch: the SMs are divided
 * among the problems in proportion to their index bytes.  All problems must have the same index width.
 * algo: AUTO, REGISTER_LUT or BUCKET_LUT.  Workspace rules as for lcd_lut_linear. */
typedef struct {
  const void* packed_weights_dev; /* device, 256-byte aligned */
  const void* header_host;        /* host */
  const uint8_t* act_idx;         /* device */
  const float* act_scale;         /* device */
  int64_t M;
  float* y;                       /* device out, fp32 [M][ldy] */
  int64_t ldy;
} lcd_linear_problem;

lcd_status lcd_lut_linear_batch_workspace_bytes(const lcd_linear_problem* problems /* host */, int count,
                                                lcd_algo algo, size_t* bytes);

lcd_status lcd_lut_linear_batch(const lcd_linear_problem* problems /* host */, int count, lcd_algo algo,
                                void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                void* cuda_stream);

/* Which family a grouped call with these shapes and this `algo` runs (what LCD_ALGO_AUTO stands for): only the
 * header_host and M fields of the problems are read.  The fused call (lcd_linear_fused_batch) chooses the same way. */
lcd_status lcd_lut_linear_batch_resolve(const lcd_linear_problem* problems /* host */, int count, lcd_algo algo,
                                        lcd_algo* resolved);

/* lcd_lut_linear_batch for 8-bit levels: every problem's act_idx points at [M][K_pad] signed bytes (see
 * lcd_lut_linear_act8); workspace size from lcd_lut_linear_batch_workspace_bytes. */
lcd_status lcd_lut_linear_batch_act8(const lcd_linear_problem* problems /* host */, int count, lcd_algo algo,
                                void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * Offline: adaptive smoothing search (Section 3.4).  For each of n_alphas candidate migration strengths alpha:
 *     s_k = xmax_k^alpha / wmax_k^(1-alpha), xmax_k = max over the calibration batch of |x_tk|, clamped to
 *           [1e-5, 1e5], s_k = 1 where either maximum is zero (binary64 powers, rounded once to binary32);
 *     mse  = mean over the batch of (x - Q_INT8(x / s) * s)^2, Q_INT8 = the per-token 8-bit quantiser of
 *           lcd_smooth_quantize_act (act_bits = 8, dynamic scale) applied with inv_smooth = 1/s.
 * The first candidate with the smallest mse is chosen.
 *   x_fp16:      device, binary16 [T][ldx], the calibration activations of one layer;
 *   wmax:        device, fp32 [K]: max over output rows of |W[n][k]| of that layer;
 *   alphas_host: host, fp32 [n_alphas], 1 <= n_alphas <= 64;
 *   workspace:   device, lcd_smoothing_search_workspace_bytes(...) bytes, 256-byte aligned, contents ignored;
 *   mse:         device out, fp64 [n_alphas];   best: device out int32 (index) or NULL;
 *   inv_smooth:  device out fp32 [K] = 1/s_k of the chosen candidate, ready for the online calls, or NULL.
 * Sums run in a fixed order: results are reproducible from run to run.
 * -------------------------------------------------------------------------------------------- */
lcd_status lcd_smoothing_search_workspace_bytes(int64_t T, int64_t K, int n_alphas, size_t* bytes);

lcd_status lcd_smoothing_search(const void* x_fp16, int64_t T, int64_t K, int64_t ldx, const float* wmax,
                                const float* alphas_host, int n_alphas, void* workspace, size_t workspace_bytes,
                                double* mse, int32_t* best, float* inv_smooth, void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * Offline: density-based centroid initialisation (DBCI, the six steps of Section 3.1) on a flat array of weights.
 *   1. sort;  2. sigma = (the 68.27 / 95.44 / 99.74 % nearest-rank percentiles of the positive weights and of the
 *   magnitudes of the negative weights, summed) / 12;  3. the smallest and the largest weight seed two clusters
 *   that take every weight within sigma of them (the right one gives way where they overlap);  4. MinPts = the
 *   smaller of the two counts, eps = sigma / MinPts;  5. DBSCAN on the remaining weights alone: a weight with at
 *   least MinPts weights (itself included) within eps is a core point, core points within eps of each other chain
 *   into one cluster, another weight within eps of a core point joins the cluster of its nearest core point (the
 *   left one on a tie), the rest is noise;  6. the centroid of a cluster is its lower median.
 * Comparisons and scalar operations are binary64 on the binary32 data.
 *   weights:   device, fp32 [n], 1 <= n < 2^31;     workspace: device, lcd_dbci_workspace_bytes(n, max_centroids)
 *              bytes, 256-byte aligned, contents ignored;
 *   centroids: device out, fp32 [max_centroids], ascending; if more clusters exist than fit
 *              (result->n_clusters_found > max_centroids + 2 or n_centroids > max_centroids) the list is cut;
 *   labels:    device out int32 [n] or NULL: cluster of every weight IN SORTED ORDER (0 = left seed cluster,
 *              1.. = DBSCAN clusters from left to right, last = right seed cluster, -1 = noise);
 *   sorted:    device out fp32 [n] or NULL: the sorted weights;     result: device out.
 * -------------------------------------------------------------------------------------------- */
typedef struct {
  double sigma, eps;
  int64_t min_pts, left, right;        /* members of the two seed clusters */
  int32_t n_centroids, n_noise, n_clusters_found;
} lcd_dbci_result;

lcd_status lcd_dbci_workspace_bytes(int64_t n, int max_centroids, size_t* bytes);

lcd_status lcd_dbci(const float* weights, int64_t n, void* workspace, size_t workspace_bytes, float* centroids,
                    int max_centroids, int32_t* labels, float* sorted, lcd_dbci_result* result, void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * Offline: reclassification of weights and centroid offsets after a round of weight updates (Section 3.2, the
 * half-gap equation and the centroid-update equation), for per-row codebooks sorted in ascending order (the
 * caller's duty; unsorted rows give meaningless moves).  A weight of cluster i with update dw moves to i - 1 when
 * dw < -(C_i - C_{i-1})/2 and to i + 1 when dw > (C_{i+1} - C_i)/2 (binary32, one subtraction and one halving;
 * the paper prints the left test without the sign; edge clusters have one side); never further than one cluster.
 *     delta_c[n][j] = sum over the weights that end up in j of (dw + (C_old - C_j))      (a sum, as printed)
 *   idx:           device, uint8 [N][K] cluster of every weight (one byte each, the packer's input form), < C
 *                  (not checked on the device: a byte >= C is reduced modulo 4, 8 or 16, whichever holds C, kept as
 *                  that value in new_idx and counted in no cluster; nothing faults);  K <= 2^25;
 *   codebook_fp16: device, binary16 [N][C], 1 <= C <= 16;     delta_w: device, fp32 [N][ldw], ldw >= K;
 *   new_idx:       device out, uint8 [N][K] (may not alias idx);
 *   delta_c:       device out, fp64 [N][C];     counts: device out, int32 [N][C] members after the move.
 * Sums run in a fixed order: results are reproducible from run to run.
 * -------------------------------------------------------------------------------------------- */
lcd_status lcd_reclassify(const uint8_t* idx, const uint16_t* codebook_fp16, const float* delta_w, int64_t N, int64_t K,
                          int64_t ldw, int C, uint8_t* new_idx, double* delta_c, int32_t* counts, void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * Online steps 1+2+3 in one call for up to LCD_MAX_BATCH independent problems; with M <= 16 (the projections
 * of one decoder layer at decode time): the lookup kernel performs the input transformation of Section 4.1
 * itself (dynamic per-token scale, 4-bit levels, the operation sequence of lcd_smooth_quantize_act, so the
 * levels and therefore y are bit-identical to the two-call path) while its first weights are already streaming,
 * and never writes the levels or scales to memory.
 *   x_fp16:     device, binary16 [M][ldx], ldx >= K of the blob;
 *   inv_smooth: device fp32 [K] or NULL;
 *   algo:       LCD_ALGO_AUTO, REGISTER_LUT or BUCKET_LUT;
 *   workspace:  as lcd_lut_linear_batch (same size: lcd_linear_fused_batch_workspace_bytes; zero-filled
 *               before first use, left zero-filled).
 * Many tokens (prefill): when EVERY problem has more than 16 tokens, algo is
 * LCD_ALGO_AUTO or LCD_ALGO_DENSE_TC and the call is: one launch that transforms the inputs of all problems (same
 * operation sequence, same levels) and writes them as the signed bytes the int8 tensor-core kernel reads, in its
 * order, into the workspace (per problem M * K_pad bytes and M scales; no zero-fill contract, the contents are
 * scratch), then that kernel once per problem: no packed 4-bit copy and no expansion pass in between.  y equals
 * the two-call result of LCD_ALGO_DENSE_TC bit for bit.  A mix of problems with at most 16 and more than 16 tokens
 * gives LCD_ERR_UNSUPPORTED (use the two calls).
 * -------------------------------------------------------------------------------------------- */
typedef struct {
  const void* packed_weights_dev; /* device, 256-byte aligned */
  const void* header_host;        /* host, the blob's first 64 bytes */
  const void* x_fp16;             /* device */
  int64_t M, ldx;
  const float* inv_smooth;        /* device or NULL */
  float* y;                       /* device out, fp32 [M][ldy] */
  int64_t ldy;
} lcd_fused_problem;

lcd_status lcd_linear_fused_batch_workspace_bytes(const lcd_fused_problem* problems /* host */, int count,
                                                  lcd_algo algo, size_t* bytes);

lcd_status lcd_linear_fused_batch(const lcd_fused_problem* problems /* host */, int count, lcd_algo algo,
                                  void* workspace, size_t workspace_bytes, int32_t* status_word_dev,
                                  void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * lcd_lut_linear for M <= 16 without a caller-provided workspace.  (No counterpart in the paper: this is a
 * convenience of the library.)
 *
 * Who needs it: code that is not in a position to allocate device memory when it wants to run a layer.  A
 * plug-in running inside a host application that owns the GPU's memory pool, a serving loop that promised
 * its scheduler never to call cudaMalloc after start-up (the call synchronises the whole device and can fail
 * when memory is fragmented), or a component that only ever sees buffers handed to it, cannot obtain the
 * zero-filled workspace lcd_lut_linear asks for.  Here the integer partial sums and arrival counters live in a
 * fixed array of LCD_STATIC_SCRATCH_BYTES that is part of the library's device image: every GPU on which the
 * library is loaded holds that much memory until the process ends, and nothing is allocated or freed by this
 * call (no cudaMalloc / cudaFree, no allocating library routine).
 *
 * Arguments as lcd_lut_linear (inputs and outputs are still the caller's); algo is AUTO, REGISTER_LUT or
 * BUCKET_LUT.  A layer whose scratch need (lcd_lut_linear_workspace_bytes) exceeds LCD_STATIC_SCRATCH_BYTES
 * is refused with LCD_ERR_BUFFER_TOO_SMALL before anything is enqueued; M > 16 gives LCD_ERR_UNSUPPORTED.
 * The first call on each device looks up the array's device address (with that device current) and keeps
 * it; make that first call outside any stream capture.  Every call uses the same array and finds what the
 * previous call left in it, so each call first clears the part it needs (a memset enqueued on cuda_stream).
 * Two calls that can overlap on the GPU - different streams, or different host threads on different streams -
 * race on the array and give wrong results: serialise them, or use lcd_lut_linear with separate workspaces.
 * -------------------------------------------------------------------------------------------- */
#define LCD_STATIC_SCRATCH_BYTES (4u << 20)

lcd_status lcd_lut_linear_static(const void* packed_weights_dev, const void* header_host, const uint8_t* act_idx,
                                 const float* act_scale, int64_t M, float* y, int64_t ldy, lcd_algo algo,
                                 int32_t* status_word_dev, void* cuda_stream);

/* ----------------------------------------------------------------------------------------------
 * The whole online path (Section 4: input transformation -> bucket table lookup -> accumulation) from
 * HOST activations to HOST outputs, for callers that keep activations on the host: copies x to the
 * device, runs lcd_smooth_quantize_act (dynamic mode) and lcd_lut_linear (LCD_ALGO_AUTO), copies y back.
 * All copies and kernels are enqueued on cuda_stream; the call returns without synchronising, y_host is
 * valid after the stream is synchronised.  x_host / y_host should be pinned for the copies to be async.
 *   x_host_fp16: host, binary16 [M][K] dense;   y_host: host out, fp32 [M][N] dense;
 *   inv_smooth:  device fp32 [K] or NULL;
 *   scratch:     device, >= lcd_linear_host_scratch_bytes(...) bytes, 256-byte aligned.  The caller zero-fills it
 *                once before its first use (the lookup kernels keep partial sums and counters in part of it and
 *                leave that part zero-filled, see lcd_lut_linear); it must be zero-filled again after a reported
 *                LCD_ERR_TIMEOUT.  Two calls that may overlap on the device need separate scratch buffers;
 *   status_word_dev: device int32 or NULL, as for lcd_lut_linear.
 * -------------------------------------------------------------------------------------------- */
lcd_status lcd_linear_host_scratch_bytes(const void* header_host, int64_t M, size_t* bytes);

lcd_status lcd_linear_host(const void* packed_weights_dev, const void* header_host, const void* x_host_fp16,
                           int64_t M, const float* inv_smooth, float* y_host, void* scratch,
                           size_t scratch_bytes, int32_t* status_word_dev, void* cuda_stream);

/* The same for up to LCD_MAX_BATCH independent problems with M <= 16 and equal index width (the projections of
 * a decoder layer): ONE host-to-device copy of all inputs, one grouped quantise launch, one grouped lookup
 * launch (a single launch that does both when every problem has one token), ONE device-to-host copy of all
 * outputs (none when the outputs total at most 512 KB and y_host_all is pinned memory the device can address: the
 * kernels then store y into it directly).  The host staging buffers are laid out by the library:
 * problem i's x (fp16 [M][K], dense) starts at the sum of the earlier problems' M*K*2 bytes rounded up to 16,
 * its y (fp32 [M][N], dense) at the sum of the earlier problems' M*N*4 bytes rounded up to 16;
 * lcd_linear_host_batch_sizes returns the total sizes (any of the three outputs may be NULL).  x_host_all and
 * y_host_all should be pinned; y_host_all is valid once cuda_stream is synchronised.  scratch and status_word_dev as
 * for lcd_linear_host (zero-filled once by the caller, left usable by every call). */
typedef struct {
  const void* packed_weights_dev; /* device, 256-byte aligned */
  const void* header_host;        /* host */
  const float* inv_smooth;        /* device fp32 [K] or NULL */
  int64_t M;
} lcd_host_problem;

lcd_status lcd_linear_host_batch_sizes(const lcd_host_problem* problems /* host */, int count, size_t* x_host_bytes,
                                       size_t* y_host_bytes, size_t* scratch_bytes);

lcd_status lcd_linear_host_batch(const lcd_host_problem* problems /* host */, int count, const void* x_host_all,
                                 void* y_host_all, void* scratch, size_t scratch_bytes, int32_t* status_word_dev,
                                 void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LCD_H_ */
