/*
 * snip.h -- C ABI of the B200 (sm_100a) library for SNIP's layerwise mixed-precision linear
 * layer: per-block-scaled BF16 -> FP8 E4M3 / FP4 E2M1 quantizers with fused error-norm
 * statistics, and the forward / input-gradient / weight-gradient GEMMs on the tcgen05 tensor
 * cores with FP32 accumulation.
 *
 * Conventions
 *   - Every function returns a snip_status_t (0 = SNIP_OK).  Nothing throws, nothing allocates
 *     device memory, nothing synchronizes the host: all device work is enqueued on the caller's
 *     stream.  (The host-only solver snip_select_scheme uses ordinary host heap memory.)
 *   - The caller owns every buffer.  Pointers are DEVICE pointers unless the name ends in
 *     `_host`.  Device pointers must be 16-byte aligned.  Outputs are fully overwritten.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Matrices are row-major.  M = tokens, K = in-features, N = out-features;
 *     X[M,K], W[N,K], Y[M,N], dY[M,N], dX[M,K], dW[N,K]  (paper Sec. 4.2, 4.3).
 *   - All matrix dimensions must be positive multiples of 64 (SNIP_ERR_SHAPE otherwise); a
 *     dimension that is not a multiple of 128 ends in one 64-wide tile.
 *   - bf16 data is passed as raw 16-bit words (void* / uint16_t*).
 *   - Errors: SNIP_ERR_ARG (null pointer, bad enum), SNIP_ERR_SHAPE, SNIP_ERR_ALIGN,
 *     SNIP_ERR_UNSUPPORTED (precision pair, layout, or a device that is not sm_100),
 *     SNIP_ERR_WORKSPACE (workspace too small), SNIP_ERR_CUDA (a CUDA call failed; see
 *     snip_last_cuda_error), SNIP_ERR_TIMEOUT (a device-side bounded wait ran out; reported by
 *     snip_poll_status).  On any error before launch nothing is enqueued.
 */
#ifndef SNIP_H_
#define SNIP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SNIP_OK = 0,
    SNIP_ERR_ARG = 1,
    SNIP_ERR_SHAPE = 2,
    SNIP_ERR_ALIGN = 3,
    SNIP_ERR_UNSUPPORTED = 4,
    SNIP_ERR_WORKSPACE = 5,
    SNIP_ERR_CUDA = 6,
    SNIP_ERR_TIMEOUT = 7
} snip_status_t;

/* Element formats (paper Sec. 2.3 "Quantization Format"): BF16 is the unquantized baseline,
 * FP8 is E4M3 (max 448), FP4 is E2M1 of the MX specification (max 6). */
typedef enum { SNIP_FMT_BF16 = 0, SNIP_FMT_FP8_E4M3 = 1, SNIP_FMT_FP4_E2M1 = 2 } snip_fmt_t;

/* Scaling granularity (paper Sec. 2.3 "Quantization granularity"): 1x128 tiles for activations
 * and gradients, 128x128 blocks for weights.  A 1x128 tile runs along the contraction dimension
 * of the GEMM that consumes the operand: ROW = along the contiguous (column) index,
 * COL = along the row index (128 consecutive rows of one column). */
typedef enum {
    SNIP_BLOCK_ROW_1x128 = 0, SNIP_BLOCK_COL_128x1 = 1, SNIP_BLOCK_BLK_128x128 = 2,
    /* 32-long tiles, power-of-two scales only (snip_quantize_mx, snip_quantize_dual with pow2_scale): an added option */
    SNIP_BLOCK_ROW_1x32 = 3, SNIP_BLOCK_COL_32x1 = 4,
    /* 16-long tiles of the two-level option (snip_quantize_nvfp4_dual, snip_gemm_nvfp4): an added option */
    SNIP_BLOCK_ROW_1x16 = 5, SNIP_BLOCK_COL_16x1 = 6
} snip_block_t;

/* Output element type of a GEMM.  BF16 is the paper's choice (Sec. 2.2 keeps GEMM outputs in
 * BF16 while the operands are FPX); FP32 exposes the accumulator for parity checks and for
 * weight-gradient accumulation. */
typedef enum { SNIP_OUT_BF16 = 0, SNIP_OUT_FP32 = 1 } snip_out_t;

typedef enum { SNIP_OP_FWD = 0, SNIP_OP_DGRAD = 1, SNIP_OP_WGRAD = 2 } snip_op_t;

/* snip_quantize flags */
#define SNIP_Q_TRANSPOSED 0x1u /* store the codes as the transpose: element (r,c) at [c][r]   */
#define SNIP_Q_STATS      0x2u /* write *stats (needs a workspace)                            */
#define SNIP_Q_NO_CODES   0x4u /* statistics only: codes and scales are not written           */

/* Error-norm statistics of one tensor (paper Sec. 3.1, Step 1: Frobenius norm of a tensor and
 * of its quantization error; Sec. 4.1: error = x - q(x)).  Lives in device memory.
 * Norms are the square roots of the two sums. */
typedef struct {
    double sumsq_x;   /* sum of x^2                                  */
    double sumsq_err; /* sum of (x - dequant(quant(x)))^2            */
    float amax;       /* max |x| over the whole tensor               */
    uint32_t reserved;
} snip_stats_t;

/* A quantized matrix, described to the GEMM.  No ownership is taken.
 *   rows, cols : logical shape of the matrix that was quantized
 *   codes      : FP8: one byte per element; FP4: two per byte, even index of the contiguous
 *                dimension in bits [3:0], odd in [7:4]; BF16: the original bf16 words.
 *                Stored [rows][cols] or, if `transposed`, [cols][rows].
 *   scales     : FP32 scale S = FPX_MAX / amax of each tile (paper Sec. 2.3), NULL for BF16:
 *                ROW  [ceil(cols/128)][rows],  COL  [ceil(rows/128)][cols],
 *                BLK  [ceil(rows/128)][ceil(cols/128)].
 */
typedef struct {
    const void *codes;
    const float *scales;
    int64_t rows, cols;
    int32_t fmt;        /* snip_fmt_t   */
    int32_t block;      /* snip_block_t */
    int32_t transposed; /* 0 or 1       */
    int32_t reserved;
} snip_qtensor_t;

/* Tensors of one linear layer for snip_layer_stats; any pointer may be NULL (skipped). */
typedef struct {
    const void *X, *W, *Y, *dY, *dX, *dW; /* bf16, shapes as in the header comment */
    int64_t M, N, K;
} snip_layer_tensors_t;

/* Result of snip_layer_stats (device memory).  Indices: tensor 0..5 = X, W, Y, dY, dX, dW.
 * sumsq_err[t][f][b]: t in {0:X, 1:W, 2:dY}, f in {0:FP8, 1:FP4}, b = snip_block_t.  Filled for
 * the tile kinds the tensor is consumed with (X, dY: ROW and COL; W: BLK); others are 0. */
typedef struct {
    double sumsq[6];
    double sumsq_err[3][2][3];
} snip_layer_stats_t;

/* Rounding of the codes: nearest-even (Sec. 2.3) or stochastic (Sec. 6.1, FP4 output gradients). */
typedef enum { SNIP_ROUND_NEAREST_EVEN = 0, SNIP_ROUND_STOCHASTIC = 1 } snip_rounding_t;

/* One output of snip_quantize_dual: format (FP8 or FP4), destination buffers (device), optional UE8M0
 * scale-factor atoms (power-of-two rule only, else NULL) and optional statistics (device; give both
 * outputs' or neither). */
typedef struct {
    int32_t fmt;
    int32_t rounding; /* snip_rounding_t; stochastic needs fmt = FP4 and row / column tiles */
    void *codes;
    float *scales;
    void *sf;
    snip_stats_t *stats;
    uint64_t seed;    /* stochastic rounding: key of the generator */
} snip_qout_t;

/* Tile kinds of the two outputs of snip_quantize_dual. */
typedef enum {
    SNIP_DUAL_ROW_COLT = 0, /* as stored: 1x128 tiles along the columns; transposed: 128x1 tiles along the rows */
    SNIP_DUAL_BLK_BLKT = 1, /* 128x128 blocks, as stored and transposed */
    SNIP_DUAL_ROW32_COL32T = 2 /* 1x32 tiles as stored, 32x1 tiles transposed; power-of-two scales only */
} snip_dual_kind_t;

/* ---- library information ----------------------------------------------------------------- */

/* Version of this ABI as major*10000 + minor*100 + patch.  (No counterpart in the paper.) */
int snip_version(void);
/* Static, NUL-terminated name of a status code.  (No counterpart in the paper.) */
const char *snip_status_string(int status);
/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char *snip_last_cuda_error(void);

/* ---- quantizer (paper Sec. 2.3: scale = FPX_MAX / max|x|, y = Op(Quant(x*scale))/scale) ---- */

/*
 * Byte sizes of the outputs and of the workspace that snip_quantize needs for a rows x cols
 * input.  Host-only.  Any of the three output pointers may be NULL.
 * codes_bytes: rows*cols (FP8), rows*cols/2 (FP4; plus 64 bytes of tail slack when a dimension is
 * not a multiple of 128: the GEMM may read, and ignores, up to 32 bytes past the last code), 0
 * (BF16 or NO_CODES).
 * scales_bytes: 4 * number of tiles (0 for BF16 or NO_CODES).
 * ws_bytes: 0 unless SNIP_Q_STATS is set or row_stats will be requested (the value returned
 * covers both).
 */
int snip_quantize_sizes(int64_t rows, int64_t cols, int fmt, int block, uint32_t flags,
                        size_t *codes_bytes_host, size_t *scales_bytes_host, size_t *ws_bytes_host);

/*
 * Quantize a row-major bf16 matrix x[rows][ld] (ld >= cols, in elements, multiple of 8).
 * Per tile: amax = max|x|; S = FPX_MAX/amax as an IEEE binary32 quotient (S = 1 for an all-zero
 * tile, clamped to FLT_MAX on overflow); code = round-to-nearest-even, saturating, of the
 * binary32 product x*S.  Codes and scales are written in the layouts of snip_qtensor_t
 * (codes transposed if SNIP_Q_TRANSPOSED).  With SNIP_Q_STATS the two sums and the global amax
 * go to *stats in the same pass; with row_stats != NULL, row_stats[2*r] and [2*r+1] receive the
 * per-row sums (paper Sec. 6.2: the row-wise form keeps one value per row).
 * fmt = BF16 is the identity: nothing is encoded, the error sum is 0; only statistics are
 * produced.  ws / ws_bytes: scratch of at least the size snip_quantize_sizes reports (may be
 * NULL / 0 when that size is 0); its contents are undefined afterwards.
 * Inputs must be finite.  One statistics kernel follows the main kernel on the same stream.
 */
int snip_quantize(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block,
                  uint32_t flags, void *codes, float *scales, snip_stats_t *stats,
                  double *row_stats, void *ws, size_t ws_bytes, void *stream);

/*
 * snip_quantize for callers that cannot hand the library any scratch memory.  (The paper has no
 * counterpart; this is a deployment convenience.)  Meant for hosts that run under a fixed memory
 * budget they do not control, or whose steady-state loop must never call the CUDA allocator: the
 * statistics scratch is a 512 KiB array built into the library's device image, so this entry
 * point allocates nothing, on the host or on the device.  Price: every GPU that loads the library
 * holds those 512 KiB until the process exits.
 *   - Same arguments and results as snip_quantize, minus row_stats / ws / ws_bytes (per-row sums
 *     are not offered here).  Inputs up to 16384 tiles of 128x128 (e.g. 16384 x 16384 elements);
 *     larger ones return SNIP_ERR_WORKSPACE and snip_last_cuda_error() says how much was needed.
 *   - The first call on each device looks up the array's device address (one runtime query, no
 *     allocation).  Make that first call outside any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing in it needs
 *     clearing (each call overwrites what it later reads), but two calls that may run on the GPU at
 *     the same time (different streams, no dependency) race on it: serialize them.
 */
int snip_quantize_noalloc(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block,
                          uint32_t flags, void *codes, float *scales, snip_stats_t *stats, void *stream);

/*
 * Both quantized copies of a tensor from one read.  Every tensor of a linear layer is consumed by
 * two GEMMs with different contraction indices (paper Fig. 5): X by fwd (tiles along K) and wgrad
 * (tiles along M), dY by dgrad (along N) and wgrad (along M), W by fwd and dgrad (the 128x128 block
 * grid serves both, but dgrad wants the transposed storage).  This call produces, from a single pass
 * over x[rows][ld], exactly what two snip_quantize calls would:
 *   as_stored:  kind ROW_COLT -> (fmt, SNIP_BLOCK_ROW_1x128, no flags); BLK_BLKT -> (fmt, SNIP_BLOCK_BLK_128x128, no flags)
 *   transposed: kind ROW_COLT -> (fmt, SNIP_BLOCK_COL_128x1, SNIP_Q_TRANSPOSED); BLK_BLKT -> (fmt, BLK, SNIP_Q_TRANSPOSED)
 * with independent formats, so codes, scales and statistics are bit-identical to those calls.
 * pow2_scale != 0 selects the power-of-two rule of snip_quantize_mx (and allows sf != NULL).
 * kind ROW32_COL32T (needs pow2_scale != 0): as_stored = (fmt, SNIP_BLOCK_ROW_1x32), transposed =
 * (fmt, SNIP_BLOCK_COL_32x1, SNIP_Q_TRANSPOSED), the block-32 form of snip_quantize_mx; FP4 outputs of
 * this kind may be rounded stochastically like those of kind ROW_COLT.
 * Algorithmic bytes per element: 2 + the two outputs' code and scale bytes, instead of 4 + those.
 * The paper does not prescribe how the copies are produced; it only fixes what they contain (Sec. 2.3).
 * ws_bytes >= snip_quantize_dual_workspace() when statistics are requested (else ws may be NULL).
 */
int snip_quantize_dual_workspace(int64_t rows, int64_t cols, size_t *ws_bytes_host);
int snip_quantize_dual(const void *x, int64_t rows, int64_t cols, int64_t ld, int kind, int pow2_scale,
                       const snip_qout_t *as_stored_host, const snip_qout_t *transposed_host,
                       void *ws, size_t ws_bytes, void *stream);

/*
 * Stochastic rounding for FP4 E2M1 codes (paper Sec. 6.1: FP4 output gradients are rounded
 * probabilistically to one of the two nearest representable values so that small gradients do not
 * vanish systematically).  Same tiles, scales, layouts and statistics as snip_quantize with
 * fmt = FP4; only the rounding of the binary32 product t = x*S differs.  The paper cites the method
 * without fixing a rule or a generator; this library's rule: with a = min(|t|, 6) and lo <= a < hi
 * the neighbouring representable magnitudes, the code is hi iff (a - lo)/(hi - lo) > (u + 1/2)/2^16,
 * else lo, sign copied from t; u is the element's 16-bit uniform: Philox4x32 with 10 rounds, counter
 * = (idx/8 as two 32-bit words, 0, 0) with idx = r*cols + c (position in x, whatever the storage of
 * the codes), key = the two words of `seed`; element idx uses bits [16*(idx%2), +16) of output word
 * (idx%8)/2.  The result is a pure function of (x, seed): reruns are bit-identical.
 * block: SNIP_BLOCK_ROW_1x128 (flags without SNIP_Q_TRANSPOSED) or SNIP_BLOCK_COL_128x1 (with it),
 * the two forms an output gradient is consumed in; SNIP_Q_STATS as in snip_quantize (sumsq_err is the
 * squared distance to the stochastic values).  pow2_scale / sf as in snip_quantize_mx.
 */
int snip_quantize_sr(const void *x, int64_t rows, int64_t cols, int64_t ld, int block, uint32_t flags,
                     uint64_t seed, int pow2_scale, void *codes, float *scales, void *sf,
                     snip_stats_t *stats, void *ws, size_t ws_bytes, void *stream);

/*
 * Power-of-two scale option (an added quantization option in the sense of paper Sec. 3.2, which lets
 * new quantization methods join the per-layer choices; power-of-two block scales are those of the MX
 * formats cited in Sec. 2.3).  Identical to snip_quantize except for the scale rule:
 * S = 2^e with the largest e such that amax * 2^e <= FPX_MAX (e clamped to [-126, 127], S = 1 for an
 * all-zero tile), so x*S is exact and 1/S is an 8-bit exponent the tensor core can apply itself.
 * `scales` receives S as FP32 in the usual layout (so the results also feed snip_gemm_quantized).
 * `sf` (may be NULL) receives the UE8M0 bytes of 1/S (byte = 127 - e) as 512-byte atoms, one per
 * 128x128 tile, atom index [operand row tile][contraction chunk] for the orientation the GEMM
 * consumes (ROW: as stored; COL: transposed storage required; BLK: follows SNIP_Q_TRANSPOSED);
 * inside an atom the byte of tile line r is stored four times at (r % 32) * 16 + (r / 32) * 4.
 * snip_quantize_mx_sizes gives the byte size of sf.  Per-row statistics are not offered here.
 * Block-32 form (the tile length of the microscaling formats): block = SNIP_BLOCK_ROW_1x32 (as stored) or
 * SNIP_BLOCK_COL_32x1 (with SNIP_Q_TRANSPOSED) gives every 32-long piece of a 128-long tile its own scale by
 * the same rule.  `scales` is then [ceil(cols/32)][rows] resp. [ceil(rows/32)][cols] (snip_quantize_sizes
 * knows these kinds), and the four bytes of a tile line in its atom are those of its four pieces in order
 * instead of one byte four times; snip_gemm_mx consumes such atoms unchanged (the tensor core applies one
 * byte per 32 elements either way).  Only snip_gemm_mx can multiply these operands.
 */
int snip_quantize_mx_sizes(int64_t rows, int64_t cols, size_t *sf_bytes_host);
int snip_quantize_mx(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block,
                     uint32_t flags, void *codes, float *scales, void *sf, snip_stats_t *stats,
                     void *ws, size_t ws_bytes, void *stream);

/* ---- GEMMs (paper Fig. 5; Sec. 2.2: GEMM in FPX, output in BF16) -------------------------- */

/*
 * Workspace bytes for one GEMM call of the given op and shape, and for the snip_linear_* call
 * of the same op (which also holds the quantized operands).  Host-only.  For SNIP_OP_WGRAD over
 * quantized operands gemm_bytes includes room (about 21 MB) that lets the kernel cut the tiles of
 * its last, partly filled wave over the SMs into slices of the contraction (their FP32 sums are
 * added in slice order, so results do not depend on timing); any GEMM also runs, unsliced, with
 * the 256-byte minimum.
 */
int snip_workspace_size(int op, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b,
                        size_t *gemm_bytes_host, size_t *linear_bytes_host);

/*
 * GEMM over already-quantized operands (lets W be quantized once per optimizer step).
 *   FWD   : out[M,N] = A.B^T, A = X  (ROW tiles, codes [M,K]),            B = W (BLK, [N,K])
 *   DGRAD : out[M,K] = A.B^T, A = dY (ROW tiles, codes [M,N]),            B = W (BLK, codes
 *           stored transposed, i.e. [K,N])
 *   WGRAD : out[N,K] = A.B^T, A = dY (COL tiles, codes transposed [N,M]), B = X (COL tiles,
 *           codes transposed [K,M])
 * i.e. both operands always have the contraction index contiguous.  Each 128-long chunk of the
 * contraction is multiplied on the tensor cores (FP32 accumulation), then scaled by
 * 1/(S_a*S_b) of that chunk in FP32 and added to an FP32 accumulator (Sec. 2.3 removes the scale
 * after the low-precision operator by dividing by it); the result is rounded to nearest-even
 * to bf16 or stored as FP32.  accumulate != 0 adds to the existing contents of out (FP32 output
 * only).  Operand formats: (BF16,BF16), (FP8,FP8), (FP4,FP4), (FP8,FP4), (FP4,FP8); pairs
 * that mix BF16 with a quantized operand return SNIP_ERR_UNSUPPORTED.
 * ws must hold at least 256 bytes (gemm_bytes of snip_workspace_size to allow slicing, see there);
 * its first word is the device status word read by snip_poll_status.  The call itself zeroes that word on the stream before the
 * kernel starts (a 4-byte memset node), so the workspace needs no initialisation by the caller.
 */
int snip_gemm_quantized(int op, const snip_qtensor_t *a_host, const snip_qtensor_t *b_host,
                        void *out, int out_dtype, int accumulate, void *ws, size_t ws_bytes,
                        void *stream);

/*
 * GEMM for the power-of-two scale option: same three products and operand layouts as
 * snip_gemm_quantized, over operands produced by snip_quantize_mx; sf_a / sf_b are their UE8M0
 * atoms.  The tensor core applies 2^-e per 128-long chunk itself (block-scaled MMA), so the whole
 * contraction accumulates in FP32 tensor memory with no per-chunk promotion.  Operand formats: FP8
 * and FP4 in any combination (no BF16).  ws: at least 256 bytes, first word = device status word.
 * (An added option: the paper's rule stays snip_gemm_quantized.)
 */
int snip_gemm_mx(int op, const snip_qtensor_t *a_host, const void *sf_a, const snip_qtensor_t *b_host,
                 const void *sf_b, void *out, int out_dtype, void *ws, size_t ws_bytes, void *stream);

/*
 * Two-level block scaling in the style of NVFP4 (an added option in the sense of paper Sec. 3.2; the paper
 * does not define it, the rule below is this library's): E2M1 codes in tiles of 16 along the contraction of
 * the consuming GEMM, one E4M3 scale byte per tile (used unsigned), one binary32 factor per tensor.
 *   enc  = 2688 / bound (binary32 quotient; 2688 = 448 * 6; enc = 1 if bound == 0), bound = *tensor_amax,
 *          a device value >= 0: the tensor's maximum magnitude, or an estimate of it (e.g. the amax that an
 *          earlier call left in a snip_stats_t); values beyond the estimate saturate
 *   sf   = E4M3 code nearest (ties to even, saturating at 448) to the binary32 value (amax_tile / 6) * enc
 *   code = E2M1 code nearest to the binary32 product x * (enc / value(sf)); all codes 0 where value(sf) == 0
 *   dequantized value = value(code) * value(sf) / enc
 * snip_quantize_nvfp4_dual reads x[rows][ld] once and writes both copies a linear layer needs: as_stored
 * (1x16 tiles along the columns, codes [rows][cols/2]) and transposed (16x1 tiles along the rows, codes
 * stored transposed [cols][rows/2]); FP4 packing as in snip_quantize.  Scale bytes come as 512-byte atoms in
 * the order the tensor core wants them: [operand line tile of 128][128-long chunk of the contraction][half of
 * the chunk], the word of tile line r (the bytes of its four tiles of that half, in order) at
 * (r % 32) * 16 + (r / 32) * 4; lines and tiles beyond the matrix hold 0.  snip_quantize_nvfp4_sizes gives
 * the byte sizes.  stats_* (device, may both be NULL): sum x^2, sum (x - dequantized)^2 and amax of each copy;
 * ws as for snip_quantize_dual.  rounding = SNIP_ROUND_STOCHASTIC rounds the E2M1 codes of both copies
 * stochastically with `seed` (paper Sec. 6.1, meant for output gradients; rule and generator of snip_quantize_sr,
 * applied to the same binary32 product); the scale bytes are not affected.
 * snip_gemm_nvfp4: the three products of snip_gemm_quantized over such operands (a / b: codes, rows, cols,
 * fmt = FP4, block = SNIP_BLOCK_ROW_1x16 or SNIP_BLOCK_COL_16x1 with transposed set, scales unused) on
 * tcgen05.mma kind::mxf4nvf4 with scale_vec::4X: the tensor core multiplies every 16 products by both scale
 * bytes and accumulates the whole contraction in FP32 tensor memory; the epilogue divides by enc_a * enc_b
 * (from the same two bounds) and rounds.  ws: at least 256 bytes, first word = device status word.
 */
int snip_quantize_nvfp4_sizes(int64_t rows, int64_t cols, size_t *codes_bytes_host, size_t *sf_bytes_host);
int snip_quantize_nvfp4_dual(const void *x, int64_t rows, int64_t cols, int64_t ld, const float *tensor_amax,
                             void *codes_stored, void *sf_stored, snip_stats_t *stats_stored,
                             void *codes_transposed, void *sf_transposed, snip_stats_t *stats_transposed,
                             int rounding, uint64_t seed, void *ws, size_t ws_bytes, void *stream);
int snip_gemm_nvfp4(int op, const snip_qtensor_t *a_host, const void *sf_a, const float *amax_a,
                    const snip_qtensor_t *b_host, const void *sf_b, const float *amax_b, void *out,
                    int out_dtype, void *ws, size_t ws_bytes, void *stream);
/*
 * One linear layer, forward and both gradients, under the two-level option (the composition of
 * snip_linear_fwd_bwd): X, W and dY each go through snip_quantize_nvfp4_dual once, then Y = X W^T, dX = dY W,
 * dW = dY^T X through snip_gemm_nvfp4.  bounds3 (device): the magnitude bounds of X, W and dY, in this order.
 * dy_rounding / dy_seed: stochastic rounding of both copies of dY (Sec. 6.1).  stats6 (device, may be NULL):
 * X/1x16, X/16x1, W/1x16, W/16x1, dY/1x16, dY/16x1.
 */
int snip_linear_fwd_bwd_nvfp4_workspace(int64_t M, int64_t N, int64_t K, size_t *ws_bytes_host);
int snip_linear_fwd_bwd_nvfp4(const void *X, const void *W, const void *dY, void *Y, void *dX, void *dW,
                              int64_t M, int64_t N, int64_t K, int out_dtype, const float *bounds3,
                              int dy_rounding, uint64_t dy_seed, snip_stats_t *stats6, void *ws,
                              size_t ws_bytes, void *stream);

/*
 * One linear layer's forward GEMM under a precision choice: quantize X (1x128 tiles along K)
 * and W (128x128 blocks) into the workspace, then Y = Xq.Wq^T.  stats_x / stats_w may be NULL;
 * if given they receive the statistics of the two quantizations.  (Fig. 5, forward pass.)
 */
int snip_linear_fwd(const void *X, const void *W, void *Y, int64_t M, int64_t N, int64_t K,
                    int fmt_x, int fmt_w, int out_dtype, snip_stats_t *stats_x,
                    snip_stats_t *stats_w, void *ws, size_t ws_bytes, void *stream);

/* Input gradient: quantize dY (1x128 tiles along N) and W (128x128 blocks), dX = dYq.Wq.
 * (Fig. 5, backward pass; Sec. 4.3.) */
int snip_linear_dgrad(const void *dY, const void *W, void *dX, int64_t M, int64_t N, int64_t K,
                      int fmt_dy, int fmt_w, int out_dtype, snip_stats_t *stats_dy,
                      snip_stats_t *stats_w, void *ws, size_t ws_bytes, void *stream);

/* Weight gradient: quantize dY and X with 128x1 tiles along M (the contraction),
 * dW = dYq^T.Xq.  accumulate != 0 adds to dW (FP32 output only).  (Fig. 5; Sec. 4.3.) */
int snip_linear_wgrad(const void *dY, const void *X, void *dW, int64_t M, int64_t N, int64_t K,
                      int fmt_dy, int fmt_x, int out_dtype, int accumulate,
                      snip_stats_t *stats_dy, snip_stats_t *stats_x, void *ws, size_t ws_bytes,
                      void *stream);

/*
 * The three products of a linear layer under the power-of-two scale option: op = SNIP_OP_FWD (A = X,
 * B = W, out = Y), SNIP_OP_DGRAD (A = dY, B = W, out = dX) or SNIP_OP_WGRAD (A = dY, B = X, out = dW).
 * Quantizes both operands with snip_quantize_mx's rule and the tile kinds of the paper-rule calls
 * above, then runs snip_gemm_mx.  FP8 / FP4 tags only.  Workspace from snip_linear_mx_workspace.
 */
int snip_linear_mx(int op, const void *A, const void *B, void *out, int64_t M, int64_t N, int64_t K,
                   int fmt_a, int fmt_b, int out_dtype, snip_stats_t *stats_a, snip_stats_t *stats_b,
                   void *ws, size_t ws_bytes, void *stream);
int snip_linear_mx_workspace(int op, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b, size_t *bytes_host);

/* ---- statistics (paper Sec. 3.1, Step 1) -------------------------------------------------- */

/*
 * Frobenius-norm statistics of one linear layer: sum of squares of each given tensor, and the
 * quantization-error sum of squares of X, W and dY under every format selected in fmt_mask
 * (bit 1 = FP8, bit 2 = FP4) and every tile kind the tensor is consumed with, one read per
 * tensor.  These are the quantities the loss- and weight-divergence estimates are built from
 * (Sec. 4.2, 4.3).  ws_bytes must be at least snip_layer_stats_workspace().
 */
int snip_layer_stats(const snip_layer_tensors_t *t_host, uint32_t fmt_mask,
                     snip_layer_stats_t *out, void *ws, size_t ws_bytes, void *stream);
int snip_layer_stats_workspace(int64_t M, int64_t N, int64_t K, size_t *ws_bytes_host);

/*
 * One linear layer, forward and both gradients, under a precision triple (one tag per GEMM, FP8 or FP4;
 * paper Fig. 5) with every tensor read once: X, W and dY each go through snip_quantize_dual, which
 * leaves the copy for the second GEMM that consumes the tensor, then Y = X W^T, dX = dY W, dW = dY^T X.
 *   X:  1x128 tiles, fmt_fwd (fwd)    + 128x1 tiles transposed, fmt_wgrad (wgrad)
 *   W:  128x128 blocks, fmt_fwd (fwd) + the same blocks transposed, fmt_dgrad (dgrad)
 *   dY: 1x128 tiles, fmt_dgrad (dgrad) + 128x1 tiles transposed, fmt_wgrad (wgrad)
 * Results equal those of snip_linear_fwd / _dgrad / _wgrad (pow2_scale = 0) or snip_linear_mx
 * (pow2_scale = 1) called with the same tags.  pow2_scale = 2: power-of-two scales on 32-long tiles
 * along each GEMM's contraction for all three tensors (W too: 1x32 tiles for fwd, 32x1 tiles
 * transposed for dgrad; see the block-32 form of snip_quantize_mx).  stats6 (device, may be NULL): six snip_stats_t in the
 * order X/1x128, X/128x1, W/fwd format, W/dgrad format, dY/1x128, dY/128x1.  out_dtype applies to all
 * three outputs.  dy_rounding = SNIP_ROUND_STOCHASTIC rounds the FP4 copies of dY stochastically with
 * dy_seed (Sec. 6.1; see snip_quantize_sr), FP8 copies stay nearest-even.  BF16 tags are not offered
 * here (use the three separate calls).  A training loop that
 * separates forward and backward in time keeps the quantized copies instead of the bf16 activations;
 * this entry point runs the two halves back to back.
 */
int snip_linear_fwd_bwd_workspace(int64_t M, int64_t N, int64_t K, int fmt_fwd, int fmt_dgrad, int fmt_wgrad,
                                  int pow2_scale, size_t *ws_bytes_host);
int snip_linear_fwd_bwd(const void *X, const void *W, const void *dY, void *Y, void *dX, void *dW,
                        int64_t M, int64_t N, int64_t K, int fmt_fwd, int fmt_dgrad, int fmt_wgrad,
                        int out_dtype, int pow2_scale, int dy_rounding, uint64_t dy_seed,
                        snip_stats_t *stats6, void *ws, size_t ws_bytes, void *stream);

/* ---- optimizer statistics (paper Sec. 4.3) ------------------------------------------------- */

/*
 * Sum over a parameter tensor of T^2 with
 *     T = (1 - beta1) / (sqrt(v) + eps)  -  (1 - beta2) m g / ( sqrt(v) (sqrt(v) + eps)^2 ),
 * elementwise over the AdamW moments m, v (binary32, after they absorbed g) and the gradient g
 * (bf16 or binary32, g_dtype = SNIP_OUT_BF16 / SNIP_OUT_FP32).  T is the derivative of the AdamW
 * direction m / (sqrt(v) + eps) with respect to g; Step 1 collects ||T||_F per layer, and the weight
 * divergence of a quantization option is estimated as that norm times the option's gradient error
 * norm (Sec. 4.3).  Where v == 0 the second term is taken as 0 (a reading: AdamW then has m = g = 0).
 * n: number of elements, a multiple of 4; m, v 16-byte aligned, g 8-byte (bf16) or 16-byte aligned.
 * *sumsq (device, binary64) receives the sum.  Arithmetic in binary32 (reciprocal square root and
 * reciprocal to about 2 ulp), sums in binary64; agrees with the binary64 definition to about 1e-6.  One read of each input: 10 or 12 bytes per element.
 */
int snip_adamw_sensitivity_workspace(int64_t n, size_t *ws_bytes_host);
int snip_adamw_sensitivity(const float *m, const float *v, const void *g, int g_dtype, int64_t n,
                           float beta1, float beta2, float eps, double *sumsq, void *ws, size_t ws_bytes,
                           void *stream);

/* ---- scheme generation, host side (paper Sec. 4.2, 4.3, 5) --------------------------------- */

/*
 * Normalised loss divergence of one layer under one quantization option (Sec. 4.2):
 *     sqrt( (|dL/dX|_F |X - q(X)|_F / sqrt(M K))^2 + (|dL/dW|_F |W - q(W)|_F / sqrt(N K))^2 ) / |L| .
 * The gradient norms are the plain norms of dX and dW, the error norms come from snip_layer_stats /
 * snip_quantize for that option.  Host arithmetic only.
 */
double snip_loss_divergence(double grad_x_norm, double err_x_norm, int64_t M, int64_t K,
                            double grad_w_norm, double err_w_norm, int64_t N, double loss);

/*
 * Normalised weight divergence of one layer (Sec. 4.3):
 *     (1/num_layers) * lr * sqrt(1 - beta2^step) / (1 - beta1^step) * |T|_F |g_err|_F / sqrt(N K) / |W|_F
 * with |T|_F^2 from snip_adamw_sensitivity and |g_err|_F the error norm of the weight gradient under
 * the option (how it is obtained - the paper adds noise-injection passes - is the caller's business).
 */
double snip_weight_divergence(double sens_norm, double grad_err_norm, int64_t N, int64_t K, double lr,
                              double beta1, double beta2, int64_t step, double weight_norm,
                              int64_t num_layers);

/*
 * One option per layer (Sec. 5.2): minimise sum_i q[i][choice[i]] subject to
 * sum_i w[i][choice[i]] >= target, where q (m x n, row-major, finite, >= 0) is the quality loss and w
 * (m x n, >= 0) the work that option moves to the cheaper format, as an integer (FLOPs run in FP4; the
 * paper's e[i][j] is w[i][j] / total FLOPs and E_t = target / total FLOPs).  num_groups > 1 is the
 * pipeline form (Sec. 5.3): m must be a multiple of it and every group of m / num_groups consecutive
 * layers must reach ceil(target / num_groups) by itself.  Exact (Pareto-frontier dynamic programme
 * over integer work); returns SNIP_ERR_UNSUPPORTED if the target cannot be reached or the frontier
 * outgrows the solver's cap, SNIP_ERR_ARG / SNIP_ERR_SHAPE for malformed input.  Among assignments of
 * equal loss any one may be returned.  choice: m ints; q_total / w_total may be NULL.  Host only.
 */
int snip_select_scheme(int m, int n, const double *q, const int64_t *w, int64_t target, int num_groups,
                       int *choice, double *q_total, int64_t *w_total);

/* ---- device status ------------------------------------------------------------------------ */

/*
 * Testing hooks, process-wide and off by default.  (No counterpart in the paper.)
 *   SNIP_DEBUG_WAIT_LIMIT_NS : bound of every device-side wait of the GEMM kernels, the hardware-scaled
 *                              ones (snip_gemm_mx, snip_gemm_nvfp4) included (default 2e9).
 *   SNIP_DEBUG_TX_SKEW_BYTES : a multiple of 16 added to the byte count a pipeline stage's barrier
 *                              expects.  Non-zero makes the first stage of every GEMM incomplete for
 *                              ever while every copy still lands: the kernel's waits run out, it
 *                              leaves on its own and snip_poll_status reports SNIP_ERR_TIMEOUT.
 *                              Nothing traps or faults; used with a short wait limit by the tests.
 *   SNIP_DEBUG_GEMM_KERNEL   : 0 or 1 = the single-CTA kernels (the default), 2 = the CTA-pair
 *                              kernels for every quantized GEMM (an alternative form of the same
 *                              product, kept for A/B comparisons in the benchmark).
 *   SNIP_DEBUG_GEMM_SLICING  : 1 (default) = the weight-gradient product may slice its last wave
 *                              when its workspace has room (snip_workspace_size), 0 = never.
 * Returns SNIP_ERR_ARG for an unknown key or a value out of range.
 */
#define SNIP_DEBUG_WAIT_LIMIT_NS 0
#define SNIP_DEBUG_TX_SKEW_BYTES 1
#define SNIP_DEBUG_GEMM_KERNEL   2
#define SNIP_DEBUG_GEMM_SLICING  3
int snip_debug_set(int key, long long value);

/*
 * Read the device status word of a GEMM workspace.  Call after the stream has been
 * synchronized.  *status_host becomes SNIP_OK or SNIP_ERR_TIMEOUT (a bounded device-side wait
 * expired and the kernel returned early; outputs are then invalid).  Every GEMM entry point
 * zeroes the word before its kernels run (snip_linear_fwd_bwd once, before its three GEMMs), so
 * the value always belongs to the last call made with that workspace.  Performs a small
 * device-to-host copy.  (No counterpart in the paper.)
 */
int snip_poll_status(const void *ws, int *status_host);

#ifdef __cplusplus
}
#endif
#endif /* SNIP_H_ */
