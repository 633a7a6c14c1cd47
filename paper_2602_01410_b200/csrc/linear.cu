// The three GEMMs of one linear layer under a precision choice (paper Fig. 5): quantize the two
// operands with the tile kind their contraction calls for, then run the block-scaled GEMM.
// Host-side composition only; all arithmetic is in the kernels of quantize.cu, gemm.cu and gemm_mx.cu.
#include "common.cuh"

namespace snip {

int quantize_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, void *codes,
                  float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes, cudaStream_t st);
int gemm_impl(int fmt_a, int fmt_b, const void *a_codes, const void *b_codes, int64_t Mo, int64_t No, int64_t Kc, const float *sa,
              int64_t sa_chunk_stride, const float *sb, int64_t sb_chunk_stride, int64_t sb_blk_stride, int scale_mode, void *out,
              int out_dtype, int accumulate, void *ws, size_t ws_bytes, cudaStream_t st, bool clear_status);
int gemm_clear_status(void *ws, cudaStream_t st);
int quantize_impl_ex(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, int pow2, void *sf,
                     void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes, cudaStream_t st);
int gemm_mx_impl(int fmt_a, int fmt_b, const void *a_codes, const void *b_codes, const void *sfa, const void *sfb, int64_t Mo, int64_t No,
                 int64_t Kc, void *out, int out_dtype, void *ws, size_t ws_bytes, cudaStream_t st, bool clear_status);
int transpose_bf16(const void *in, void *out, int64_t rows, int64_t cols, cudaStream_t st);
size_t gemm_ws_bytes();
size_t gemm_ws_bytes_sliced();   // with room for the weight-gradient product's contraction slices
int quantize_dual_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, int kind, int pow2, const DualOut &oa, const DualOut &ob,
                       void *ws, size_t ws_bytes, cudaStream_t st);
int quantize_nvfp4_dual_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, const float *tensor_amax, void *codes_a, void *sf_a,
                             snip_stats_t *stats_a, void *codes_b, void *sf_b, snip_stats_t *stats_b, int rounding, uint64_t seed, void *ws,
                             size_t ws_bytes, cudaStream_t st);
int gemm_nvfp4_impl(const void *a_codes, const void *b_codes, const void *sfa, const void *sfb, const float *amax_a, const float *amax_b,
                    int64_t Mo, int64_t No, int64_t Kc, void *out, int out_dtype, void *ws, size_t ws_bytes, cudaStream_t st, bool clear_status);
int gemm_clear_status(void *ws, cudaStream_t st);

namespace {

enum { SCALE_NONE = 0, SCALE_BLOCK_B = 1, SCALE_VEC_B = 2 };

size_t code_bytes(int fmt, int64_t rows, int64_t cols)
{
    if (fmt == SNIP_FMT_FP8_E4M3) return (size_t)(rows * cols);
    if (fmt == SNIP_FMT_FP4_E2M1) return (size_t)(rows * cols / 2) + 64;  // + tail slack, see snip_quantize_sizes
    return (size_t)(rows * cols * 2);  // bf16 transposed copy
}
size_t scale_bytes(int block, int64_t rows, int64_t cols)
{
    const int64_t tr = ceil_div(rows, 128), tc = ceil_div(cols, 128);
    int64_t n = block == SNIP_BLOCK_ROW_1x128 ? tc * rows : block == SNIP_BLOCK_COL_128x1 ? tr * cols : tr * tc;
    if (block == SNIP_BLOCK_ROW_1x32) n = ceil_div(cols, 32) * rows;
    if (block == SNIP_BLOCK_COL_32x1) n = ceil_div(rows, 32) * cols;
    return (size_t)n * sizeof(float);
}
size_t stats_bytes(int64_t rows, int64_t cols)
{
    size_t w = 0;
    snip_quantize_sizes(rows, cols, SNIP_FMT_FP8_E4M3, SNIP_BLOCK_ROW_1x128, SNIP_Q_STATS, nullptr, nullptr, &w);
    return w;
}

// Carves the workspace of a linear call: [status 256][codes A][scales A][codes B][scales B][stats scratch]
struct Carve {
    uint8_t *base;
    size_t off = 0, cap;
    Carve(void *p, size_t c) : base(static_cast<uint8_t *>(p)), cap(c) {}
    void *take(size_t bytes)
    {
        void *r = base ? base + off : nullptr;
        off += align_up(bytes, 256);
        return r;
    }
};

struct LinearPlan {
    // operand A: rows_a x cols_a logical matrix, quantized with block_a, stored transposed or not
    int64_t rows_a, cols_a, rows_b, cols_b;
    int block_a, block_b;
    bool tr_a, tr_b;
    int64_t Mo, No, Kc;
    int scale_mode;
};

LinearPlan plan_for(int op, int64_t M, int64_t N, int64_t K)
{
    LinearPlan p{};
    if (op == SNIP_OP_FWD) {
        p = {M, K, N, K, SNIP_BLOCK_ROW_1x128, SNIP_BLOCK_BLK_128x128, false, false, M, N, K, SCALE_BLOCK_B};
    } else if (op == SNIP_OP_DGRAD) {
        p = {M, N, N, K, SNIP_BLOCK_ROW_1x128, SNIP_BLOCK_BLK_128x128, false, true, M, K, N, SCALE_BLOCK_B};
    } else {
        p = {M, N, M, K, SNIP_BLOCK_COL_128x1, SNIP_BLOCK_COL_128x1, true, true, N, K, M, SCALE_VEC_B};
    }
    return p;
}

size_t sf_bytes(int64_t rows, int64_t cols) { return (size_t)(ceil_div(rows, 128) * ceil_div(cols, 128)) * 512; }

size_t linear_ws_bytes(int op, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b, bool mx = false)
{
    const LinearPlan p = plan_for(op, M, N, K);
    Carve c(nullptr, 0);
    c.take(gemm_ws_bytes_sliced());
    const bool need_a = fmt_a != SNIP_FMT_BF16 || p.tr_a, need_b = fmt_b != SNIP_FMT_BF16 || p.tr_b;
    if (need_a) { c.take(code_bytes(fmt_a, p.rows_a, p.cols_a)); c.take(scale_bytes(p.block_a, p.rows_a, p.cols_a)); }
    if (need_b) { c.take(code_bytes(fmt_b, p.rows_b, p.cols_b)); c.take(scale_bytes(p.block_b, p.rows_b, p.cols_b)); }
    c.take(stats_bytes(p.rows_a, p.cols_a));
    c.take(stats_bytes(p.rows_b, p.cols_b));
    if (mx) { c.take(sf_bytes(p.rows_a, p.cols_a)); c.take(sf_bytes(p.rows_b, p.cols_b)); }
    return c.off;
}

int linear_impl(int op, const void *A, const void *B, void *out, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b, int out_dtype,
                int accumulate, snip_stats_t *stats_a, snip_stats_t *stats_b, void *ws, size_t ws_bytes, cudaStream_t st, bool mx = false)
{
    if (mx && (fmt_a == SNIP_FMT_BF16 || fmt_b == SNIP_FMT_BF16 || accumulate)) return SNIP_ERR_UNSUPPORTED;
    if (!A || !B || !out) return SNIP_ERR_ARG;
    if (!valid_fmt(fmt_a) || !valid_fmt(fmt_b)) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    if ((fmt_a == SNIP_FMT_BF16) != (fmt_b == SNIP_FMT_BF16)) return SNIP_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < linear_ws_bytes(op, M, N, K, fmt_a, fmt_b, mx)) return SNIP_ERR_WORKSPACE;
    if (!aligned16(ws)) return SNIP_ERR_ALIGN;
    const LinearPlan p = plan_for(op, M, N, K);
    Carve c(ws, ws_bytes);
    void *gws = c.take(gemm_ws_bytes_sliced());
    const bool q = fmt_a != SNIP_FMT_BF16;
    const bool need_a = q || p.tr_a, need_b = q || p.tr_b;
    void *codes_a = nullptr, *codes_b = nullptr;
    float *scales_a = nullptr, *scales_b = nullptr;
    if (need_a) { codes_a = c.take(code_bytes(fmt_a, p.rows_a, p.cols_a)); scales_a = static_cast<float *>(c.take(scale_bytes(p.block_a, p.rows_a, p.cols_a))); }
    if (need_b) { codes_b = c.take(code_bytes(fmt_b, p.rows_b, p.cols_b)); scales_b = static_cast<float *>(c.take(scale_bytes(p.block_b, p.rows_b, p.cols_b))); }
    const size_t sws_a_bytes = stats_bytes(p.rows_a, p.cols_a), sws_b_bytes = stats_bytes(p.rows_b, p.cols_b);
    void *sws_a = c.take(sws_a_bytes), *sws_b = c.take(sws_b_bytes);
    void *sf_a = nullptr, *sf_b = nullptr;
    if (mx) { sf_a = c.take(sf_bytes(p.rows_a, p.cols_a)); sf_b = c.take(sf_bytes(p.rows_b, p.cols_b)); }

    int rc;
    const void *ga = A, *gb = B;
    if (q) {
        rc = quantize_impl_ex(A, p.rows_a, p.cols_a, p.cols_a, fmt_a, p.block_a, (p.tr_a ? SNIP_Q_TRANSPOSED : 0u) | (stats_a ? SNIP_Q_STATS : 0u),
                              mx ? 1 : 0, sf_a, codes_a, scales_a, stats_a, nullptr, sws_a, sws_a_bytes, st);
        if (rc) return rc;
        rc = quantize_impl_ex(B, p.rows_b, p.cols_b, p.cols_b, fmt_b, p.block_b, (p.tr_b ? SNIP_Q_TRANSPOSED : 0u) | (stats_b ? SNIP_Q_STATS : 0u),
                              mx ? 1 : 0, sf_b, codes_b, scales_b, stats_b, nullptr, sws_b, sws_b_bytes, st);
        if (rc) return rc;
        ga = codes_a; gb = codes_b;
        if (mx) return gemm_mx_impl(fmt_a, fmt_b, ga, gb, sf_a, sf_b, p.Mo, p.No, p.Kc, out, out_dtype, gws, gemm_ws_bytes(), st, true);
    } else {
        // BF16 tag: identity quantization; only operands whose contraction index is not contiguous are copied
        if (p.tr_a) { rc = transpose_bf16(A, codes_a, p.rows_a, p.cols_a, st); if (rc) return rc; ga = codes_a; }
        if (p.tr_b) { rc = transpose_bf16(B, codes_b, p.rows_b, p.cols_b, st); if (rc) return rc; gb = codes_b; }
        if (stats_a) { rc = quantize_impl(A, p.rows_a, p.cols_a, p.cols_a, SNIP_FMT_BF16, SNIP_BLOCK_BLK_128x128, SNIP_Q_STATS, nullptr, nullptr, stats_a, nullptr, sws_a, sws_a_bytes, st); if (rc) return rc; }
        if (stats_b) { rc = quantize_impl(B, p.rows_b, p.cols_b, p.cols_b, SNIP_FMT_BF16, SNIP_BLOCK_BLK_128x128, SNIP_Q_STATS, nullptr, nullptr, stats_b, nullptr, sws_b, sws_b_bytes, st); if (rc) return rc; }
    }
    int64_t sa_cs = p.Mo, sb_cs, sb_bs;
    if (op == SNIP_OP_FWD) { sb_bs = ceil_div(K, 128); sb_cs = 1; }
    else if (op == SNIP_OP_DGRAD) { sb_bs = 1; sb_cs = ceil_div(K, 128); }
    else { sb_bs = 0; sb_cs = p.No; }
    return gemm_impl(fmt_a, fmt_b, ga, gb, p.Mo, p.No, p.Kc, scales_a, sa_cs, scales_b, sb_cs, sb_bs, q ? p.scale_mode : SCALE_NONE, out,
                     out_dtype, accumulate, gws, gemm_ws_bytes_sliced(), st, true);
}


// ---- forward + both gradients of one linear layer with each tensor read once ------------------

// Buffers of the six quantized copies: X as stored (fwd) / transposed (wgrad), W as stored (fwd) /
// transposed (dgrad), dY as stored (dgrad) / transposed (wgrad).
struct FwdBwdCarve {
    void *gws;
    void *codes[6];
    float *scales[6];
    void *sf[6];
    void *stats_ws;
    size_t stats_ws_bytes;
    size_t total;
};

// mx: 0 = the paper's scale rule, 1 = power-of-two scales on the paper's tiles, 2 = power-of-two scales on 32-long tiles
// (every tensor, W included, then has 1x32 tiles as stored and 32x1 tiles transposed).
FwdBwdCarve carve_fwd_bwd(void *ws, int64_t M, int64_t N, int64_t K, const int (&fmt)[6], int mx)
{
    // index: 0 X/ROW, 1 X/COL^T, 2 W/BLK, 3 W/BLK^T, 4 dY/ROW, 5 dY/COL^T
    const int64_t rows[6] = {M, M, N, N, M, M}, cols[6] = {K, K, K, K, N, N};
    const int block128[6] = {SNIP_BLOCK_ROW_1x128, SNIP_BLOCK_COL_128x1, SNIP_BLOCK_BLK_128x128, SNIP_BLOCK_BLK_128x128, SNIP_BLOCK_ROW_1x128,
                             SNIP_BLOCK_COL_128x1};
    const int block32[6] = {SNIP_BLOCK_ROW_1x32, SNIP_BLOCK_COL_32x1, SNIP_BLOCK_ROW_1x32, SNIP_BLOCK_COL_32x1, SNIP_BLOCK_ROW_1x32,
                            SNIP_BLOCK_COL_32x1};
    const int (&block)[6] = mx == 2 ? block32 : block128;
    FwdBwdCarve f{};
    Carve c(ws, 0);
    f.gws = c.take(gemm_ws_bytes_sliced());
    for (int i = 0; i < 6; ++i) {
        f.codes[i] = c.take(code_bytes(fmt[i], rows[i], cols[i]));
        f.scales[i] = static_cast<float *>(c.take(scale_bytes(block[i], rows[i], cols[i])));
        f.sf[i] = mx ? c.take(sf_bytes(rows[i], cols[i])) : nullptr;
    }
    size_t sb = 0;
    for (int i = 0; i < 6; i += 2) {
        size_t w = 0;
        snip_quantize_dual_workspace(rows[i], cols[i], &w);
        if (w > sb) sb = w;
    }
    f.stats_ws = c.take(sb);
    f.stats_ws_bytes = sb;
    f.total = c.off;
    return f;
}
}  // namespace
}  // namespace snip

extern "C" int snip_workspace_size(int op, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b, size_t *gemm_bytes, size_t *linear_bytes)
{
    using namespace snip;
    if (op < SNIP_OP_FWD || op > SNIP_OP_WGRAD || !valid_fmt(fmt_a) || !valid_fmt(fmt_b)) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    if (gemm_bytes) *gemm_bytes = (op == SNIP_OP_WGRAD && fmt_a != SNIP_FMT_BF16 && fmt_b != SNIP_FMT_BF16) ? gemm_ws_bytes_sliced() : gemm_ws_bytes();
    if (linear_bytes) *linear_bytes = linear_ws_bytes(op, M, N, K, fmt_a, fmt_b);
    return SNIP_OK;
}

extern "C" int snip_linear_fwd(const void *X, const void *W, void *Y, int64_t M, int64_t N, int64_t K, int fmt_x, int fmt_w, int out_dtype,
                               snip_stats_t *stats_x, snip_stats_t *stats_w, void *ws, size_t ws_bytes, void *stream)
{
    return snip::linear_impl(SNIP_OP_FWD, X, W, Y, M, N, K, fmt_x, fmt_w, out_dtype, 0, stats_x, stats_w, ws, ws_bytes,
                             static_cast<cudaStream_t>(stream));
}

extern "C" int snip_linear_dgrad(const void *dY, const void *W, void *dX, int64_t M, int64_t N, int64_t K, int fmt_dy, int fmt_w,
                                 int out_dtype, snip_stats_t *stats_dy, snip_stats_t *stats_w, void *ws, size_t ws_bytes, void *stream)
{
    return snip::linear_impl(SNIP_OP_DGRAD, dY, W, dX, M, N, K, fmt_dy, fmt_w, out_dtype, 0, stats_dy, stats_w, ws, ws_bytes,
                             static_cast<cudaStream_t>(stream));
}

extern "C" int snip_linear_wgrad(const void *dY, const void *X, void *dW, int64_t M, int64_t N, int64_t K, int fmt_dy, int fmt_x,
                                 int out_dtype, int accumulate, snip_stats_t *stats_dy, snip_stats_t *stats_x, void *ws, size_t ws_bytes,
                                 void *stream)
{
    return snip::linear_impl(SNIP_OP_WGRAD, dY, X, dW, M, N, K, fmt_dy, fmt_x, out_dtype, accumulate, stats_dy, stats_x, ws, ws_bytes,
                             static_cast<cudaStream_t>(stream));
}

// Power-of-two scale option of the three calls above in one entry point (op selects the product).
extern "C" int snip_linear_mx(int op, const void *A, const void *B, void *out, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b,
                              int out_dtype, snip_stats_t *stats_a, snip_stats_t *stats_b, void *ws, size_t ws_bytes, void *stream)
{
    if (op < SNIP_OP_FWD || op > SNIP_OP_WGRAD) return SNIP_ERR_ARG;
    return snip::linear_impl(op, A, B, out, M, N, K, fmt_a, fmt_b, out_dtype, 0, stats_a, stats_b, ws, ws_bytes, static_cast<cudaStream_t>(stream), true);
}

extern "C" int snip_linear_mx_workspace(int op, int64_t M, int64_t N, int64_t K, int fmt_a, int fmt_b, size_t *bytes)
{
    using namespace snip;
    if (!bytes || op < SNIP_OP_FWD || op > SNIP_OP_WGRAD || !valid_fmt(fmt_a) || !valid_fmt(fmt_b)) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    *bytes = linear_ws_bytes(op, M, N, K, fmt_a, fmt_b, true);
    return SNIP_OK;
}

// One linear layer, forward and both gradients, under a precision triple (one tag per GEMM).
extern "C" int snip_linear_fwd_bwd_workspace(int64_t M, int64_t N, int64_t K, int fmt_fwd, int fmt_dgrad, int fmt_wgrad, int pow2_scale,
                                             size_t *bytes)
{
    using namespace snip;
    if (!bytes) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    const int fmt[6] = {fmt_fwd, fmt_wgrad, fmt_fwd, fmt_dgrad, fmt_dgrad, fmt_wgrad};
    for (int f : fmt)
        if (f != SNIP_FMT_FP8_E4M3 && f != SNIP_FMT_FP4_E2M1) return SNIP_ERR_UNSUPPORTED;
    if (pow2_scale < 0 || pow2_scale > 2) return SNIP_ERR_ARG;
    *bytes = carve_fwd_bwd(nullptr, M, N, K, fmt, pow2_scale).total;
    return SNIP_OK;
}

extern "C" int snip_linear_fwd_bwd(const void *X, const void *W, const void *dY, void *Y, void *dX, void *dW, int64_t M, int64_t N, int64_t K,
                                   int fmt_fwd, int fmt_dgrad, int fmt_wgrad, int out_dtype, int pow2_scale, int dy_rounding, uint64_t dy_seed,
                                   snip_stats_t *stats6, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!X || !W || !dY || !Y || !dX || !dW) return SNIP_ERR_ARG;
    size_t need = 0;
    int rc = snip_linear_fwd_bwd_workspace(M, N, K, fmt_fwd, fmt_dgrad, fmt_wgrad, pow2_scale, &need);
    if (rc) return rc;
    if (!ws || ws_bytes < need) return SNIP_ERR_WORKSPACE;
    if (!aligned16(ws) || (stats6 && (reinterpret_cast<uintptr_t>(stats6) & 7u))) return SNIP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool mx = pow2_scale != 0;
    const int fmt[6] = {fmt_fwd, fmt_wgrad, fmt_fwd, fmt_dgrad, fmt_dgrad, fmt_wgrad};
    const FwdBwdCarve f = carve_fwd_bwd(ws, M, N, K, fmt, pow2_scale);
    const int kind_xdy = pow2_scale == 2 ? SNIP_DUAL_ROW32_COL32T : SNIP_DUAL_ROW_COLT;
    const int kind_w = pow2_scale == 2 ? SNIP_DUAL_ROW32_COL32T : SNIP_DUAL_BLK_BLKT;
    if (dy_rounding != SNIP_ROUND_NEAREST_EVEN && dy_rounding != SNIP_ROUND_STOCHASTIC) return SNIP_ERR_ARG;
    // stochastic rounding applies to the FP4 copies of dY (indices 4 and 5); an FP8 copy keeps nearest-even
    auto out_of = [&](int i) {
        const int sr = (i >= 4 && dy_rounding == SNIP_ROUND_STOCHASTIC && fmt[i] == SNIP_FMT_FP4_E2M1) ? 1 : 0;
        return DualOut{fmt[i], f.codes[i], f.scales[i], f.sf[i], stats6 ? stats6 + i : nullptr, sr, dy_seed};
    };
    auto gemm = [&](int op, int ia, int ib, void *out) -> int {
        const LinearPlan p = plan_for(op, M, N, K);
        if (mx) return gemm_mx_impl(fmt[ia], fmt[ib], f.codes[ia], f.codes[ib], f.sf[ia], f.sf[ib], p.Mo, p.No, p.Kc, out, out_dtype, f.gws, gemm_ws_bytes(), st, false);
        int64_t sb_cs, sb_bs;
        if (op == SNIP_OP_FWD) { sb_bs = ceil_div(K, 128); sb_cs = 1; }
        else if (op == SNIP_OP_DGRAD) { sb_bs = 1; sb_cs = ceil_div(K, 128); }
        else { sb_bs = 0; sb_cs = p.No; }
        return gemm_impl(fmt[ia], fmt[ib], f.codes[ia], f.codes[ib], p.Mo, p.No, p.Kc, f.scales[ia], p.Mo, f.scales[ib], sb_cs, sb_bs, p.scale_mode, out,
                         out_dtype, 0, f.gws, gemm_ws_bytes_sliced(), st, false);
    };
    // one status word serves the three GEMMs of this call: cleared once, so that a timeout of the first is not erased
    rc = gemm_clear_status(f.gws, st);
    if (rc) return rc;
    // forward: X and W are read once each and leave both of their quantized copies behind
    rc = quantize_dual_impl(X, M, K, K, kind_xdy, mx, out_of(0), out_of(1), f.stats_ws, f.stats_ws_bytes, st);
    if (rc) return rc;
    rc = quantize_dual_impl(W, N, K, K, kind_w, mx, out_of(2), out_of(3), f.stats_ws, f.stats_ws_bytes, st);
    if (rc) return rc;
    rc = gemm(SNIP_OP_FWD, 0, 2, Y);
    if (rc) return rc;
    // backward: dY is read once; dgrad and wgrad consume the stored copies
    rc = quantize_dual_impl(dY, M, N, N, kind_xdy, mx, out_of(4), out_of(5), f.stats_ws, f.stats_ws_bytes, st);
    if (rc) return rc;
    rc = gemm(SNIP_OP_DGRAD, 4, 3, dX);
    if (rc) return rc;
    return gemm(SNIP_OP_WGRAD, 5, 1, dW);
}

// ---- the same composition under the two-level (NVFP4-style) option ---------------------------------

namespace snip {
namespace {
struct NvCarve {
    void *gws;
    void *codes[6];
    void *sf[6];
    void *stats_ws;
    size_t stats_ws_bytes, total;
};
NvCarve carve_nvfp4(void *ws, int64_t M, int64_t N, int64_t K)
{
    // index: 0 X/1x16, 1 X/16x1^T, 2 W/1x16, 3 W/16x1^T, 4 dY/1x16, 5 dY/16x1^T
    const int64_t rows[6] = {M, M, N, N, M, M}, cols[6] = {K, K, K, K, N, N};
    NvCarve f{};
    Carve c(ws, 0);
    f.gws = c.take(gemm_ws_bytes());
    size_t sb = 0;
    for (int i = 0; i < 6; ++i) {
        size_t cb = 0, fb = 0;
        snip_quantize_nvfp4_sizes(rows[i], cols[i], &cb, &fb);
        f.codes[i] = c.take(cb);
        f.sf[i] = c.take(fb);
        size_t w = 0;
        snip_quantize_dual_workspace(rows[i], cols[i], &w);
        if (w > sb) sb = w;
    }
    f.stats_ws = c.take(sb);
    f.stats_ws_bytes = sb;
    f.total = c.off;
    return f;
}
}  // namespace
}  // namespace snip

extern "C" int snip_linear_fwd_bwd_nvfp4_workspace(int64_t M, int64_t N, int64_t K, size_t *bytes)
{
    using namespace snip;
    if (!bytes) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    *bytes = carve_nvfp4(nullptr, M, N, K).total;
    return SNIP_OK;
}

extern "C" int snip_linear_fwd_bwd_nvfp4(const void *X, const void *W, const void *dY, void *Y, void *dX, void *dW, int64_t M, int64_t N, int64_t K,
                                         int out_dtype, const float *bounds3, int dy_rounding, uint64_t dy_seed, snip_stats_t *stats6, void *ws,
                                         size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!X || !W || !dY || !Y || !dX || !dW || !bounds3) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    if (dy_rounding != SNIP_ROUND_NEAREST_EVEN && dy_rounding != SNIP_ROUND_STOCHASTIC) return SNIP_ERR_ARG;
    const NvCarve f = carve_nvfp4(ws, M, N, K);
    if (!ws || ws_bytes < f.total) return SNIP_ERR_WORKSPACE;
    if (!aligned16(ws) || (stats6 && (reinterpret_cast<uintptr_t>(stats6) & 7u))) return SNIP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float *bx = bounds3, *bw = bounds3 + 1, *bdy = bounds3 + 2;
    auto stat = [&](int i) { return stats6 ? stats6 + i : nullptr; };
    int rc = gemm_clear_status(f.gws, st);   // one status word for the three GEMMs
    if (rc) return rc;
    rc = quantize_nvfp4_dual_impl(X, M, K, K, bx, f.codes[0], f.sf[0], stat(0), f.codes[1], f.sf[1], stat(1), SNIP_ROUND_NEAREST_EVEN, 0, f.stats_ws,
                                  f.stats_ws_bytes, st);
    if (rc) return rc;
    rc = quantize_nvfp4_dual_impl(W, N, K, K, bw, f.codes[2], f.sf[2], stat(2), f.codes[3], f.sf[3], stat(3), SNIP_ROUND_NEAREST_EVEN, 0, f.stats_ws,
                                  f.stats_ws_bytes, st);
    if (rc) return rc;
    rc = gemm_nvfp4_impl(f.codes[0], f.codes[2], f.sf[0], f.sf[2], bx, bw, M, N, K, Y, out_dtype, f.gws, gemm_ws_bytes(), st, false);
    if (rc) return rc;
    rc = quantize_nvfp4_dual_impl(dY, M, N, N, bdy, f.codes[4], f.sf[4], stat(4), f.codes[5], f.sf[5], stat(5), dy_rounding, dy_seed, f.stats_ws,
                                  f.stats_ws_bytes, st);
    if (rc) return rc;
    rc = gemm_nvfp4_impl(f.codes[4], f.codes[3], f.sf[4], f.sf[3], bdy, bw, M, K, N, dX, out_dtype, f.gws, gemm_ws_bytes(), st, false);
    if (rc) return rc;
    return gemm_nvfp4_impl(f.codes[5], f.codes[1], f.sf[5], f.sf[1], bdy, bx, N, K, M, dW, out_dtype, f.gws, gemm_ws_bytes(), st, false);
}
