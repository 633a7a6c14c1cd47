// Layer statistics in one read per tensor (paper Sec. 3.1, Step 1): sum x^2 of a bf16 tensor and,
// for the tensors that get quantized (X, W, dY), the error sums  sum (x - code/S)^2  under every
// candidate format (FP8 E4M3, FP4 E2M1) and every tile kind the tensor is consumed with
// (X, dY: 1x128 along the columns and 128x1 along the rows; W: 128x128), all from the same
// registers.  The scheme-generation step needs the error of every option (Sec. 4.4), not only of
// the format currently in use.
//
// One CTA owns a 128x128 tile, each thread an 8x8 sub-block (the quantizer's load pattern).  The
// arithmetic per option is the quantizer's: S = FPX_MAX/amax (binary32 quotient), code =
// RNE_fmt(fl32(x*S)), error term x - value(code)/S.  HBM-bound on the read (2 bytes per element)
// only when one option is selected; with all four options of X / dY the conversions make it
// ALU-bound at roughly 1.5x the read time, still far below four separate passes.
#include "common.cuh"
#include "quant_device.cuh"

namespace snip {

namespace {

constexpr int kTile = 128;
constexpr int kThreads = 256;

enum { MODE_PLAIN = 0, MODE_BLK = 1, MODE_ROWCOL = 2 };

// per CTA: [0] sum x^2; [1] FP8 kind A; [2] FP8 kind B; [3] FP4 kind A; [4] FP4 kind B
// (ROWCOL: A = ROW, B = COL; BLK: A = BLK, B unused)
struct StatsPartial {
    double v[8];
};

struct LayerStatsArgs {
    const uint16_t *x;
    int64_t rows, cols;
    StatsPartial *partials;
};

// Adds, for the 8 elements of one 128-bit load, the squared error under format FMT with the scale
// pairs s2 / negated reciprocal pairs n2 (element pair i uses s2[i], n2[i]).
template <int FMT>
__device__ __forceinline__ void err8(const uint4 &v, const float2 (&s2)[4], const float2 (&n2)[4], float2 &se2)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 x = make_float2(bf16lo(w[i]), bf16hi(w[i]));
        const float2 t = __fmul2_rn(x, s2[i]);
        float2 d;
        if (FMT == SNIP_FMT_FP8_E4M3) d = dec_e4m3x2(cvt_e4m3x2(t.x, t.y));
        else d = dec_e2m1x2(cvt_e2m1x2(t.x, t.y));
        const float2 e = __ffma2_rn(d, n2[i], x);
        se2 = __ffma2_rn(e, e, se2);
    }
}

template <int FMT>
__device__ __forceinline__ float ninv_of(float amax)
{
    constexpr float kMax = (FMT == SNIP_FMT_FP8_E4M3) ? 448.0f : 6.0f;
    return -amax * (1.0f / kMax);
}

// One format's error sums for this thread's 8x8 sub-block.  row_am[p]: amax of the 1x128 tile of
// row p; col_am[j]: amax of the 128x1 tile of column j; blk_am: amax of the 128x128 block.
template <int FMT, int MODE>
__device__ __forceinline__ void format_errors(const uint4 (&v)[8], const float (&row_am)[8], const float (&col_am)[8], float blk_am,
                                              float &err_a, float &err_b)
{
    float2 ea = make_float2(0.0f, 0.0f), eb = make_float2(0.0f, 0.0f);
    if (MODE == MODE_BLK) {
        const float s = tile_scale<FMT>(blk_am, 0), n = ninv_of<FMT>(blk_am);
        float2 s2[4], n2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { s2[i] = make_float2(s, s); n2[i] = make_float2(n, n); }
#pragma unroll
        for (int p = 0; p < 8; ++p) err8<FMT>(v[p], s2, n2, ea);
    } else {
        float2 cs2[4], cn2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            cs2[i] = make_float2(tile_scale<FMT>(col_am[2 * i], 0), tile_scale<FMT>(col_am[2 * i + 1], 0));
            cn2[i] = make_float2(ninv_of<FMT>(col_am[2 * i]), ninv_of<FMT>(col_am[2 * i + 1]));
        }
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const float s = tile_scale<FMT>(row_am[p], 0), n = ninv_of<FMT>(row_am[p]);
            float2 rs2[4], rn2[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { rs2[i] = make_float2(s, s); rn2[i] = make_float2(n, n); }
            err8<FMT>(v[p], rs2, rn2, ea);
            err8<FMT>(v[p], cs2, cn2, eb);
        }
    }
    err_a = ea.x + ea.y;
    err_b = eb.x + eb.y;
}

template <int MODE, bool F8, bool F4>
__global__ void __launch_bounds__(kThreads) layer_stats_kernel(const LayerStatsArgs a)
{
    __shared__ uint32_t col_amax[8][kTile / 2];  // packed bf16 pairs, one row per warp
    __shared__ float col_amax_f[kTile];
    __shared__ float red[8][5];
    __shared__ float red_m[8];

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t r0 = (int64_t)blockIdx.y * kTile, c0 = (int64_t)blockIdx.x * kTile;
    const int64_t rbase = r0 + 8 * ty, cbase = c0 + 8 * tx;

    uint4 v[8];
    {
        const uint16_t *xb = a.x + rbase * a.cols + cbase;
        const bool ok = rbase < a.rows && cbase < a.cols;  // dims are multiples of 64: all 64 elements or none
        const uint32_t ld32 = (uint32_t)a.cols;
#pragma unroll
        for (int p = 0; p < 8; ++p) v[p] = ok ? __ldg(reinterpret_cast<const uint4 *>(xb + p * ld32)) : make_uint4(0, 0, 0, 0);
    }

    float row_am[8], col_am[8], blk_am = 0.0f;
#pragma unroll
    for (int p = 0; p < 8; ++p) { row_am[p] = 0.0f; col_am[p] = 0.0f; }
    if (MODE == MODE_ROWCOL) {
        // rows: fold the 8 columns of this thread, pack two rows per register, reduce over the 16 lanes of a row
        uint32_t pk[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t m0 = absmax2(absmax2(absmax2(absmax2(0u, v[2 * q].x), v[2 * q].y), v[2 * q].z), v[2 * q].w);
            uint32_t m1 = absmax2(absmax2(absmax2(absmax2(0u, v[2 * q + 1].x), v[2 * q + 1].y), v[2 * q + 1].z), v[2 * q + 1].w);
            m0 = max2(m0, m0 >> 16);
            m1 = max2(m1, m1 << 16);
            pk[q] = (m0 & 0xFFFFu) | (m1 & 0xFFFF0000u);
        }
#pragma unroll
        for (int off = 1; off < 16; off <<= 1)
#pragma unroll
            for (int q = 0; q < 4; ++q) pk[q] = max2(pk[q], __shfl_xor_sync(0xFFFFFFFFu, pk[q], off));
#pragma unroll
        for (int q = 0; q < 4; ++q) { row_am[2 * q] = bf16lo(pk[q]); row_am[2 * q + 1] = bf16hi(pk[q]); }
        // columns: this thread's 8 rows, the two row groups of the warp, then the 8 warps through shared memory
        uint32_t cm[4] = {0, 0, 0, 0};
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            cm[0] = absmax2(cm[0], v[p].x);
            cm[1] = absmax2(cm[1], v[p].y);
            cm[2] = absmax2(cm[2], v[p].z);
            cm[3] = absmax2(cm[3], v[p].w);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) cm[q] = max2(cm[q], __shfl_xor_sync(0xFFFFFFFFu, cm[q], 16));
        if (lane < 16) *reinterpret_cast<uint4 *>(&col_amax[warp][4 * tx]) = make_uint4(cm[0], cm[1], cm[2], cm[3]);
        __syncthreads();
        if (tid < kTile) {
            const uint16_t *h = reinterpret_cast<const uint16_t *>(&col_amax[0][0]);
            uint32_t m = 0;
#pragma unroll
            for (int w = 0; w < 8; ++w) m = max(m, (uint32_t)h[w * kTile + tid]);  // non-negative bf16: integer order
            col_amax_f[tid] = __uint_as_float(m << 16);
        }
        __syncthreads();
        const float4 c0v = *reinterpret_cast<const float4 *>(&col_amax_f[8 * tx]);
        const float4 c1v = *reinterpret_cast<const float4 *>(&col_amax_f[8 * tx + 4]);
        col_am[0] = c0v.x; col_am[1] = c0v.y; col_am[2] = c0v.z; col_am[3] = c0v.w;
        col_am[4] = c1v.x; col_am[5] = c1v.y; col_am[6] = c1v.z; col_am[7] = c1v.w;
    } else if (MODE == MODE_BLK) {
        uint32_t m = 0;
#pragma unroll
        for (int p = 0; p < 8; ++p) m = absmax2(absmax2(absmax2(absmax2(m, v[p].x), v[p].y), v[p].z), v[p].w);
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) m = max2(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
        if (lane == 0) red_m[warp] = fmaxf(bf16lo(m), bf16hi(m));
        __syncthreads();
        blk_am = red_m[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) blk_am = fmaxf(blk_am, red_m[w]);
    }

    float acc[5] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    {
        float2 sx2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const uint32_t w[4] = {v[p].x, v[p].y, v[p].z, v[p].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 x = make_float2(bf16lo(w[i]), bf16hi(w[i]));
                sx2 = __ffma2_rn(x, x, sx2);
            }
        }
        acc[0] = sx2.x + sx2.y;
    }
    if (MODE != MODE_PLAIN) {
        if (F8) format_errors<SNIP_FMT_FP8_E4M3, MODE>(v, row_am, col_am, blk_am, acc[1], acc[2]);
        if (F4) format_errors<SNIP_FMT_FP4_E2M1, MODE>(v, row_am, col_am, blk_am, acc[3], acc[4]);
    }

#pragma unroll
    for (int k = 0; k < 5; ++k) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[k] += __shfl_xor_sync(0xFFFFFFFFu, acc[k], off);
    }
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 5; ++k) red[warp][k] = acc[k];
    }
    __syncthreads();
    if (tid < 5) {
        double d = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) d += (double)red[w][tid];
        a.partials[(int64_t)blockIdx.y * gridDim.x + blockIdx.x].v[tid] = d;
    }
}

// Fixed-order sum of the per-CTA partials; dst[k] (null = skip) receives column k.
struct ReduceDst {
    double *p[5];
};
__global__ void __launch_bounds__(1024) layer_stats_reduce_kernel(const StatsPartial *partials, int64_t n, const ReduceDst dst)
{
    __shared__ double sh[32][5];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    double d[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
    for (int64_t i = threadIdx.x; i < n; i += 1024) {
#pragma unroll
        for (int k = 0; k < 5; ++k) d[k] += partials[i].v[k];
    }
#pragma unroll
    for (int k = 0; k < 5; ++k) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d[k] += __shfl_xor_sync(0xFFFFFFFFu, d[k], off);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 5; ++k) sh[warp][k] = d[k];
    }
    __syncthreads();
    if (threadIdx.x < 5 && dst.p[threadIdx.x]) {
        double t = 0.0;
        for (int w = 0; w < 32; ++w) t += sh[w][threadIdx.x];
        *dst.p[threadIdx.x] = t;
    }
}

template <int MODE>
void launch_mode(const LayerStatsArgs &a, uint32_t fmt_mask, dim3 grid, cudaStream_t st)
{
    const bool f8 = (fmt_mask & 2u) != 0, f4 = (fmt_mask & 4u) != 0;
    if (f8 && f4) layer_stats_kernel<MODE, true, true><<<grid, kThreads, 0, st>>>(a);
    else if (f8) layer_stats_kernel<MODE, true, false><<<grid, kThreads, 0, st>>>(a);
    else layer_stats_kernel<MODE, false, true><<<grid, kThreads, 0, st>>>(a);
}

size_t tensor_ws_bytes(int64_t rows, int64_t cols)
{
    return align_up((size_t)(ceil_div(rows, kTile) * ceil_div(cols, kTile)) * sizeof(StatsPartial), 256);
}

}  // namespace
}  // namespace snip

extern "C" int snip_layer_stats_workspace(int64_t M, int64_t N, int64_t K, size_t *ws_bytes)
{
    using namespace snip;
    if (!ws_bytes) return SNIP_ERR_ARG;
    if (!valid_dim(M) || !valid_dim(N) || !valid_dim(K)) return SNIP_ERR_SHAPE;
    // one scratch region per tensor, so that the six passes need no ordering among themselves
    *ws_bytes = 2 * (tensor_ws_bytes(M, K) + tensor_ws_bytes(N, K) + tensor_ws_bytes(M, N));
    return SNIP_OK;
}

extern "C" int snip_layer_stats(const snip_layer_tensors_t *t, uint32_t fmt_mask, snip_layer_stats_t *out, void *ws, size_t ws_bytes,
                                void *stream)
{
    using namespace snip;
    if (!t || !out || !ws) return SNIP_ERR_ARG;
    if (fmt_mask & ~6u) return SNIP_ERR_ARG;
    size_t need = 0;
    int rc = snip_layer_stats_workspace(t->M, t->N, t->K, &need);
    if (rc) return rc;
    if (ws_bytes < need) return SNIP_ERR_WORKSPACE;
    if (!aligned16(ws) || !aligned16(out)) return SNIP_ERR_ALIGN;
    rc = require_sm100();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t M = t->M, N = t->N, K = t->K;
    struct T { const void *p; int64_t r, c; int qidx; } tens[6] = {
        {t->X, M, K, 0}, {t->W, N, K, 1}, {t->Y, M, N, -1}, {t->dY, M, N, 2}, {t->dX, M, K, -1}, {t->dW, N, K, -1}};
    // every argument is checked before anything is enqueued
    for (int i = 0; i < 6; ++i) {
        if (!tens[i].p) continue;
        if (!aligned16(tens[i].p)) return SNIP_ERR_ALIGN;
        if (ceil_div(tens[i].r, kTile) > 65535) return SNIP_ERR_SHAPE;
    }
    SNIP_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(snip_layer_stats_t), st));
    uint8_t *cursor = static_cast<uint8_t *>(ws);
    for (int i = 0; i < 6; ++i) {
        const size_t region = tensor_ws_bytes(tens[i].r, tens[i].c);
        StatsPartial *parts = reinterpret_cast<StatsPartial *>(cursor);
        cursor += region;
        if (!tens[i].p) continue;
        const int64_t tr = ceil_div(tens[i].r, kTile), tc = ceil_div(tens[i].c, kTile);
        LayerStatsArgs a;
        a.x = static_cast<const uint16_t *>(tens[i].p);
        a.rows = tens[i].r; a.cols = tens[i].c;
        a.partials = parts;
        dim3 grid((unsigned)tc, (unsigned)tr);
        const int q = tens[i].qidx;
        ReduceDst dst = {{&out->sumsq[i], nullptr, nullptr, nullptr, nullptr}};
        if (q < 0 || !(fmt_mask & 6u)) {
            layer_stats_kernel<MODE_PLAIN, false, false><<<grid, kThreads, 0, st>>>(a);
        } else if (q == 1) {
            launch_mode<MODE_BLK>(a, fmt_mask, grid, st);
            if (fmt_mask & 2u) dst.p[1] = &out->sumsq_err[q][0][SNIP_BLOCK_BLK_128x128];
            if (fmt_mask & 4u) dst.p[3] = &out->sumsq_err[q][1][SNIP_BLOCK_BLK_128x128];
        } else {
            launch_mode<MODE_ROWCOL>(a, fmt_mask, grid, st);
            if (fmt_mask & 2u) { dst.p[1] = &out->sumsq_err[q][0][SNIP_BLOCK_ROW_1x128]; dst.p[2] = &out->sumsq_err[q][0][SNIP_BLOCK_COL_128x1]; }
            if (fmt_mask & 4u) { dst.p[3] = &out->sumsq_err[q][1][SNIP_BLOCK_ROW_1x128]; dst.p[4] = &out->sumsq_err[q][1][SNIP_BLOCK_COL_128x1]; }
        }
        SNIP_CUDA_TRY(cudaGetLastError());
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1);
        cfg.blockDim = dim3(1024);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const StatsPartial *cparts = parts;
        const int64_t nparts = tr * tc;
        SNIP_CUDA_TRY(cudaLaunchKernelEx(&cfg, layer_stats_reduce_kernel, cparts, nparts, dst));
    }
    return SNIP_OK;
}
