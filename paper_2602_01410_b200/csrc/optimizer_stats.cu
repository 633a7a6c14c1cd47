// AdamW sensitivity-term norm (paper Sec. 4.3): sum over a parameter tensor of T^2 with
//   T = (1 - beta1) / (sqrt(v) + eps)  -  (1 - beta2) m g / ( sqrt(v) (sqrt(v) + eps)^2 ),
// the derivative of the AdamW direction with respect to the gradient; Step 1 collects its Frobenius
// norm per layer for the weight-divergence estimate.
//
// HBM-bound: reads m and v (binary32) and g (bf16 or binary32) once, 10 or 12 bytes per element, and
// writes one binary64 partial per CTA; a second, one-CTA kernel adds the partials in fixed order.
#include "common.cuh"

namespace snip {

int gemm_sm_count();

namespace {

constexpr int kThreads = 256;
constexpr int kCtasPerSm = 8;

__device__ __forceinline__ float sens_term_sq(float m, float v, float g, float omb1, float omb2, float eps)
{
    // reciprocal square root and reciprocal from the special-function unit (about 2 ulp and 1 ulp): far
    // inside the 1e-4 the norm is compared at, and a third of the instructions of IEEE sqrt + two divisions
    const float rs = rsqrtf(v);              // +inf for v == 0, handled below
    const float s = v * rs;
    const float rd = __frcp_rn((v == 0.0f ? 0.0f : s) + eps);
    // (1 - beta2) * (m / s) * (g / d^2): |m| <~ s in AdamW, so neither factor over- or underflows early
    const float second = v == 0.0f ? 0.0f : omb2 * (m * rs) * (g * rd * rd);
    const float t = omb1 * rd - second;
    return t * t;
}

template <bool G_BF16>
__global__ void __launch_bounds__(kThreads) adamw_sensitivity_kernel(const float *__restrict__ m, const float *__restrict__ v, const void *__restrict__ g,
                                                                     int64_t n4, float omb1, float omb2, float eps, double *partials)
{
    __shared__ double red[kThreads / 32];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    double acc = 0.0;
    const float4 *m4 = reinterpret_cast<const float4 *>(m), *v4 = reinterpret_cast<const float4 *>(v);
    auto load_g = [&](int64_t i) {
        if (G_BF16) {
            const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(g) + i);
            return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u), __uint_as_float(raw.y << 16),
                               __uint_as_float(raw.y & 0xFFFF0000u));
        }
        return __ldg(reinterpret_cast<const float4 *>(g) + i);
    };
    auto four = [&](const float4 &mm, const float4 &vv, const float4 &gg) {
        return (sens_term_sq(mm.x, vv.x, gg.x, omb1, omb2, eps) + sens_term_sq(mm.y, vv.y, gg.y, omb1, omb2, eps)) +
               (sens_term_sq(mm.z, vv.z, gg.z, omb1, omb2, eps) + sens_term_sq(mm.w, vv.w, gg.w, omb1, omb2, eps));
    };
    // two groups of four elements per iteration: 80 (bf16 g) or 96 bytes in flight per thread
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    for (; i + stride < n4; i += 2 * stride) {
        const float4 m0 = __ldg(m4 + i), v0 = __ldg(v4 + i), m1 = __ldg(m4 + i + stride), v1 = __ldg(v4 + i + stride);
        const float4 g0 = load_g(i), g1 = load_g(i + stride);
        acc += (double)(four(m0, v0, g0) + four(m1, v1, g1));
    }
    if (i < n4) acc += (double)four(__ldg(m4 + i), __ldg(v4 + i), load_g(i));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) t += red[w];
        partials[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(1024) sum_partials_kernel(const double *partials, int n, double *out)
{
    __shared__ double red[32];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += 1024) acc += partials[i];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 32; ++w) t += red[w];
        *out = t;
    }
}

int grid_for(int64_t n4)
{
    const int64_t cap = (int64_t)kCtasPerSm * gemm_sm_count();
    const int64_t need = ceil_div(n4, kThreads);
    return (int)(need < cap ? (need > 0 ? need : 1) : cap);
}

}  // namespace
}  // namespace snip

extern "C" int snip_adamw_sensitivity_workspace(int64_t n, size_t *ws_bytes)
{
    using namespace snip;
    if (!ws_bytes) return SNIP_ERR_ARG;
    if (n <= 0 || (n % 4) != 0) return SNIP_ERR_SHAPE;
    // one binary64 partial per CTA of the largest grid any device of this family launches
    *ws_bytes = align_up(sizeof(double) * 8 * 1024, 256);
    return SNIP_OK;
}

extern "C" int snip_adamw_sensitivity(const float *m, const float *v, const void *g, int g_dtype, int64_t n, float beta1, float beta2, float eps,
                                      double *sumsq, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!m || !v || !g || !sumsq || !ws) return SNIP_ERR_ARG;
    if (g_dtype != SNIP_OUT_BF16 && g_dtype != SNIP_OUT_FP32) return SNIP_ERR_ARG;
    if (n <= 0 || (n % 4) != 0) return SNIP_ERR_SHAPE;
    if (!aligned16(m) || !aligned16(v) || (reinterpret_cast<uintptr_t>(g) & (g_dtype == SNIP_OUT_BF16 ? 7u : 15u)) || (reinterpret_cast<uintptr_t>(sumsq) & 7u) ||
        !aligned16(ws))
        return SNIP_ERR_ALIGN;
    int rc = require_sm100();
    if (rc) return rc;
    const int64_t n4 = n / 4;
    const int grid = grid_for(n4);
    if (ws_bytes < sizeof(double) * (size_t)grid) return SNIP_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double *partials = static_cast<double *>(ws);
    if (g_dtype == SNIP_OUT_BF16) adamw_sensitivity_kernel<true><<<grid, kThreads, 0, st>>>(m, v, g, n4, 1.0f - beta1, 1.0f - beta2, eps, partials);
    else adamw_sensitivity_kernel<false><<<grid, kThreads, 0, st>>>(m, v, g, n4, 1.0f - beta1, 1.0f - beta2, eps, partials);
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
    const double *cparts = partials;
    SNIP_CUDA_TRY(cudaLaunchKernelEx(&cfg, sum_partials_kernel, cparts, grid, sumsq));
    return SNIP_OK;
}
