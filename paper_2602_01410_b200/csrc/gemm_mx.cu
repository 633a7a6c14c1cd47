// GEMMs for the power-of-two scale option: out[Mo,No] = A[Mo,Kc] . B[No,Kc]^T where every 128-long
// chunk of the contraction carries a power-of-two scale per operand line.  The tensor core applies
// the scales itself (tcgen05.mma ... block_scale with UE8M0 scale factors in tensor memory), so the
// whole contraction accumulates in tensor memory and the epilogue runs once per output tile.
// (Power-of-two block scales are the MX-format convention the paper cites in Sec. 2.3; the paper's own
// rule FPX_MAX/amax needs the per-chunk FP32 promotion of gemm.cu.)
//
// One CTA per SM, persistent, 384 threads: warp 0 streams operand tiles (TMA) and 512-byte
// scale-factor atoms (bulk copies) into a shared-memory ring; warp 1 copies each stage's atoms into
// tensor memory (tcgen05.cp) and issues the MMAs; warps 4-11 drain the 128x256 FP32 accumulator
// (one buffer: 256 columns, next to 12 or 24 scale-factor columns), round, and store through the TMA unit.
// Warps 0 and 1 walk their loops as whole warps and one elected lane issues.  Every wait is bounded, as in gemm.cu.
//
// The bytes may differ within a chunk (32-long tiles: byte k belongs to the k-th 32 elements; the MMA of that step
// selects it through the descriptor's scale-factor id).  A third instantiation serves the two-level option in the
// style of NVFP4: E2M1 codes, an E4M3 scale byte per 16 elements (a word per line and 64-long MMA step, two atoms per
// chunk), tcgen05.mma kind::mxf4nvf4 with scale_vec::4X, and one division by the two per-tensor factors at the end.
#include <cuda.h>
#include <cuda_bf16.h>
#include <float.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "sm100.cuh"

namespace snip {

using namespace sm100;

namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int kThreads = 384;
constexpr int kNumEpiWarps = 8;
constexpr int kSfaCol = 256;   // tensor-memory columns: accumulator 0..255, SFA 256..259, SFB 260..267
constexpr int kSfbCol = 260;
constexpr int kNvSfbCol = 264; // two-level option: a word per line and MMA: SFA 256..263 (two MMAs), SFB 264..279
constexpr int kTmemCols = 512;

struct MxArgs {
    int32_t Mo, No, Kc;
    const uint8_t *sfa;        // atoms [ceil(Mo/128)][chunks][512]
    const uint8_t *sfb;        // atoms [ceil(No/128)][chunks][512]
    int32_t n_atoms_b;         // ceil(No/128)
    uint32_t stage_tx_bytes;   // bytes reported to a stage's barrier (operands + scale-factor atoms)
    uint32_t *status;
    const float *amax_a, *amax_b;   // two-level option: the tensors' magnitude bounds (device); else null
    uint64_t wait_limit_ns;    // bound of every device-side wait
};

template <MmaKind KIND>
struct MxCfg {
    static constexpr bool kNv = KIND == MmaKind::NVF4;
    static constexpr int kChunksPerStage = (KIND == MmaKind::MXF4 || kNv) ? 2 : 1;   // packed FP4: 256 elements per 128-byte row
    static constexpr int kABytes = BM * 128;
    static constexpr int kBBytes = BN * 128;
    // per chunk: SFA 512 + SFB 2 x 512 (+ pad); two-level option: an atom per 64 elements, SFA 2 x 512 + SFB 4 x 512
    static constexpr int kSfChunkBytes = kNv ? 3072 : 2048;
    static constexpr int kSfBytes = kSfChunkBytes * kChunksPerStage;
    static constexpr int kStageBytes = kABytes + kBBytes + kSfBytes;
    static constexpr int kStages = kNv ? 3 : 4;
    static constexpr int kOutStageBytes = kNumEpiWarps * 2048;
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutStageBytes + 256 + 1024;
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

__device__ __forceinline__ void mx_tile_coords(int t, int num_m, int num_n, int &m_idx, int &n_idx)
{
    constexpr int kGroupM = 16;
    const int group_size = kGroupM * num_n;
    const int g = t / group_size;
    const int first_m = g * kGroupM;
    const int gm = min(num_m - first_m, kGroupM);
    const int r = t - g * group_size;
    m_idx = first_m + r % gm;
    n_idx = r / gm;
}

__device__ __forceinline__ uint32_t mx_pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <MmaKind KIND, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_mx_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmO,
               const MxArgs g, const uint32_t idesc)
{
    using C = MxCfg<KIND>;
    constexpr int S = C::kStages;
    constexpr int CPS = C::kChunksPerStage;
    constexpr int HALF = BN / 2;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    auto a_tile = [&](int s) { return smem_base + s * C::kStageBytes; };
    auto b_tile = [&](int s) { return smem_base + s * C::kStageBytes + C::kABytes; };
    auto sf_tile = [&](int s) { return smem_base + s * C::kStageBytes + C::kABytes + C::kBBytes; };
    const uint32_t out_stage0 = smem_base + S * C::kStageBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_gen + S * C::kStageBytes + C::kOutStageBytes);
    const uint32_t bar0 = smem_base + S * C::kStageBytes + C::kOutStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    const uint32_t tfull_bar = bar0 + 8u * (2 * S), tempty_bar = bar0 + 8u * (2 * S + 1);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * S + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_m = (g.Mo + BM - 1) / BM, num_n = (g.No + BN - 1) / BN;
    const int num_tiles = num_m * num_n;
    const int num_chunks = (g.Kc + 127) / 128;
    const int num_kstages = (num_chunks + CPS - 1) / CPS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, kNumEpiWarps);
        *abort_flag = 0u;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        prefetch_tensormap(&tmO);
    }
    if (warp == 1) {
        tmem_alloc<false>(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish<false>();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================= producer: operand tiles and scale-factor atoms =================
        // (whole warp in the loop, one elected lane issues: see the MMA warp)
        {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                int m_idx, n_idx;
                mx_tile_coords(t, num_m, num_n, m_idx, n_idx);
                const int nb0 = 2 * n_idx, nb1 = min(2 * n_idx + 1, g.n_atoms_b - 1);
                for (int ks = 0; ks < num_kstages; ++ks, ++it) {
                    const int s = it % S;
                    if (!__all_sync(0xFFFFFFFFu, mbar_wait(empty_bar(s), ((it / S) & 1u) ^ 1u, abort_flag, g.wait_limit_ns))) { ok = false; break; }
                    if (elect_one()) {
                        mbar_arrive_expect_tx(full_bar(s), g.stage_tx_bytes);
                        tma_load_2d(a_tile(s), &tmA, full_bar(s), ks * 128, m_idx * BM);
                        tma_load_2d(b_tile(s), &tmB, full_bar(s), ks * 128, n_idx * BN);
#pragma unroll
                        for (int h = 0; h < CPS; ++h) {
                            const int c = min(ks * CPS + h, num_chunks - 1);   // a stage's unused second chunk reloads a valid atom
                            const uint32_t dst = sf_tile(s) + h * C::kSfChunkBytes;
                            if (C::kNv) {   // [A: two halves][B rows 0-127: two halves][B rows 128-255: two halves]
                                bulk_load_1d(dst, g.sfa + ((int64_t)m_idx * num_chunks + c) * 1024, 1024, full_bar(s));
                                bulk_load_1d(dst + 1024, g.sfb + ((int64_t)nb0 * num_chunks + c) * 1024, 1024, full_bar(s));
                                bulk_load_1d(dst + 2048, g.sfb + ((int64_t)nb1 * num_chunks + c) * 1024, 1024, full_bar(s));
                            } else {
                                bulk_load_1d(dst, g.sfa + ((int64_t)m_idx * num_chunks + c) * 512, 512, full_bar(s));
                                bulk_load_1d(dst + 512, g.sfb + ((int64_t)nb0 * num_chunks + c) * 512, 512, full_bar(s));
                                bulk_load_1d(dst + 1024, g.sfb + ((int64_t)nb1 * num_chunks + c) * 512, 512, full_bar(s));
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp == 1) {
        // ================= scale-factor copies and MMA issue =================
        // The whole warp walks the loop and one elected lane issues: under `elect.sync` the operands of the tcgen05
        // instructions stay in uniform registers, which makes each of them several times cheaper for the issuing thread than
        // under a `lane == 0` branch; with up to seventeen of them per stage that thread is what the tensor core waits for.
        {
            uint32_t it = 0, tiles_done = 0;
            bool ok = true;
            const uint32_t sfa = tmem_base + kSfaCol, sfb = tmem_base + (C::kNv ? kNvSfbCol : kSfbCol);
            auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag, g.wait_limit_ns)); };
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tiles_done) {
                // the single accumulator must have been drained by the epilogue of the previous tile
                if (!wait_all(tempty_bar, (tiles_done & 1u) ^ 1u)) { ok = false; break; }
                tc_fence_after_sync();
                for (int ks = 0; ks < num_kstages && ok; ++ks, ++it) {
                    const int s = it % S;
                    if (!wait_all(full_bar(s), (it / S) & 1u)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t adesc = make_smem_desc_k128(a_tile(s));
                    const uint64_t bdesc = make_smem_desc_k128(b_tile(s));
                    if (elect_one()) {
#pragma unroll
                        for (int h = 0; h < CPS; ++h) {
                            if (ks * CPS + h < num_chunks) {
                                const uint32_t sf = sf_tile(s) + h * C::kSfChunkBytes;
                                if (C::kNv) {
                                    // MMA k of the chunk reads a whole word per line: SFA columns 4k.., SFB columns 8k.. (two 128-line groups)
                                    tmem_cp_sf_atom(sfa, sf);             tmem_cp_sf_atom(sfa + 4, sf + 512);
                                    tmem_cp_sf_atom(sfb, sf + 1024);      tmem_cp_sf_atom(sfb + 8, sf + 1536);
                                    tmem_cp_sf_atom(sfb + 4, sf + 2048);  tmem_cp_sf_atom(sfb + 12, sf + 2560);
                                } else {
                                    tmem_cp_sf_atom(sfa, sf);
                                    tmem_cp_sf_atom(sfb, sf + 512);
                                    tmem_cp_sf_atom(sfb + 4, sf + 1024);
                                }
                                constexpr int kMmas = 4 / CPS;   // 32 bytes of K per MMA: four per 128-byte row
#pragma unroll
                                for (int k = 0; k < kMmas; ++k) {
                                    const int kk = h * kMmas + k;
                                    // which of the line's four scale bytes this MMA applies: byte k for the 32-long blocks of
                                    // kind::mxf8f6f4, bytes 2k and 2k+1 for the two halves of kind::mxf4's 64-long step
                                    // (descriptor fields b_sf_id at bit 4, a_sf_id at bit 29); the two-level option reads whole words
                                    const uint32_t sf_id = C::kNv ? 0u : (KIND == MmaKind::MXF4) ? 2u * k : (uint32_t)k;
                                    mma_ss<KIND, false>(tmem_base, adesc + 2 * kk, bdesc + 2 * kk, idesc | (sf_id << 4) | (sf_id << 29),
                                                        (ks > 0 || kk > 0) ? 1u : 0u, sfa + (C::kNv ? 4 * k : 0), sfb + (C::kNv ? 8 * k : 0));
                                }
                            }
                        }
                        tc_commit<false>(empty_bar(s));
                        if (ks == num_kstages - 1) tc_commit<false>(tfull_bar);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp >= 4) {
        // ================= epilogue: drain, round, store =================
        const int e = warp - 4, q = warp & 3, h = e >> 2;
        const uint32_t stage_u32 = out_stage0 + e * 2048;
        uint32_t tiles_done = 0;
        bool ok = true;
        // two-level option: the sums carry both tensors' factors 2688 / bound; they are divided out here, once per output
        float out_scale = 1.0f;
        if (C::kNv) {
            const float ba = *g.amax_a, bb = *g.amax_b;
            const float ea = ba == 0.0f ? 1.0f : fminf(__fdiv_rn(2688.0f, ba), FLT_MAX), eb = bb == 0.0f ? 1.0f : fminf(__fdiv_rn(2688.0f, bb), FLT_MAX);
            out_scale = __fdiv_rn(1.0f, ea * eb);
        }
        for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tiles_done) {
            int m_idx, n_idx;
            mx_tile_coords(t, num_m, num_n, m_idx, n_idx);
            const int row0 = m_idx * BM + q * 32;
            const int col0 = n_idx * BN + h * HALF;
            const bool got = mbar_wait(tfull_bar, tiles_done & 1u, abort_flag, g.wait_limit_ns);
            if (!__all_sync(0xFFFFFFFFu, got)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + h * HALF;
            uint32_t v[4][32];
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) tmem_ld32(taddr + 32 * gi, v[gi]);
            tmem_ld_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);   // the next tile's MMAs may start
            if (C::kNv) {
#pragma unroll
                for (int gi = 0; gi < 4; ++gi)
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[gi][i] = __float_as_uint(__uint_as_float(v[gi][i]) * out_scale);
            }
            constexpr int kPerBox = OUT_F32 ? 16 : 32;   // output columns per 64-byte box row
#pragma unroll
            for (int b = 0; b < HALF / kPerBox; ++b) {
                if (lane == 0) bulk_wait_read0();
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 o;
                    if (OUT_F32) {
                        const uint32_t *src = &v[(b * 16) / 32][(b * 16) % 32 + 4 * j];
                        o = make_uint4(src[0], src[1], src[2], src[3]);
                    } else {
                        const uint32_t *src = &v[b][8 * j];
                        o = make_uint4(mx_pack_bf16x2(__uint_as_float(src[0]), __uint_as_float(src[1])), mx_pack_bf16x2(__uint_as_float(src[2]), __uint_as_float(src[3])),
                                       mx_pack_bf16x2(__uint_as_float(src[4]), __uint_as_float(src[5])), mx_pack_bf16x2(__uint_as_float(src[6]), __uint_as_float(src[7])));
                    }
                    st_shared_v4(stage_u32 + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4), o);
                }
                fence_proxy_async();
                __syncwarp();
                const int col = col0 + b * kPerBox;
                if (lane == 0 && col < g.No && row0 < g.Mo) { tma_store_2d(&tmO, stage_u32, col, row0); bulk_commit(); }
            }
        }
        if (lane == 0) bulk_wait_all0();
    }

    // ---- teardown ----
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        if (threadIdx.x == 0) atomicExch(g.status, (uint32_t)SNIP_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc<false>(tmem_base, kTmemCols);
    }
}


template <MmaKind KIND, bool OUT_F32>
int launch_mx(const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmO, const MxArgs &g, uint32_t idesc, int sms, cudaStream_t st)
{
    using C = MxCfg<KIND>;
    auto kern = gemm_mx_kernel<KIND, OUT_F32>;
    // a per-function, per-device attribute; setting it on every launch is cheap and correct on any device
    SNIP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
    const int num_tiles = (int)(ceil_div(g.Mo, BM) * ceil_div(g.No, BN));
    const int grid = num_tiles < sms ? num_tiles : sms;
    kern<<<grid, kThreads, C::kSmemBytes, st>>>(tmA, tmB, tmO, g, idesc);
    SNIP_CUDA_TRY(cudaGetLastError());
    return SNIP_OK;
}

}  // namespace

int make_tiled_map_2d(CUtensorMap *map, const void *ptr, int dtype, int64_t rows, int64_t inner_elems, int64_t row_bytes, int box_x_elems,
                      int box_rows, int swizzle);
int gemm_clear_status(void *ws, cudaStream_t st);
int gemm_sm_count();
void gemm_debug_hooks(uint64_t *wait_limit_ns, int *tx_skew);   // testing hooks of snip_debug_set (gemm.cu)

// a_codes [Mo][Kc], b_codes [No][Kc] contraction-major; sfa / sfb: UE8M0 atoms [line tile][chunk][512].
int gemm_mx_impl(int fmt_a, int fmt_b, const void *a_codes, const void *b_codes, const void *sfa, const void *sfb, int64_t Mo, int64_t No,
                 int64_t Kc, void *out, int out_dtype, void *ws, size_t ws_bytes, cudaStream_t st, bool clear_status)
{
    if (!a_codes || !b_codes || !sfa || !sfb || !out) return SNIP_ERR_ARG;
    if (!valid_dim(Mo) || !valid_dim(No) || !valid_dim(Kc) || Mo > INT32_MAX || No > INT32_MAX || Kc > INT32_MAX) return SNIP_ERR_SHAPE;
    if (out_dtype != SNIP_OUT_BF16 && out_dtype != SNIP_OUT_FP32) return SNIP_ERR_ARG;
    if (fmt_a == SNIP_FMT_BF16 || fmt_b == SNIP_FMT_BF16) return SNIP_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < 256) return SNIP_ERR_WORKSPACE;
    if (!aligned16(a_codes) || !aligned16(b_codes) || !aligned16(sfa) || !aligned16(sfb) || !aligned16(out) || !aligned16(ws)) return SNIP_ERR_ALIGN;
    int rc = require_sm100();
    if (rc != SNIP_OK) return rc;
    if (clear_status) { rc = gemm_clear_status(ws, st); if (rc) return rc; }   // see gemm_impl
    const bool f32 = out_dtype == SNIP_OUT_FP32;
    const bool a4 = fmt_a == SNIP_FMT_FP4_E2M1, b4 = fmt_b == SNIP_FMT_FP4_E2M1;

    MxArgs g;
    g.Mo = (int32_t)Mo; g.No = (int32_t)No; g.Kc = (int32_t)Kc;
    g.sfa = static_cast<const uint8_t *>(sfa);
    g.sfb = static_cast<const uint8_t *>(sfb);
    g.n_atoms_b = (int32_t)ceil_div(No, 128);
    g.status = static_cast<uint32_t *>(ws);
    int tx_skew = 0;
    gemm_debug_hooks(&g.wait_limit_ns, &tx_skew);
    g.amax_a = g.amax_b = nullptr;

    CUtensorMap tmA, tmB, tmO;
    rc = f32 ? make_tiled_map_2d(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Mo, No, No * 4, 16, 32, CU_TENSOR_MAP_SWIZZLE_64B)
             : make_tiled_map_2d(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Mo, No, No * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    if (rc) return rc;
    const int sms = gemm_sm_count();
    if (a4 && b4) {
        // packed FP4: kind::mxf4, 256 elements per 128-byte row, two scale chunks per stage
        rc = make_tiled_map_2d(&tmA, a_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, Kc / 2, Kc / 2, 128, BM, CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        rc = make_tiled_map_2d(&tmB, b_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, No, Kc / 2, Kc / 2, 128, BN, CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        g.stage_tx_bytes = (BM + BN) * 128 + 2 * 1536 + tx_skew;
        const uint32_t idesc = make_idesc_block_scaled(1, 1, BM, BN);
        return f32 ? launch_mx<MmaKind::MXF4, true>(tmA, tmB, tmO, g, idesc, sms, st) : launch_mx<MmaKind::MXF4, false>(tmA, tmB, tmO, g, idesc, sms, st);
    }
    const int64_t kpad = ceil_div(Kc, 128) * 128;   // see gemm.cu: the expanding 4-bit map wants a multiple of 128
    rc = make_tiled_map_2d(&tmA, a_codes, a4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, a4 ? kpad : Kc,
                           a4 ? Kc / 2 : Kc, 128, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tiled_map_2d(&tmB, b_codes, b4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, No, b4 ? kpad : Kc,
                           b4 ? Kc / 2 : Kc, 128, BN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    g.stage_tx_bytes = BM * (a4 ? 64 : 128) + BN * (b4 ? 64 : 128) + 1536 + tx_skew;
    const uint32_t idesc = make_idesc_block_scaled(a4 ? 5 : 0, b4 ? 5 : 0, BM, BN);
    return f32 ? launch_mx<MmaKind::MXF8, true>(tmA, tmB, tmO, g, idesc, sms, st) : launch_mx<MmaKind::MXF8, false>(tmA, tmB, tmO, g, idesc, sms, st);
}

// Two-level option: packed E2M1 codes, E4M3 scale bytes per 16-long tile as atoms [line tile][chunk][half][512], and the
// two tensors' magnitude bounds (device pointers).  out = (sum of block-scaled products) / (enc_a * enc_b), enc = 2688 / bound.
int gemm_nvfp4_impl(const void *a_codes, const void *b_codes, const void *sfa, const void *sfb, const float *amax_a, const float *amax_b,
                    int64_t Mo, int64_t No, int64_t Kc, void *out, int out_dtype, void *ws, size_t ws_bytes, cudaStream_t st, bool clear_status)
{
    if (!a_codes || !b_codes || !sfa || !sfb || !amax_a || !amax_b || !out) return SNIP_ERR_ARG;
    if (!valid_dim(Mo) || !valid_dim(No) || !valid_dim(Kc) || Mo > INT32_MAX || No > INT32_MAX || Kc > INT32_MAX) return SNIP_ERR_SHAPE;
    if (out_dtype != SNIP_OUT_BF16 && out_dtype != SNIP_OUT_FP32) return SNIP_ERR_ARG;
    if (!ws || ws_bytes < 256) return SNIP_ERR_WORKSPACE;
    if (!aligned16(a_codes) || !aligned16(b_codes) || !aligned16(sfa) || !aligned16(sfb) || !aligned16(out) || !aligned16(ws)) return SNIP_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(amax_a) & 3u) || (reinterpret_cast<uintptr_t>(amax_b) & 3u)) return SNIP_ERR_ALIGN;
    int rc = require_sm100();
    if (rc != SNIP_OK) return rc;
    if (clear_status) { rc = gemm_clear_status(ws, st); if (rc) return rc; }
    const bool f32 = out_dtype == SNIP_OUT_FP32;
    MxArgs g;
    g.Mo = (int32_t)Mo; g.No = (int32_t)No; g.Kc = (int32_t)Kc;
    g.sfa = static_cast<const uint8_t *>(sfa);
    g.sfb = static_cast<const uint8_t *>(sfb);
    g.n_atoms_b = (int32_t)ceil_div(No, 128);
    g.status = static_cast<uint32_t *>(ws);
    int tx_skew = 0;
    gemm_debug_hooks(&g.wait_limit_ns, &tx_skew);
    g.amax_a = amax_a; g.amax_b = amax_b;
    CUtensorMap tmA, tmB, tmO;
    rc = f32 ? make_tiled_map_2d(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Mo, No, No * 4, 16, 32, CU_TENSOR_MAP_SWIZZLE_64B)
             : make_tiled_map_2d(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Mo, No, No * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    if (rc) return rc;
    rc = make_tiled_map_2d(&tmA, a_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, Kc / 2, Kc / 2, 128, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tiled_map_2d(&tmB, b_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, No, Kc / 2, Kc / 2, 128, BN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    g.stage_tx_bytes = (BM + BN) * 128 + 2 * 3072 + tx_skew;
    const uint32_t idesc = make_idesc_block_scaled_e4m3(1, 1, BM, BN);
    const int sms = gemm_sm_count();
    return f32 ? launch_mx<MmaKind::NVF4, true>(tmA, tmB, tmO, g, idesc, sms, st) : launch_mx<MmaKind::NVF4, false>(tmA, tmB, tmO, g, idesc, sms, st);
}

}  // namespace snip

// A quantized operand of the power-of-two option: codes as in snip_qtensor_t plus its UE8M0 atoms.
extern "C" int snip_gemm_mx(int op, const snip_qtensor_t *a, const void *sf_a, const snip_qtensor_t *b, const void *sf_b, void *out,
                            int out_dtype, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!a || !b || op < SNIP_OP_FWD || op > SNIP_OP_WGRAD) return SNIP_ERR_ARG;
    if (!valid_fmt(a->fmt) || !valid_fmt(b->fmt)) return SNIP_ERR_ARG;
    int64_t Mo, No, Kc;
    if (op == SNIP_OP_FWD) {
        if (a->cols != b->cols || a->transposed || b->transposed) return SNIP_ERR_SHAPE;
        // the paper's tiles, or 32-long tiles along the contraction on both sides
        if (!((a->block == SNIP_BLOCK_ROW_1x128 && b->block == SNIP_BLOCK_BLK_128x128) || (a->block == SNIP_BLOCK_ROW_1x32 && b->block == SNIP_BLOCK_ROW_1x32)))
            return SNIP_ERR_UNSUPPORTED;
        Mo = a->rows; No = b->rows; Kc = a->cols;
    } else if (op == SNIP_OP_DGRAD) {
        if (a->cols != b->rows || a->transposed || !b->transposed) return SNIP_ERR_SHAPE;
        if (!((a->block == SNIP_BLOCK_ROW_1x128 && b->block == SNIP_BLOCK_BLK_128x128) || (a->block == SNIP_BLOCK_ROW_1x32 && b->block == SNIP_BLOCK_COL_32x1)))
            return SNIP_ERR_UNSUPPORTED;
        Mo = a->rows; No = b->cols; Kc = a->cols;
    } else {
        if (a->rows != b->rows || !a->transposed || !b->transposed) return SNIP_ERR_SHAPE;
        if (!((a->block == SNIP_BLOCK_COL_128x1 && b->block == SNIP_BLOCK_COL_128x1) || (a->block == SNIP_BLOCK_COL_32x1 && b->block == SNIP_BLOCK_COL_32x1)))
            return SNIP_ERR_UNSUPPORTED;
        Mo = a->cols; No = b->cols; Kc = a->rows;
    }
    return gemm_mx_impl(a->fmt, b->fmt, a->codes, b->codes, sf_a, sf_b, Mo, No, Kc, out, out_dtype, ws, ws_bytes, static_cast<cudaStream_t>(stream), true);
}

extern "C" int snip_gemm_nvfp4(int op, const snip_qtensor_t *a, const void *sf_a, const float *amax_a, const snip_qtensor_t *b, const void *sf_b,
                               const float *amax_b, void *out, int out_dtype, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!a || !b || op < SNIP_OP_FWD || op > SNIP_OP_WGRAD) return SNIP_ERR_ARG;
    if (a->fmt != SNIP_FMT_FP4_E2M1 || b->fmt != SNIP_FMT_FP4_E2M1) return SNIP_ERR_UNSUPPORTED;
    int64_t Mo, No, Kc;
    if (op == SNIP_OP_FWD) {
        if (a->cols != b->cols || a->transposed || b->transposed) return SNIP_ERR_SHAPE;
        if (a->block != SNIP_BLOCK_ROW_1x16 || b->block != SNIP_BLOCK_ROW_1x16) return SNIP_ERR_UNSUPPORTED;
        Mo = a->rows; No = b->rows; Kc = a->cols;
    } else if (op == SNIP_OP_DGRAD) {
        if (a->cols != b->rows || a->transposed || !b->transposed) return SNIP_ERR_SHAPE;
        if (a->block != SNIP_BLOCK_ROW_1x16 || b->block != SNIP_BLOCK_COL_16x1) return SNIP_ERR_UNSUPPORTED;
        Mo = a->rows; No = b->cols; Kc = a->cols;
    } else {
        if (a->rows != b->rows || !a->transposed || !b->transposed) return SNIP_ERR_SHAPE;
        if (a->block != SNIP_BLOCK_COL_16x1 || b->block != SNIP_BLOCK_COL_16x1) return SNIP_ERR_UNSUPPORTED;
        Mo = a->cols; No = b->cols; Kc = a->rows;
    }
    return gemm_nvfp4_impl(a->codes, b->codes, sf_a, sf_b, amax_a, amax_b, Mo, No, Kc, out, out_dtype, ws, ws_bytes, static_cast<cudaStream_t>(stream), true);
}
