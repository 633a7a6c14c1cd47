// Block-scaled GEMM with the paper's FP32 tile scales, CTA-pair form:  out[Mo,No] = A[Mo,Kc] . B[No,Kc]^T,
// both operands contraction-major, each 128-long chunk of the contraction multiplied on the tensor
// cores into its own tensor-memory buffer and then scaled by 1/(S_a*S_b) and added into FP32 register
// accumulators (Sec. 2.3: the operator's output is divided by the scales that were multiplied in;
// Fig. 5: the three GEMMs of a linear layer).
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one tcgen05.mma.cta_group::2: the tile is
// 256 rows x 128 columns, each CTA holds 128 rows of A, 64 rows of B and a 128 x 128 slice of the
// accumulator.  That slice is only a quarter of the register file, which leaves room for SIXTEEN
// promotion warps (four per scheduler) - the FP32 multiply-adds of the promotion, not the tensor
// pipe, set the pace of these kernels - and its tensor-memory image is 128 columns, so three or four
// chunks can be in flight between the MMA issuer and the promotion warps.
//
// Roles in one CTA (640 threads):
//   warp 0      : TMA producer  - this CTA's halves of the operand tiles into a shared-memory ring;
//                                 byte counts are reported to the leader's barrier (no multicast)
//   warp 1      : MMA issuer    - leader CTA only, one thread; owns the tensor-memory allocation
//   warp 2 (,3) : scale loader  - reads the chunk's scale factors from global memory some chunks
//                                 ahead, turns them into reciprocal factors and leaves them in a
//                                 shared-memory ring (warp 3: the per-column factors of wgrad)
//   warps 4..19 : promotion     - 32 rows x 32 columns each
// Every wait is bounded; on a timeout both CTAs leave cleanly and a status word is raised.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "sm100.cuh"

namespace snip {

using namespace sm100;

int make_tiled_map_2d(CUtensorMap *map, const void *ptr, int dtype, int64_t rows, int64_t inner_elems, int64_t row_bytes, int box_x_elems,
                      int box_rows, int swizzle);

namespace {

constexpr int kThreads = 640;
constexpr int kEpiWarps = 16;
constexpr int CM = 128;       // rows of A / of the accumulator per CTA
constexpr int TM = 2 * CM;    // rows of one tile (CTA pair)
constexpr int TN = 128;       // columns of one tile = one 128-wide scale block of B
constexpr int kBRows = TN / 2;  // rows of B held by one CTA
constexpr int kSD = 16;       // depth of the scale-factor ring, in chunks
constexpr int kSlotFloats = 256;   // per chunk: [0,128) row factors of this CTA, [128,256) column factors (wgrad)
constexpr int kSfCols = 32;   // tensor-memory columns of constant scale factors (kind::mxf4)

enum { PSCALE_BLOCK_B = 1, PSCALE_VEC_B = 2 };

struct PairArgs {
    int32_t Mo, No, Kc;
    const float *sa;           // A scales [chunks][Mo]
    int64_t sa_chunk_stride;
    const float *sb;           // B scales: block mode [blk*sb_blk_stride + chunk*sb_chunk_stride], vector mode [chunk*sb_chunk_stride + n]
    int64_t sb_chunk_stride;
    int64_t sb_blk_stride;
    void *out;
    int64_t ldo;
    int32_t accumulate;
    uint32_t stage_tx_bytes;   // bytes the two TMA loads of ONE CTA report per stage
    uint64_t wait_limit_ns;    // bound of every device-side wait
    uint32_t *status;
};

template <MmaKind KIND>
struct PCfg {
    static constexpr int kCPS = (KIND == MmaKind::MXF4) ? 2 : 1;       // 128-long chunks per shared-memory stage
    static constexpr int kNBuf = (KIND == MmaKind::MXF4) ? 3 : 4;      // accumulator buffers in tensor memory
    static constexpr int kStages = (KIND == MmaKind::MXF4) ? 5 : 6;
    static constexpr int kABytes = CM * 128;
    static constexpr int kBBytes = kBRows * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kRingBytes = kSD * kSlotFloats * 4;
    static constexpr int kOutBytes = kEpiWarps * 2048;                 // per-warp staging tile: 32 rows x 64 bytes
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = kStages * kStageBytes + kRingBytes + kOutBytes + kBarBytes + 1024;
    static constexpr int kSfCol0 = kNBuf * TN;
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    static_assert(kNBuf * TN + (KIND == MmaKind::MXF4 ? kSfCols : 0) <= 512, "tensor memory budget");
    // A ring slot is rewritten once the stage of its new chunk is free again; by then the promotion warps have
    // released the buffer of a chunk at most kStages*kCPS + kCPS + kNBuf older, i.e. finished reading its slot.
    static_assert(kSD >= kStages * kCPS + kCPS + kNBuf, "scale ring too shallow for the implicit slot hand-back");
    static_assert((2 * kStages + 2 * kNBuf + kSD) * 8 + 8 <= kBarBytes, "barrier area");
};

__device__ __forceinline__ void pair_tile_coords(int t, int num_m, int num_n, int &m_idx, int &n_idx)
{
    // groups of 8 row-tiles (2048 rows) share their B panels in L2 while they are resident together
    constexpr int kGroupM = 8;
    const int group_size = kGroupM * num_n;
    const int g = t / group_size;
    const int first_m = g * kGroupM;
    const int gm = min(num_m - first_m, kGroupM);
    const int r = t - g * group_size;
    m_idx = first_m + r % gm;
    n_idx = r / gm;
}

__device__ __forceinline__ float rcp_fast(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ uint32_t bf16x2_bits(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <MmaKind KIND, int SCALE, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmO,
                 const PairArgs g, const uint32_t idesc)
{
    using C = PCfg<KIND>;
    constexpr int S = C::kStages, NB = C::kNBuf, CPS = C::kCPS;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // operand tiles: 1024-byte aligned (128-byte swizzle)
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t smem_a0 = smem_base;
    const uint32_t smem_b0 = smem_base + S * C::kABytes;
    float *ring = reinterpret_cast<float *>(smem_gen + S * C::kStageBytes);
    const uint32_t out_stage0 = smem_base + S * C::kStageBytes + C::kRingBytes;
    const uint32_t bar0 = out_stage0 + C::kOutBytes;
    uint8_t *bar_gen = smem_gen + S * C::kStageBytes + C::kRingBytes + C::kOutBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };                      // leader: operand bytes of both CTAs have landed
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };               // each CTA: the MMAs reading stage s are done
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * S + b); };           // each CTA: buffer b holds a chunk's partial sums
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * S + NB + b); };     // leader: all 32 promotion warps have drained buffer b
    auto sfull_bar = [&](int d) { return bar0 + 8u * (2 * S + 2 * NB + d); };  // each CTA: ring slot d holds a chunk's factors
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_gen + 8 * (2 * S + 2 * NB + kSD));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();   // 0 = leader
    const int num_m = (g.Mo + TM - 1) / TM, num_n = (g.No + TN - 1) / TN;
    const int num_tiles = num_m * num_n;
    const int first_tile = (int)(blockIdx.x >> 1), tile_step = (int)(gridDim.x >> 1);
    const int nacc = (g.Kc + 127) / 128;                    // chunks per tile
    const int num_kstages = (nacc + CPS - 1) / CPS;
    const uint64_t limit = g.wait_limit_ns;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < NB; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 2 * kEpiWarps); }
        for (int d = 0; d < kSD; ++d) mbar_init(sfull_bar(d), SCALE == PSCALE_VEC_B ? 2 : 1);
        *abort_flag = 0u;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        prefetch_tensormap(&tmO);
    }
    if (warp == 1) {
        tmem_alloc<true>(smem_u32(tmem_slot), 512);
        tmem_relinquish<true>();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (KIND == MmaKind::MXF4) {
        // constant scale factors 2^0 (UE8M0 byte 127) for every row of A and B, in both CTAs
        if (warp >= 4 && warp < 8) {
            const uint32_t q = warp & 3;
            for (int c = 0; c < kSfCols; ++c) tmem_st1(tmem_base + ((q * 32u) << 16) + C::kSfCol0 + c, 0x7F7F7F7Fu);
            tmem_st_wait();
        }
        tc_fence_before_sync();
        __syncthreads();
    }
    cluster_sync();   // both CTAs' barriers and tensor memory exist before anyone signals across the pair
    tc_fence_after_sync();

    // Raise the abort flag of both CTAs (the other CTA's waits then fall through at their next check).
    auto abort_pair = [&]() {
        *abort_flag = 1u;
        st_cluster_u32(mapa(smem_u32(const_cast<uint32_t *>(abort_flag)), rank ^ 1u), 1u);
    };
    auto wait = [&](uint32_t bar, uint32_t parity) {
        const bool got = mbar_wait(bar, parity, abort_flag, limit);
        if (!got) abort_pair();
        return got;
    };

    if (warp == 0) {
        // ================= TMA producer (both CTAs) =================
        if (lane == 0) {
            uint32_t it = 0, cs = 0;
            bool ok = true;
            const uint32_t lead_full0 = mapa(full_bar(0), 0);
            for (int t = first_tile; t < num_tiles && ok; t += tile_step) {
                int m_idx, n_idx;
                pair_tile_coords(t, num_m, num_n, m_idx, n_idx);
                for (int ks = 0; ks < num_kstages; ++ks, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1u;
                    if (!wait(empty_bar(s), ph ^ 1u)) { ok = false; break; }
                    // The factors of this stage's chunks are in the ring before its operands are requested, so a
                    // promotion warp that sees the chunk's partial sums complete may read them without a wait of its own.
                    const int here = min(CPS, nacc - ks * CPS);
                    for (int h = 0; h < here && ok; ++h, ++cs) ok = wait(sfull_bar(cs % kSD), (cs / kSD) & 1u);
                    if (!ok) break;
                    if (rank == 0) mbar_arrive_expect_tx(full_bar(s), 2u * g.stage_tx_bytes);
                    tma_load_2d_pair(smem_a0 + s * C::kABytes, &tmA, lead_full0 + 8u * s, ks * 128, m_idx * TM + (int)rank * CM);
                    tma_load_2d_pair(smem_b0 + s * C::kBBytes, &tmB, lead_full0 + 8u * s, ks * 128, n_idx * TN + (int)rank * kBRows);
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (leader only) =================
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, cc = 0;
            bool ok = true;
            const uint32_t sfa = tmem_base + C::kSfCol0, sfb = tmem_base + C::kSfCol0 + 16;
            // completion of everything issued so far, signalled to the same barrier of both CTAs
            auto commit_both = [&](uint32_t bar) {
                tc_commit<true>(bar);
                tc_commit<true>(mapa(bar, 1));
            };
            for (int t = first_tile; t < num_tiles && ok; t += tile_step) {
                for (int ks = 0; ks < num_kstages && ok; ++ks, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1u;
                    if (!wait(full_bar(s), ph)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t adesc = make_smem_desc_k128(smem_a0 + s * C::kABytes);
                    const uint64_t bdesc = make_smem_desc_k128(smem_b0 + s * C::kBBytes);
#pragma unroll
                    for (int h = 0; h < CPS; ++h) {
                        if (ks * CPS + h < nacc) {
                            const uint32_t b = cc % NB;
                            if (!wait(tempty_bar(b), ((cc / NB) & 1u) ^ 1u)) { ok = false; break; }
                            tc_fence_after_sync();
                            constexpr int kPerChunk = 4 / CPS;   // 32-byte K steps per chunk
#pragma unroll
                            for (int k = 0; k < kPerChunk; ++k)
                                mma_ss<KIND, true>(tmem_base + b * TN, adesc + 2 * (kPerChunk * h + k), bdesc + 2 * (kPerChunk * h + k), idesc,
                                                   k > 0 ? 1u : 0u, sfa, sfb);
                            commit_both(tfull_bar(b));
                            ++cc;
                        }
                    }
                    if (ok) commit_both(empty_bar(s));
                }
            }
        }
    } else if (warp == 2 || warp == 3) {
        // ================= scale loaders =================
        // warp 2: factors of this CTA's 128 rows; block mode: 1/(S_a*S_b), vector mode: 1/S_a.
        // warp 3 (vector mode only): 1/S_b of the tile's 128 columns.
        const bool rows_side = (warp == 2);
        if (rows_side || SCALE == PSCALE_VEC_B) {
            constexpr int PD = 4;        // chunks whose global loads are in flight in registers
            float4 qv[PD];
            float qb[PD];
            int pt = first_tile, pj = 0;   // tile and chunk of the next load to issue
            auto issue = [&](float4 &dv, float &db) {
                dv = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
                db = 1.0f;
                if (pt < num_tiles) {
                    int m_idx, n_idx;
                    pair_tile_coords(pt, num_m, num_n, m_idx, n_idx);
                    if (rows_side) {
                        // rows outside the matrix repeat the last four rows' factors (their sums are never stored)
                        const int r = min(m_idx * TM + (int)rank * CM + 4 * lane, g.Mo - 4);
                        dv = __ldg(reinterpret_cast<const float4 *>(g.sa + (int64_t)pj * g.sa_chunk_stride + r));
                        if (SCALE == PSCALE_BLOCK_B) db = __ldg(g.sb + (int64_t)n_idx * g.sb_blk_stride + (int64_t)pj * g.sb_chunk_stride);
                    } else {
                        const int c = min(n_idx * TN + 4 * lane, g.No - 4);
                        dv = __ldg(reinterpret_cast<const float4 *>(g.sb + (int64_t)pj * g.sb_chunk_stride + c));
                    }
                    if (++pj == nacc) { pj = 0; pt += tile_step; }
                }
            };
#pragma unroll
            for (int u = 0; u < PD; ++u) issue(qv[u], qb[u]);
            // Chunks are walked as one sequence over all of this pair's tiles, PD at a time, so that the register
            // slot of a chunk is a compile-time index (a run-time choice among the slots would wait for every load
            // in flight, not only for the chunk's own).
            const int my_tiles = first_tile < num_tiles ? (num_tiles - first_tile + tile_step - 1) / tile_step : 0;
            const uint32_t total = (uint32_t)my_tiles * (uint32_t)nacc;
            uint32_t it_base = 0;   // first stage of the tile being consumed
            int cj = 0;             // chunk within that tile
            bool ok = true;
            for (uint32_t c0 = 0; c0 < total && ok; c0 += PD) {
#pragma unroll
                for (int u = 0; u < PD; ++u) {
                    const uint32_t cc = c0 + u;
                    if (cc < total && ok) {
                        const float4 v = qv[u];
                        const float bsc = qb[u];
                        issue(qv[u], qb[u]);   // chunk cc + PD
                        float4 r;
                        r.x = rcp_fast(v.x * bsc); r.y = rcp_fast(v.y * bsc); r.z = rcp_fast(v.z * bsc); r.w = rcp_fast(v.w * bsc);
                        // the slot is free once the stage this chunk travels in is free (see PCfg)
                        const uint32_t its = it_base + (uint32_t)(cj / CPS);
                        if (!wait(empty_bar(its % S), ((its / S) & 1u) ^ 1u)) { ok = false; }
                        else {
                            const uint32_t d = cc % kSD;
                            *reinterpret_cast<float4 *>(ring + d * kSlotFloats + (rows_side ? 0 : 128) + 4 * lane) = r;
                            __syncwarp();
                            if (lane == 0) mbar_arrive(sfull_bar(d));
                            if (++cj == nacc) { cj = 0; it_base += (uint32_t)num_kstages; }
                        }
                    }
                }
            }
        }
    } else {
        // ================= promotion / epilogue warps =================
        const int e = warp - 4;          // 0..15
        const int q = warp & 3;          // tensor-memory lane quarter this warp may access (= e & 3)
        const int cg = e >> 2;           // 32-column group
        const uint32_t stage_u32 = out_stage0 + e * 2048;
        const uint32_t tempty_lead0 = mapa(tempty_bar(0), 0);
        uint32_t cc = 0;
        bool ok = true;
        for (int t = first_tile; t < num_tiles && ok; t += tile_step) {
            int m_idx, n_idx;
            pair_tile_coords(t, num_m, num_n, m_idx, n_idx);
            const int row0 = m_idx * TM + (int)rank * CM + q * 32;
            const int row = row0 + lane;
            const int col0 = n_idx * TN + cg * 32;
            float2 acc[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = make_float2(0.0f, 0.0f);
            for (int j = 0; j < nacc; ++j, ++cc) {
                const uint32_t b = cc % NB;
                const float *slot = ring + (cc % kSD) * kSlotFloats;
                {
                    const bool got = wait(tfull_bar(b), (cc / NB) & 1u);
                    if (!__all_sync(0xFFFFFFFFu, got)) { ok = false; break; }
                }
                tc_fence_after_sync();
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + b * TN + cg * 32, v);
                const float f = slot[q * 32 + lane];   // in the shadow of the load
                tmem_ld_wait();
                // this warp's reads of buffer b are done: hand it back to the MMA issuer
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(tempty_lead0 + 8u * b);
                const float2 ff = make_float2(f, f);
                if (SCALE == PSCALE_BLOCK_B) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        acc[i] = __ffma2_rn(make_float2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), ff, acc[i]);
                } else {
                    const float4 *cf = reinterpret_cast<const float4 *>(slot + 128 + cg * 32);   // reciprocal column scales, broadcast reads
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 s4 = cf[i];
                        const float2 p0 = __fmul2_rn(make_float2(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1])), make_float2(s4.x, s4.y));
                        const float2 p1 = __fmul2_rn(make_float2(__uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3])), make_float2(s4.z, s4.w));
                        acc[2 * i] = __ffma2_rn(p0, ff, acc[2 * i]);
                        acc[2 * i + 1] = __ffma2_rn(p1, ff, acc[2 * i + 1]);
                    }
                }
            }
            if (!ok) break;
            const float *av = reinterpret_cast<const float *>(acc);
            if (!g.accumulate) {
                // round, stage 32 rows x 64 bytes (16-byte pieces XOR-swizzled as the output map's 64-byte swizzle
                // expects) and let the TMA unit write the box; parts outside the matrix are clipped by the hardware
                constexpr int kPerBox = OUT_F32 ? 16 : 32;
#pragma unroll
                for (int bx = 0; bx < 32 / kPerBox; ++bx) {
                    if (lane == 0) bulk_wait_read0();     // the previous box has left the staging tile
                    __syncwarp();
                    const float *src = av + bx * kPerBox;
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        uint4 o;
                        if (OUT_F32) o = make_uint4(__float_as_uint(src[4 * p]), __float_as_uint(src[4 * p + 1]), __float_as_uint(src[4 * p + 2]), __float_as_uint(src[4 * p + 3]));
                        else o = make_uint4(bf16x2_bits(src[8 * p], src[8 * p + 1]), bf16x2_bits(src[8 * p + 2], src[8 * p + 3]),
                                            bf16x2_bits(src[8 * p + 4], src[8 * p + 5]), bf16x2_bits(src[8 * p + 6], src[8 * p + 7]));
                        st_shared_v4(stage_u32 + lane * 64 + ((p ^ ((lane >> 1) & 3)) << 4), o);
                    }
                    fence_proxy_async();
                    __syncwarp();
                    const int col = col0 + bx * kPerBox;
                    if (lane == 0 && col < g.No && row0 < g.Mo) { tma_store_2d(&tmO, stage_u32, col, row0); bulk_commit(); }
                }
            } else if (row < g.Mo) {
                // FP32 accumulation into the existing output (gradient accumulation)
                float *dst = static_cast<float *>(g.out) + (int64_t)row * g.ldo + col0;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    if (col0 + i < g.No) {
                        float4 o = *reinterpret_cast<const float4 *>(dst + i);
                        o.x += av[i]; o.y += av[i + 1]; o.z += av[i + 2]; o.w += av[i + 3];
                        *reinterpret_cast<float4 *>(dst + i) = o;
                    }
                }
            }
            __syncwarp();
        }
        if (lane == 0) bulk_wait_all0();   // outstanding output stores have read their staging tiles
    }

    // ---- teardown: every role ends here; tensor memory is always released ---------------------
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync();   // the other CTA sends no more arrivals here and the pair's MMAs read no more of this CTA's memory
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before the CTA's resources go away
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        if (threadIdx.x == 0) atomicExch(g.status, (uint32_t)SNIP_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc<true>(tmem_base, 512);
    }
}

template <MmaKind KIND, int SCALE, bool OUT_F32>
int launch_pair(const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmO, const PairArgs &g, uint32_t idesc, cudaStream_t st)
{
    using C = PCfg<KIND>;
    auto kern = gemm_pair_kernel<KIND, SCALE, OUT_F32>;
    SNIP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
    const int num_tiles = (int)(ceil_div(g.Mo, TM) * ceil_div(g.No, TN));
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // The kernel is persistent: no more CTA pairs than can be resident at once (a host-side query,
    // made once per kernel and device).
    static thread_local int slots = 0, slots_dev = -1;
    int dev = 0;
    SNIP_CUDA_TRY(cudaGetDevice(&dev));
    if (slots == 0 || slots_dev != dev) {
        int sms = 0;
        SNIP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        cfg.gridDim = dim3((unsigned)(sms / 2 * 2));
        int nclusters = 0;
        SNIP_CUDA_TRY(cudaOccupancyMaxActiveClusters(&nclusters, kern, &cfg));
        slots = nclusters > 0 ? nclusters : 1;
        slots_dev = dev;
    }
    cfg.gridDim = dim3((unsigned)(2 * (num_tiles < slots ? num_tiles : slots)));
    SNIP_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmO, g, idesc));
    return SNIP_OK;
}

template <MmaKind KIND>
int launch_pair_scale(int scale, bool out_f32, const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmO, const PairArgs &g,
                      uint32_t idesc, cudaStream_t st)
{
    if (scale == PSCALE_BLOCK_B)
        return out_f32 ? launch_pair<KIND, PSCALE_BLOCK_B, true>(tmA, tmB, tmO, g, idesc, st)
                       : launch_pair<KIND, PSCALE_BLOCK_B, false>(tmA, tmB, tmO, g, idesc, st);
    return out_f32 ? launch_pair<KIND, PSCALE_VEC_B, true>(tmA, tmB, tmO, g, idesc, st)
                   : launch_pair<KIND, PSCALE_VEC_B, false>(tmA, tmB, tmO, g, idesc, st);
}

}  // namespace

// CTA-pair GEMM over stored, quantized operands (arguments as gemm_impl, already validated there).
// tx_skew / wait_limit_ns: see snip_debug_set.
int gemm_pair_impl(int fmt_a, int fmt_b, const void *a_codes, const void *b_codes, int64_t Mo, int64_t No, int64_t Kc, const float *sa,
                   int64_t sa_chunk_stride, const float *sb, int64_t sb_chunk_stride, int64_t sb_blk_stride, int scale_mode, void *out,
                   int out_dtype, int accumulate, uint32_t *status, uint64_t wait_limit_ns, int tx_skew, cudaStream_t st)
{
    PairArgs g;
    g.Mo = (int32_t)Mo; g.No = (int32_t)No; g.Kc = (int32_t)Kc;
    g.sa = sa; g.sa_chunk_stride = sa_chunk_stride;
    g.sb = sb; g.sb_chunk_stride = sb_chunk_stride; g.sb_blk_stride = sb_blk_stride;
    g.out = out; g.ldo = No; g.accumulate = accumulate;
    g.status = status;
    g.wait_limit_ns = wait_limit_ns;
    const bool f32 = out_dtype == SNIP_OUT_FP32;
    const bool a4 = fmt_a == SNIP_FMT_FP4_E2M1, b4 = fmt_b == SNIP_FMT_FP4_E2M1;

    CUtensorMap tmA, tmB, tmO;
    // output boxes of 32 rows x 64 bytes
    int rc = f32 ? make_tiled_map_2d(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Mo, No, No * 4, 16, 32, CU_TENSOR_MAP_SWIZZLE_64B)
                 : make_tiled_map_2d(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Mo, No, No * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    if (rc) return rc;
    if (a4 && b4) {
        // Packed FP4 on both sides: kind::mxf4 (twice the FP8 rate) on the packed bytes, fetched as plain
        // bytes with exact extents; the hardware block scales are the constant 1.
        rc = make_tiled_map_2d(&tmA, a_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, Kc / 2, Kc / 2, 128, CM, CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        rc = make_tiled_map_2d(&tmB, b_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, No, Kc / 2, Kc / 2, 128, kBRows, CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc) return rc;
        g.stage_tx_bytes = (uint32_t)((CM + kBRows) * 128 + tx_skew);
        return launch_pair_scale<MmaKind::MXF4>(scale_mode, f32, tmA, tmB, tmO, g, make_idesc_block_scaled(1, 1, TM, TN), st);
    }
    // FP8 x FP8 and the mixed pairs: kind::f8f6f4; an FP4 operand is expanded by the TMA unit to one byte per
    // code.  The expanding map type wants an inner extent that is a multiple of 128 codes: a contraction length
    // ending in a 64-wide tile is declared rounded up, and the 64 extra codes of each row (the start of the next
    // row; for the last row, slack that snip_quantize_sizes reserves) meet zero-filled FP8 codes of the other operand.
    const int64_t kpad = ceil_div(Kc, 128) * 128;
    rc = make_tiled_map_2d(&tmA, a_codes, a4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, a4 ? kpad : Kc,
                           a4 ? Kc / 2 : Kc, 128, CM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    rc = make_tiled_map_2d(&tmB, b_codes, b4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, No, b4 ? kpad : Kc,
                           b4 ? Kc / 2 : Kc, 128, kBRows, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    // an expanded FP4 operand occupies 128 B per row in shared memory but reports its 64 packed source bytes
    g.stage_tx_bytes = (uint32_t)(CM * (a4 ? 64 : 128) + kBRows * (b4 ? 64 : 128) + tx_skew);
    return launch_pair_scale<MmaKind::F8F6F4>(scale_mode, f32, tmA, tmB, tmO, g, make_idesc(a4 ? 5 : 0, b4 ? 5 : 0, TM, TN), st);
}

}  // namespace snip
