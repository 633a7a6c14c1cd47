// Block-scaled GEMM with the paper's FP32 tile scales, CTA-pair form:  out[Mo,No] = A[Mo,Kc] . B[No,Kc]^T,
// both operands contraction-major, each 128-long chunk of the contraction multiplied on the tensor
// cores into its own tensor-memory buffer and then scaled by 1/(S_a*S_b) and added into FP32 register
// accumulators (Sec. 2.3: the operator's output is divided by the scales that were multiplied in;
// Fig. 5: the three GEMMs of a linear layer).
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one tcgen05.mma.cta_group::2: the tile is
// 256 rows x 128 columns, each CTA holds 128 rows of A, 64 rows of B and a 128 x 128 slice of the
// accumulator.  That slice is only a quarter of the register file, which leaves room for sixteen
// promotion warps (four per scheduler), and its tensor-memory image is 128 columns, so three or four
// chunks can be in flight between the MMA issuers and the promotion warps.
//
// This is an ALTERNATIVE form of the product computed by gemm.cu, selected only through
// snip_debug_set(SNIP_DEBUG_GEMM_KERNEL, 2): measured on the 7B shapes it is slower than the
// single-CTA kernels (each of its hand-offs costs a warp a few hundred cycles, and with 128-column
// buffers there is one hand-off per 2 M multiply-adds instead of one per 4 M).
//
// Roles in one CTA (640 threads):
//   warps 0..15 : promotion     - 32 rows x 32 columns each (warp % 4 = tensor-memory lane quarter)
//   warp 16     : TMA producer  - this CTA's halves of the operand tiles into a shared-memory ring;
//                                 byte counts are reported to the leader's barrier (no multicast)
//   warp 17     : scale loader  - brings the chunks' scale factors into a shared-memory ring with
//                                 cp.async, well ahead of their use, and turns them into reciprocal
//                                 factors in place
//   warps 18,19 : MMA issuers   - leader CTA only, alternate chunks; the whole warp walks the loop
//                                 and one elected lane issues, so operands stay in uniform registers
// Every mbarrier wait is bounded; on a timeout both CTAs leave cleanly and a status word is raised.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "sm100.cuh"

namespace snip {

using namespace sm100;

int make_tiled_map_2d(CUtensorMap *map, const void *ptr, int dtype, int64_t rows, int64_t inner_elems, int64_t row_bytes, int box_x_elems,
                      int box_rows, int swizzle);

namespace {

constexpr int kEpiWarps = 16;      // warps 0..15: promotion / epilogue (warp % 4 = tensor-memory lane quarter)
constexpr int kProducerWarp = 16;
constexpr int kLoaderWarp = 17;
constexpr int kIssuerWarp0 = 18;   // warps 18 .. 18 + kIssuers - 1
constexpr int kIssuers = 2;
constexpr int kThreads = 32 * (kIssuerWarp0 + kIssuers);
constexpr int CM = 128;       // rows of A / of the accumulator per CTA
constexpr int TM = 2 * CM;    // rows of one tile (CTA pair)
constexpr int TN = 128;       // columns of one tile = one 128-wide scale block of B
constexpr int kBRows = TN / 2;  // rows of B held by one CTA
constexpr int kSD = 32;       // depth of the scale-factor ring, in chunks
constexpr int kSBlk = 8;      // chunks per hand-over of the ring (one full / one empty barrier per 8 slots)
constexpr int kSBlocks = kSD / kSBlk;
constexpr int kAhead = 16;    // chunks whose scale factors are on their way from global memory (cp.async groups in flight)
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
    static constexpr int kStages = 8;
    static constexpr int kABytes = CM * 128;
    static constexpr int kBBytes = kBRows * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kRingBytes = kSD * kSlotFloats * 4;
    static constexpr int kOutBytes = 0;
    static constexpr int kBarBytes = 1024;
    static constexpr int kSmemBytes = kStages * kStageBytes + kRingBytes + kOutBytes + kBarBytes + 1024;
    static constexpr int kSfCol0 = kNBuf * TN;
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    static_assert(kNBuf * TN + (KIND == MmaKind::MXF4 ? kSfCols : 0) <= 512, "tensor memory budget");
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
    constexpr int ND = S * CPS;      // "chunk done" barriers: one per chunk position of the stage ring

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
    auto done_bar = [&](int p) { return bar0 + 8u * (S + p); };                // each CTA: the MMAs of the chunk at ring position p are complete
    auto tempty_bar = [&](int b) { return bar0 + 8u * (S + ND + b); };         // leader: the promotion warps of both CTAs have drained buffer b
    auto sfull_bar = [&](int k) { return bar0 + 8u * (S + ND + NB + k); };     // each CTA: the 8 slots of ring block k hold their chunks' factors
    auto sempty_bar = [&](int k) { return bar0 + 8u * (S + ND + NB + kSBlocks + k); };   // each CTA: all 16 promotion warps are done with block k
    static_assert((S + ND + NB + 2 * kSBlocks) * 8 + 8 <= C::kBarBytes, "barrier area");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_gen + 8 * (S + ND + NB + 2 * kSBlocks));
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);   // warp-uniform by construction
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();   // 0 = leader
    const int num_m = (g.Mo + TM - 1) / TM, num_n = (g.No + TN - 1) / TN;
    const int num_tiles = num_m * num_n;
    const int first_tile = (int)(blockIdx.x >> 1), tile_step = (int)(gridDim.x >> 1);
    const int my_tiles = first_tile < num_tiles ? (num_tiles - first_tile + tile_step - 1) / tile_step : 0;
    const int nacc = (g.Kc + 127) / 128;                    // chunks per tile
    const int num_kstages = (nacc + CPS - 1) / CPS;
    const uint64_t limit = g.wait_limit_ns;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) mbar_init(full_bar(s), 1);
        for (int p = 0; p < ND; ++p) mbar_init(done_bar(p), 1);
        for (int b = 0; b < NB; ++b) mbar_init(tempty_bar(b), 2);
        for (int k = 0; k < kSBlocks; ++k) { mbar_init(sfull_bar(k), 1); mbar_init(sempty_bar(k), kEpiWarps); }
        *abort_flag = 0u;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        prefetch_tensormap(&tmO);
    }
    if (warp == kIssuerWarp0) {
        tmem_alloc<true>(smem_u32(tmem_slot), 512);
        tmem_relinquish<true>();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (KIND == MmaKind::MXF4) {
        // constant scale factors 2^0 (UE8M0 byte 127) for every row of A and B, in both CTAs
        if (warp < 4) {
            for (int c = 0; c < kSfCols; ++c) tmem_st1(tmem_base + (((uint32_t)warp * 32u) << 16) + C::kSfCol0 + c, 0x7F7F7F7Fu);
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

    // the same for a whole converged warp, with one answer for all its lanes
    auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xFFFFFFFFu, wait(bar, parity)) != 0; };

    if (warp == kProducerWarp) {
        // ================= TMA producer (both CTAs) =================
        // The whole warp walks the loop (so that every value in it is warp-uniform); one elected lane issues.
        {
            uint32_t it = 0;
            bool ok = true;
            const uint32_t lead_full0 = mapa(full_bar(0), 0);
            for (int t = first_tile; t < num_tiles && ok; t += tile_step) {
                int m_idx, n_idx;
                pair_tile_coords(t, num_m, num_n, m_idx, n_idx);
                for (int ks = 0; ks < num_kstages; ++ks, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1u;
                    // a stage is free when the MMAs of all of its chunk positions are complete
#pragma unroll
                    for (int h = 0; h < CPS; ++h) ok = ok && wait_all(done_bar(s * CPS + h), ph ^ 1u);
                    if (!ok) break;
                    if (elect_one()) {
                        if (rank == 0) mbar_arrive_expect_tx(full_bar(s), 2u * g.stage_tx_bytes);
                        tma_load_2d_pair(smem_a0 + s * C::kABytes, &tmA, lead_full0 + 8u * s, ks * 128, m_idx * TM + (int)rank * CM);
                        tma_load_2d_pair(smem_b0 + s * C::kBBytes, &tmB, lead_full0 + 8u * s, ks * 128, n_idx * TN + (int)rank * kBRows);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp >= kIssuerWarp0 && warp < kIssuerWarp0 + kIssuers) {
        // ================= MMA issuers (leader only) =================
        // The whole warp walks the loop, one elected lane issues; issuer i takes the chunk positions p = i, i + kIssuers, ... of the sequence of
        // all stages' positions (a tcgen05.commit costs its thread a few hundred cycles, more than a chunk's MMAs
        // take to run, so one thread alone cannot keep the tensor core busy).  Chunks are independent of one
        // another: each has its own accumulator buffer and its own commit.
        if (rank == 0) {
            const int me = warp - kIssuerWarp0;
            const uint32_t sfa = tmem_base + C::kSfCol0, sfb = tmem_base + C::kSfCol0 + 16;
            const uint32_t pos_per_tile = (uint32_t)num_kstages * CPS;
            const uint32_t total_pos = (uint32_t)my_tiles * pos_per_tile;
            const uint32_t holes_per_tile = pos_per_tile - (uint32_t)nacc;   // positions of a tile's last stage without a chunk
            const uint32_t done_peer0 = mapa(done_bar(0), 1);
            bool ok = true;
            for (uint32_t p = (uint32_t)me; p < total_pos && ok; p += kIssuers) {
                const uint32_t it = p / CPS, h = p % CPS;
                const uint32_t tile_seq = p / pos_per_tile, in_tile = p - tile_seq * pos_per_tile;
                const int s = it % S;
                const uint32_t ph = (it / S) & 1u;
                // The stage's operands have landed; this also puts the commit below behind the hand-over of the
                // position's previous occupant (the producer refilled the stage only after seeing that one complete).
                if (!wait_all(full_bar(s), ph)) { ok = false; break; }
                if (in_tile < (uint32_t)nacc) {
                    const uint32_t cc = p - tile_seq * holes_per_tile;   // number of the chunk among the real chunks
                    const uint32_t b = cc % NB;
                    if (!wait_all(tempty_bar(b), ((cc / NB) & 1u) ^ 1u)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t adesc = make_smem_desc_k128(smem_a0 + s * C::kABytes);
                    const uint64_t bdesc = make_smem_desc_k128(smem_b0 + s * C::kBBytes);
                    constexpr int kPerChunk = 4 / CPS;   // 32-byte K steps per chunk
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < kPerChunk; ++k)
                            mma_ss<KIND, true>(tmem_base + b * TN, adesc + 2 * (kPerChunk * h + k), bdesc + 2 * (kPerChunk * h + k), idesc,
                                               k > 0 ? 1u : 0u, sfa, sfb);
                    }
                }
                // (a position without a chunk - the second half of a last stage - is committed all the same: the
                // producer and the peer CTA count positions)
                if (elect_one()) {
                    tc_commit<true>(done_bar(s * CPS + h));
                    tc_commit<true>(done_peer0 + 8u * (s * CPS + h));
                }
                __syncwarp();
            }
        }
    } else if (warp == kLoaderWarp) {
        // ================= scale loader =================
        // Lane l brings the factors of rows 4l..4l+3 of this CTA (block mode: 1/(S_a*S_b); vector mode: 1/S_a and,
        // for the tile's columns 4l..4l+3, 1/S_b).  Chunks are walked as one sequence over all of this pair's
        // tiles.  Chunk c + kAhead is requested (16-byte cp.async copies, one commit group) as soon as the promotion
        // warps have let go of the ring slot it lands in; chunk c is then awaited, turned into reciprocals in
        // place by the lanes that fetched it, and published.  Neither the operand pipeline nor the tensor core
        // ever waits for a scale factor's trip from global memory.
        const uint32_t total = (uint32_t)my_tiles * (uint32_t)nacc;
        const uint32_t ring_u32 = smem_u32(ring);
        int pt = first_tile, pj = 0;   // tile and chunk of the next request
        uint32_t pc = 0;               // its position in the sequence
        bool ok = true;
        // source addresses of the requested tile's first chunk (recomputed when the tile changes)
        const float *src_a = g.sa, *src_b = g.sb;
        auto tile_sources = [&]() {
            int m_idx, n_idx;
            pair_tile_coords(pt < num_tiles ? pt : first_tile, num_m, num_n, m_idx, n_idx);
            // rows / columns outside the matrix repeat the last four factors (their sums are never stored)
            src_a = g.sa + min(m_idx * TM + (int)rank * CM + 4 * lane, g.Mo - 4);
            if (SCALE == PSCALE_BLOCK_B) src_b = g.sb + (int64_t)n_idx * g.sb_blk_stride;
            else src_b = g.sb + min(n_idx * TN + 4 * lane, g.No - 4);
        };
        tile_sources();
        auto request = [&]() {
            if (pc < total && ok) {
                const uint32_t d = pc % kSD;
                // the first slot of a ring block is requested once the promotion warps have handed the block back
                if ((pc % kSBlk) == 0 && !wait(sempty_bar(d / kSBlk), ((pc / kSD) & 1u) ^ 1u)) ok = false;
                else {
                    const uint32_t slot = ring_u32 + d * (kSlotFloats * 4);
                    cp_async_16(slot + 16u * lane, src_a);
                    if (SCALE == PSCALE_BLOCK_B) {
                        if (lane == 0) cp_async_4(slot + 512u, src_b);
                    } else {
                        cp_async_16(slot + 512u + 16u * lane, src_b);
                    }
                    src_a += g.sa_chunk_stride;
                    src_b += g.sb_chunk_stride;
                    if (++pj == nacc) { pj = 0; pt += tile_step; tile_sources(); }
                }
            }
            ++pc;
            cp_async_commit();   // one group per position, empty past the end, so that the count below stays uniform
        };
        for (int i = 0; i < kAhead; ++i) request();
        for (uint32_t cc = 0; cc < total && ok; ++cc) {
            request();                  // position cc + kAhead
            cp_async_wait<kAhead>();    // this lane's copies of position cc have landed
            const uint32_t d = cc % kSD;
            float4 *mine = reinterpret_cast<float4 *>(ring + d * kSlotFloats + 4 * lane);
            const float4 v = *mine;
            if (SCALE == PSCALE_BLOCK_B) {
                __syncwarp();           // lane 0's copy of the block scale is visible to the warp
                const float bsc = ring[d * kSlotFloats + 128];
                *mine = make_float4(rcp_fast(v.x * bsc), rcp_fast(v.y * bsc), rcp_fast(v.z * bsc), rcp_fast(v.w * bsc));
            } else {
                const float4 w = mine[32];
                *mine = make_float4(rcp_fast(v.x), rcp_fast(v.y), rcp_fast(v.z), rcp_fast(v.w));
                mine[32] = make_float4(rcp_fast(w.x), rcp_fast(w.y), rcp_fast(w.z), rcp_fast(w.w));
            }
            __syncwarp();
            // a block is published when its last slot (or the last chunk of all) is ready
            if (lane == 0 && ((cc % kSBlk) == kSBlk - 1 || cc + 1 == total)) mbar_arrive(sfull_bar(d / kSBlk));
        }
        cp_async_wait<0>();
    } else if (warp < kEpiWarps) {
        // ================= promotion / epilogue warps =================
        // Per chunk a warp has little arithmetic (16 packed multiply-adds) against several hand-offs, so the loop is
        // arranged for the hand-offs not to wait on one another: the scale ring is taken and given back eight
        // chunks at a time, the next chunk's completion barrier is tested (without blocking) while this chunk's
        // tensor-memory load is in flight, and buffers go back with relaxed arrivals that nobody waits for.
        const int e = warp;              // 0..15
        const int q = warp & 3;          // tensor-memory lane quarter this warp may access
        const int cg = e >> 2;           // 32-column group
        const uint32_t tempty_lead0 = mapa(tempty_bar(0), 0);
        const uint32_t total = (uint32_t)my_tiles * (uint32_t)nacc;
        const uint32_t taddr0 = tmem_base + ((uint32_t)(q * 32) << 16) + cg * 32;
        // ring position of the current chunk: stage s (parity sph), chunk h of the stage; buffer b; chunk j of the tile
        uint32_t s = 0, sph = 0, h = 0, b = 0;
        int j = 0, t = first_tile;
        int row0 = 0, col0 = 0;
        bool have = false;               // the current chunk's completion has already been seen
        bool ok = true;
        float2 acc[16];
        for (uint32_t cc = 0; cc < total; ++cc) {   // never left early: the other warps wait for this one on hardware barriers
            // (after a failed wait every later wait returns at once)
            if (j == 0) {
                int m_idx, n_idx;
                pair_tile_coords(t, num_m, num_n, m_idx, n_idx);
                row0 = m_idx * TM + (int)rank * CM + q * 32;
                col0 = n_idx * TN + cg * 32;
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = make_float2(0.0f, 0.0f);
            }
            const uint32_t d = cc % kSD;
            const float *slot = ring + d * kSlotFloats;
            const uint32_t dp = s * CPS + h;
            if ((cc % kSBlk) == 0) {
                const bool got = wait(sfull_bar(d / kSBlk), (cc / kSD) & 1u);
                if (!__all_sync(0xFFFFFFFFu, got)) ok = false;
            }
            if (!have) {
                const bool got = wait(done_bar(dp), sph);
                if (!__all_sync(0xFFFFFFFFu, got)) ok = false;
            }
            tc_fence_after_sync();
            uint32_t v[32];
            tmem_ld32(taddr0 + b * TN, v);
            const float f = slot[q * 32 + lane];
            // position of the next chunk (the tile's last stage may have fewer chunks than positions)
            const bool tile_end = (j + 1 == nacc);
            uint32_t ns = s, nsph = sph, nh = h + 1;
            if (nh == CPS || tile_end) { nh = 0; if (++ns == S) { ns = 0; nsph ^= 1u; } }
            // non-blocking look at the next chunk's barrier while the load is in flight
            const bool next_seen = (cc + 1 < total) && mbar_test_wait(done_bar(ns * CPS + nh), nsph);
            tmem_ld_wait();
            // this warp's reads of buffer b are done: hand it back to the MMA issuers
            // (the sixteen warps meet on a hardware barrier - one per buffer, fifteen arrive without waiting - and
            // the warp that waits sends ONE arrival per CTA: arrivals on one mbarrier are served one after the other,
            // and thirty-two of them per chunk would take longer than the chunk's MMAs)
            tc_fence_before_sync();
            if (e == (int)b) {
                named_bar_sync(1 + b, 32 * kEpiWarps);
                if (lane == 0) mbar_arrive_cluster_relaxed(tempty_lead0 + 8u * b);
            } else {
                named_bar_arrive(1 + b, 32 * kEpiWarps);
            }
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
            have = __all_sync(0xFFFFFFFFu, next_seen);
            if ((cc % kSBlk) == kSBlk - 1) {
                // every lane's reads of the block's slots are behind this warp barrier (their values have been used)
                __syncwarp();
                if (lane == 0) mbar_arrive(sempty_bar(d / kSBlk));
            }
            s = ns; sph = nsph; h = nh;
            if (++b == NB) b = 0;
            if (!tile_end) { ++j; continue; }
            // ---- the tile is complete: round and store ----
            j = 0;
            const int row = row0 + lane;
            const float *av = reinterpret_cast<const float *>(acc);
            if (row < g.Mo && ok) {
                // each lane owns 32 consecutive outputs of its row: 16-byte stores (L2 merges them into whole sectors)
                if (OUT_F32) {
                    float *dst = static_cast<float *>(g.out) + (int64_t)row * g.ldo + col0;
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        if (col0 + i < g.No) {
                            float4 o = make_float4(av[i], av[i + 1], av[i + 2], av[i + 3]);
                            if (g.accumulate) {   // gradient accumulation into the existing FP32 output
                                const float4 p = *reinterpret_cast<const float4 *>(dst + i);
                                o.x += p.x; o.y += p.y; o.z += p.z; o.w += p.w;
                            }
                            *reinterpret_cast<float4 *>(dst + i) = o;
                        }
                    }
                } else {
                    __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(g.out) + (int64_t)row * g.ldo + col0;
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        if (col0 + i < g.No)
                            *reinterpret_cast<uint4 *>(dst + i) = make_uint4(bf16x2_bits(av[i], av[i + 1]), bf16x2_bits(av[i + 2], av[i + 3]),
                                                                             bf16x2_bits(av[i + 4], av[i + 5]), bf16x2_bits(av[i + 6], av[i + 7]));
                    }
                }
            }
            __syncwarp();
            t += tile_step;
        }
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
    if (warp == kIssuerWarp0) {
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
