// Block-scaled GEMMs on the tcgen05 tensor cores:  out[Mo,No] = A[Mo,Kc] . B[No,Kc]^T with both
// operands contraction-major, FP32 accumulation in tensor memory, and the paper's FP32 tile
// scales applied per 128-long chunk of the contraction (Sec. 2.3: "the output is scaled back by
// dividing by the same scaling factor"; Fig. 5 for the three GEMMs of a linear layer).
//
// Structure of one CTA (persistent, one per SM, 384 threads):
//   warp 0      : TMA producer - streams 128-byte-wide operand tiles into a shared-memory ring
//   warp 1      : MMA issuer   - one thread issues tcgen05.mma; owns the tensor-memory allocation
//   warps 2..3  : weight-gradient product: loaders of the per-row / per-column scale factors (one ring of ready
//                 reciprocals for the CTA); otherwise idle (they only give their registers to the epilogue warps)
//   warps 4..11 : promotion / epilogue - pull each chunk's partial sums out of tensor memory,
//                 multiply by 1/(S_a*S_b) of that chunk and add into FP32 register accumulators
//                 (so the scaling overlaps the next chunk's MMAs, which write the other
//                 tensor-memory buffer), then round and store the tile.
// All hand-offs use mbarriers with bounded waits; on a timeout the CTA raises a status word and
// leaves cleanly (tensor memory is always released).
#include <cuda.h>
#include <cuda_bf16.h>

#include <atomic>

#include "common.cuh"
#include "sm100.cuh"

namespace snip {

using namespace sm100;

namespace {

constexpr int BM = 128;
constexpr int kGemmThreads = 384;  // warps 0-3: producer, MMA issuer, 2 scale loaders (wgrad) or idle; warps 4-11: epilogue
constexpr int kNumEpiWarps = 8;
// Slicing of the weight-gradient product's last wave (see launch_gemm)
constexpr int kMaxSlices = 4, kMinSliceStages = 8, kMaxSlicedItems = 160;
constexpr size_t kSliceCountersOffset = 256, kSliceCountersBytes = 8192;   // counters: [sliced tile][epilogue warp], 32 bits each
static_assert((size_t)kMaxSlicedItems / 2 * kNumEpiWarps * 4 <= kSliceCountersBytes, "counter area");
constexpr int kSfCols = 32;  // tensor-memory columns holding constant scale factors (kind::mxf4)

enum ScaleMode { SCALE_NONE = 0, SCALE_BLOCK_B = 1, SCALE_VEC_B = 2 };

struct GemmArgs {
    int32_t Mo, No, Kc;        // output rows / cols, contraction length in elements
    const float *sa;           // A scales [chunks][Mo]
    int64_t sa_chunk_stride;
    const float *sb;           // B scales: SCALE_BLOCK_B [blk*sb_blk_stride + chunk*sb_chunk_stride]
    int64_t sb_chunk_stride;   //           SCALE_VEC_B   [chunk*sb_chunk_stride + n]
    int64_t sb_blk_stride;
    void *out;
    int64_t ldo;
    int32_t accumulate;
    uint32_t stage_tx_bytes;   // bytes the two TMA loads of one stage report to the barrier
    uint64_t wait_limit_ns;    // bound of every device-side wait
    uint32_t *status;
    // Work items: item w < split_first is tile w over the whole contraction; the tiles from split_first on (the last,
    // partial wave of a persistent grid) are cut into nsplit contraction slices each, item split_first + r * nsplit + j
    // being slice j of tile split_first + r.  nsplit == 1: no slicing, num_items == number of tiles.
    int32_t split_first, nsplit, num_items;
    float *partials;           // [tail tile r][slice j][epilogue warp][column quad][row lane][4]: FP32 sums of a slice
    uint32_t *counters;        // [tail tile r][epilogue warp]: slices that have delivered their sums (zero at launch)
};

struct WorkItem {
    int t, ks0, ks1;       // tile, stage range of the contraction
    int tail, slice, nsl;  // index of a sliced tile among the sliced tiles, slice, number of slices (1: whole tile)
};
template <bool SLICED>   // false: every item is a whole tile (known at compile time)
__device__ __forceinline__ WorkItem work_item(const GemmArgs &g, int w, int num_kstages)
{
    WorkItem wi;
    if (!SLICED || w < g.split_first) {
        wi.t = w; wi.ks0 = 0; wi.ks1 = num_kstages; wi.tail = 0; wi.slice = 0; wi.nsl = 1;
    } else {
        const int i = w - g.split_first;
        wi.tail = i / g.nsplit;
        wi.slice = i - wi.tail * g.nsplit;
        wi.nsl = g.nsplit;
        wi.t = g.split_first + wi.tail;
        wi.ks0 = (int)((int64_t)wi.slice * num_kstages / g.nsplit);
        wi.ks1 = (int)((int64_t)(wi.slice + 1) * num_kstages / g.nsplit);
    }
    return wi;
}

template <MmaKind KIND, int BN, int SCALE>
struct Cfg {
    static constexpr int kStageElemsX = (KIND == MmaKind::F16) ? 64 : 128;   // TMA x step per stage
    static constexpr int kChunkElems = 128;                                  // scale granularity
    static constexpr int kStageK = (KIND == MmaKind::F16) ? 64 : (KIND == MmaKind::F8F6F4 ? 128 : 256);
    static constexpr int kABytes = BM * 128;
    static constexpr int kBBytes = BN * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStages = (BN >= 256) ? 4 : 5;
    // block mode (fwd / dgrad) fetches four chunks of scale factors per instruction into two alternating group slots:
    // [4 chunks][32 rows] S_a, then [2 blocks][4 chunks] S_b
    static constexpr int kGroupFloats = 144;
    static constexpr int kRingFloatsPerWarp = 2 * kGroupFloats;
    // vector mode (wgrad): ONE ring for the CTA, filled by the two loader warps: per chunk 128 row factors 1/S_a and BN column
    // factors 1/S_b, kVecDepth chunks deep, handed over kVecBlock chunks at a time
    static constexpr int kVecDepth = 16, kVecBlock = 4, kVecAhead = 8;
    static constexpr int kVecSlotFloats = 128 + BN;
    static constexpr int kSbInvBytes = (SCALE == 2) ? kVecDepth * kVecSlotFloats * 4 : kNumEpiWarps * kRingFloatsPerWarp * 4;
    // block mode (fwd / dgrad) writes its output through per-warp 2 KB staging tiles and TMA stores
    static constexpr bool kTmaOut = (SCALE == 1);
    static constexpr int kOutStageBytes = kTmaOut ? kNumEpiWarps * 2048 : 0;
    static constexpr int kSmemBytes = kStages * kStageBytes + kSbInvBytes + kOutStageBytes + 256 + 1024;  // + barriers + alignment slack
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    static_assert(kStageBytes % 1024 == 0 && kSbInvBytes % 1024 == 0, "staging tiles must stay 1024-byte aligned");
    static constexpr int kAccCols = 2 * BN;
    static constexpr int kSfCol0 = kAccCols;
    static constexpr int kTmemCols = 512;
    static_assert(kAccCols + (KIND == MmaKind::MXF4 ? kSfCols : 0) <= 512, "tensor memory budget");
};

__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int &m_idx, int &n_idx)
{
    // groups of 16 row-tiles share their B panels in L2 while they are resident together
    constexpr int kGroupM = 16;
    const int group_size = kGroupM * num_n;
    const int g = t / group_size;
    const int first_m = g * kGroupM;
    const int gm = min(num_m - first_m, kGroupM);
    const int r = t - g * group_size;
    m_idx = first_m + r % gm;
    n_idx = r / gm;
}

// Reciprocal from the special-function unit (one instruction, ~1 ulp; a subnormal result is flushed to zero,
// which only affects products of scales beyond FP32's range).
__device__ __forceinline__ float rcp_approx(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Store 32 consecutive output values of one row.
template <bool OUT_F32>
__device__ __forceinline__ void store32(const GemmArgs &g, int64_t row, int col, const float *v)
{
    if (OUT_F32) {
        float *dst = static_cast<float *>(g.out) + row * g.ldo + col;
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            if (col + i < g.No) {
                float4 o = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                if (g.accumulate) {
                    const float4 p = *reinterpret_cast<const float4 *>(dst + i);
                    o.x += p.x; o.y += p.y; o.z += p.z; o.w += p.w;
                }
                *reinterpret_cast<float4 *>(dst + i) = o;
            }
        }
    } else {
        __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(g.out) + row * g.ldo + col;
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
            if (col + i < g.No) {
                uint4 o = make_uint4(pack_bf16x2(v[i], v[i + 1]), pack_bf16x2(v[i + 2], v[i + 3]),
                                     pack_bf16x2(v[i + 4], v[i + 5]), pack_bf16x2(v[i + 6], v[i + 7]));
                *reinterpret_cast<uint4 *>(dst + i) = o;
            }
        }
    }
}

template <MmaKind KIND, int BN, int SCALE, bool OUT_F32>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmO,
            const GemmArgs g, const uint32_t idesc)
{
    using C = Cfg<KIND, BN, SCALE>;
    constexpr int S = C::kStages;
    constexpr int HALF = BN / 2;     // columns handled by one epilogue warp
    // columns per tensor-memory load: 16 in vector mode (wgrad: the promotion loop holds the column reciprocals next to the
    // staging registers and runs 1.5-4 % faster with the smaller groups), 32 otherwise (fwd / dgrad: 2.5 % faster than 16)
    constexpr int GC = (SCALE == SCALE_VEC_B) ? 16 : 32;
    constexpr int G = HALF / GC;     // groups handled by one epilogue warp per chunk

    extern __shared__ uint8_t smem_raw[];
    // operand tiles need 1024-byte alignment for the 128-byte swizzle
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t smem_a0 = smem_base;
    const uint32_t smem_b0 = smem_base + S * C::kABytes;
    float *scale_ring = reinterpret_cast<float *>(smem_gen + S * C::kStageBytes);
    const uint32_t out_stage0 = smem_base + S * C::kStageBytes + C::kSbInvBytes;   // 1024-byte aligned
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_gen + S * C::kStageBytes + C::kSbInvBytes + C::kOutStageBytes);
    const uint32_t bar0 = smem_base + S * C::kStageBytes + C::kSbInvBytes + C::kOutStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (S + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * S + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * S + 2 + a); };
    constexpr int kVBlocks = C::kVecDepth / C::kVecBlock;
    auto vfull_bar = [&](int k) { return bar0 + 8u * (2 * S + 4 + k); };              // vector mode: ring block k holds its chunks' factors
    auto vempty_bar = [&](int k) { return bar0 + 8u * (2 * S + 4 + kVBlocks + k); };  // vector mode: the eight epilogue warps are done with block k
    static_assert((2 * S + 4 + 2 * kVBlocks) * 8 + 8 <= 256, "barrier area");
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * S + 4 + 2 * kVBlocks);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_m = (g.Mo + BM - 1) / BM, num_n = (g.No + BN - 1) / BN;
    const int num_chunks = (g.Kc + C::kChunkElems - 1) / C::kChunkElems;
    const int num_kstages = (g.Kc + C::kStageK - 1) / C::kStageK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), kNumEpiWarps); }
        for (int k = 0; k < kVBlocks; ++k) { mbar_init(vfull_bar(k), 2); mbar_init(vempty_bar(k), kNumEpiWarps); }
        *abort_flag = 0u;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc<false>(smem_u32(tmem_slot), C::kTmemCols);
        tmem_relinquish<false>();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (KIND == MmaKind::MXF4) {
        // constant scale factors 2^0 (UE8M0 byte 127) for every row of A and B
        if (warp >= 4 && warp < 8) {
            const uint32_t q = warp & 3;
            for (int c = 0; c < kSfCols; ++c) tmem_st1(tmem_base + ((q * 32u) << 16) + C::kSfCol0 + c, 0x7F7F7F7Fu);
            tmem_st_wait();
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
    }

    if (warp < 4) {
      reg_dealloc<40>();  // frees (168-40)*128 = 16384 registers
      if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < g.num_items && ok; w += gridDim.x) {
                const WorkItem wi = work_item<SCALE == SCALE_VEC_B>(g, w, num_kstages);
                int m_idx, n_idx;
                tile_coords(wi.t, num_m, num_n, m_idx, n_idx);
                for (int ks = wi.ks0; ks < wi.ks1; ++ks, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, g.wait_limit_ns)) { ok = false; break; }
                    mbar_arrive_expect_tx(full_bar(s), g.stage_tx_bytes);
                    tma_load_2d(smem_a0 + s * C::kABytes, &tmA, full_bar(s), ks * C::kStageElemsX, m_idx * BM);
                    tma_load_2d(smem_b0 + s * C::kBBytes, &tmB, full_bar(s), ks * C::kStageElemsX, n_idx * BN);
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            uint32_t it = 0, cc = 0;
            bool ok = true;
            const uint32_t sfa = tmem_base + C::kSfCol0, sfb = tmem_base + C::kSfCol0 + 16;
            for (int w = blockIdx.x; w < g.num_items && ok; w += gridDim.x) {
                const WorkItem wi = work_item<SCALE == SCALE_VEC_B>(g, w, num_kstages);
                for (int ks = wi.ks0; ks < wi.ks1 && ok; ++ks, ++it) {
                    const int s = it % S;
                    const uint32_t ph = (it / S) & 1u;
                    if (!mbar_wait(full_bar(s), ph, abort_flag, g.wait_limit_ns)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t adesc = make_smem_desc_k128(smem_a0 + s * C::kABytes);
                    const uint64_t bdesc = make_smem_desc_k128(smem_b0 + s * C::kBBytes);
                    if (KIND == MmaKind::F16) {
                        const uint32_t a = cc & 1u;
                        if (ks == wi.ks0) {
                            if (!mbar_wait(tempty_bar(a), ((cc >> 1) & 1u) ^ 1u, abort_flag, g.wait_limit_ns)) { ok = false; break; }
                            tc_fence_after_sync();
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_ss<KIND, false>(tmem_base + a * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (ks > wi.ks0 || k > 0) ? 1u : 0u, 0, 0);
                        tc_commit<false>(empty_bar(s));
                        if (ks == wi.ks1 - 1) { tc_commit<false>(tfull_bar(a)); ++cc; }
                    } else if (KIND == MmaKind::F8F6F4) {
                        const uint32_t a = cc & 1u;
                        if (!mbar_wait(tempty_bar(a), ((cc >> 1) & 1u) ^ 1u, abort_flag, g.wait_limit_ns)) { ok = false; break; }
                        tc_fence_after_sync();
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            mma_ss<KIND, false>(tmem_base + a * BN, adesc + 2 * k, bdesc + 2 * k, idesc, k > 0 ? 1u : 0u, 0, 0);
                        // one commit serves both hand-offs (a stage is one chunk here): the producer takes it as
                        // "stage s is free", the epilogue warps as "the chunk's partial sums are complete"
                        tc_commit<false>(empty_bar(s));
                        ++cc;
                    } else {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (2 * ks + h < num_chunks) {
                                const uint32_t a = cc & 1u;
                                if (!mbar_wait(tempty_bar(a), ((cc >> 1) & 1u) ^ 1u, abort_flag, g.wait_limit_ns)) { ok = false; break; }
                                tc_fence_after_sync();
#pragma unroll
                                for (int k = 0; k < 2; ++k)
                                    mma_ss<KIND, false>(tmem_base + a * BN, adesc + 2 * (2 * h + k), bdesc + 2 * (2 * h + k), idesc,
                                                 k > 0 ? 1u : 0u, sfa, sfb);
                                tc_commit<false>(tfull_bar(a));
                                ++cc;
                            }
                        }
                        tc_commit<false>(empty_bar(s));
                    }
                }
            }
        }
      } else if (SCALE == SCALE_VEC_B) {
        // ================= warps 2, 3: scale loaders of the weight-gradient product =================
        // Both factors of a chunk are vectors here (1/S_a per output row, 1/S_b per output column).  Warp 2 brings the 128
        // row scales, warp 3 the BN column scales of every chunk into one ring for the CTA (cp.async, kVecAhead chunks
        // ahead), turns them into reciprocals in place and publishes them kVecBlock chunks at a time, so that the epilogue
        // warps only read ready factors: no copies, reciprocals or warp barriers of their own on the per-chunk path.
        const bool rows_side = (warp == 2);
        constexpr int kChunksPerStage = C::kStageK / C::kChunkElems;
        uint32_t total = 0;            // chunks of all of this CTA's work items
        for (int w = blockIdx.x; w < g.num_items; w += gridDim.x) {
            const WorkItem wi = work_item<SCALE == SCALE_VEC_B>(g, w, num_kstages);
            total += (uint32_t)(min(kChunksPerStage * wi.ks1, num_chunks) - kChunksPerStage * wi.ks0);
        }
        const uint32_t ring_u32 = smem_u32(scale_ring);
        int pw = blockIdx.x, pj = 0, pn = 0;   // work item and chunk of the next request, chunks of that item
        uint32_t pc = 0;               // its position in the sequence of this CTA's chunks
        bool ok = true;
        const float *src0 = nullptr, *src1 = nullptr;
        int64_t stride = 0;
        auto item_sources = [&]() {
            const WorkItem wi = work_item<SCALE == SCALE_VEC_B>(g, pw < g.num_items ? pw : (int)blockIdx.x, num_kstages);
            int m_idx, n_idx;
            tile_coords(wi.t, num_m, num_n, m_idx, n_idx);
            const int c0 = kChunksPerStage * wi.ks0;
            pn = min(kChunksPerStage * wi.ks1, num_chunks) - c0;
            // rows / columns outside the matrix repeat the last four factors (their sums are never stored)
            if (rows_side) {
                stride = g.sa_chunk_stride;
                src0 = g.sa + c0 * stride + min(m_idx * BM + 4 * lane, g.Mo - 4);
            } else {
                stride = g.sb_chunk_stride;
                src0 = g.sb + c0 * stride + min(n_idx * BN + 4 * lane, g.No - 4);
                src1 = g.sb + c0 * stride + min(n_idx * BN + 128 + 4 * lane, g.No - 4);
            }
        };
        item_sources();
        auto request = [&]() {
            if (pc < total && ok) {
                const uint32_t d = pc % C::kVecDepth;
                if ((pc % C::kVecBlock) == 0 && !__all_sync(0xFFFFFFFFu, mbar_wait(vempty_bar(d / C::kVecBlock), ((pc / C::kVecDepth) & 1u) ^ 1u, abort_flag, g.wait_limit_ns))) ok = false;
                else {
                    const uint32_t slot = ring_u32 + d * (C::kVecSlotFloats * 4);
                    if (rows_side) {
                        cp_async_16(slot + 16u * lane, src0);
                    } else {
                        cp_async_16(slot + 512u + 16u * lane, src0);
                        if (128 + 4 * lane < BN) cp_async_16(slot + 1024u + 16u * lane, src1);
                    }
                    src0 += stride;
                    src1 += stride;
                    if (++pj == pn) { pj = 0; pw += gridDim.x; item_sources(); }
                }
            }
            ++pc;
            cp_async_commit();   // one group per position, empty past the end, so that the wait below stays uniform
        };
        for (int i = 0; i < C::kVecAhead; ++i) request();
        for (uint32_t cc = 0; cc < total && ok; ++cc) {
            request();                       // position cc + kVecAhead
            cp_async_wait<C::kVecAhead>();   // this lane's copies of position cc have landed
            const uint32_t d = cc % C::kVecDepth;
            float4 *mine = reinterpret_cast<float4 *>(scale_ring + d * C::kVecSlotFloats + (rows_side ? 0 : 128) + 4 * lane);
            const float4 v = mine[0];
            mine[0] = make_float4(rcp_approx(v.x), rcp_approx(v.y), rcp_approx(v.z), rcp_approx(v.w));
            if (!rows_side && 128 + 4 * lane < BN) {
                const float4 w = mine[32];
                mine[32] = make_float4(rcp_approx(w.x), rcp_approx(w.y), rcp_approx(w.z), rcp_approx(w.w));
            }
            __syncwarp();
            // a block is published when its last slot (or the last chunk of all) is ready
            if (lane == 0 && ((cc % C::kVecBlock) == C::kVecBlock - 1 || cc + 1 == total)) mbar_arrive(vfull_bar(d / C::kVecBlock));
        }
        cp_async_wait<0>();
      }
    } else {
        reg_alloc<232>();    // needs (232-168)*256 = 16384 <= 16384 (an unsatisfiable request would block forever)
        // ================= promotion / epilogue warps =================
        const int e = warp - 4;          // 0..7
        const int q = warp & 3;          // tensor-memory lane quarter this warp may access
        const int h = e >> 2;            // column half
        // Block mode: per-warp scale-factor buffers, filled ahead with cp.async so that no global-memory latency
        // sits between two chunks.  S_a of this warp's 32 rows comes four chunks at a time into two alternating
        // group slots [4 chunks][32 rows], with the S_b of its one or two 128-column blocks next to them
        // ([2 blocks][4 chunks] at float 128 of the group).  Vector mode reads the CTA's ring of ready factors.
        float *ring = scale_ring + e * C::kRingFloatsPerWarp;
        const uint32_t ring_u32 = smem_u32(ring);
        const uint32_t stage_u32 = out_stage0 + e * 2048;   // this warp's staging tile: 32 rows x 64 bytes
        uint32_t cc = 0;
        bool ok = true;
        for (int w = blockIdx.x; w < g.num_items && ok; w += gridDim.x) {
            const WorkItem wi = work_item<SCALE == SCALE_VEC_B>(g, w, num_kstages);
            int m_idx, n_idx;
            tile_coords(wi.t, num_m, num_n, m_idx, n_idx);
            const int row0 = m_idx * BM + q * 32;
            const int row = row0 + lane;
            const int col0 = n_idx * BN + h * HALF;
            const bool row_ok = row < g.Mo;
            constexpr int kChunksPerStage = C::kStageK / C::kChunkElems;
            const int nacc = (KIND == MmaKind::F16) ? 1 : min(kChunksPerStage * wi.ks1, num_chunks) - kChunksPerStage * wi.ks0;
            const int blk0 = col0 >> 7;
            const int blk_last = (g.No - 1) >> 7;

            // Block mode: the scale factors of four consecutive chunks with two instructions per warp.  Lane L
            // fetches 16 bytes = S_a of rows 4*(L%8) .. +3 of chunk 4*gn + L/8 (the warp's 32 rows lie inside or
            // outside the matrix together: row counts are multiples of 64); lanes 0..3 (0..7 with two blocks)
            // fetch S_b of one chunk each.  Group gn lands in slot gn % 2.
            constexpr int kBlocksPerWarp = ((HALF % 128) == 0) ? 1 : 2;
            auto prefetch_group = [&](int gn) {
                if (4 * gn < nacc) {
                    const uint32_t slot = ring_u32 + (gn & 1) * C::kGroupFloats * 4;
                    const int ci = lane >> 3, r4 = (lane & 7) * 4, chunk = 4 * gn + ci;
                    if (row0 < g.Mo && chunk < nacc)
                        cp_async_16(slot + (ci * 32 + r4) * 4, g.sa + (int64_t)chunk * g.sa_chunk_stride + row0 + r4);
                    if (lane < 4 * kBlocksPerWarp) {
                        const int blk = min(blk0 + (lane >> 2), blk_last), cb = 4 * gn + (lane & 3);
                        if (cb < nacc) cp_async_4(slot + (128 + lane) * 4, g.sb + (int64_t)blk * g.sb_blk_stride + (int64_t)cb * g.sb_chunk_stride);
                    }
                }
                cp_async_commit();
            };

            float2 acc[SCALE == SCALE_NONE ? 1 : HALF / 2];
            if (SCALE != SCALE_NONE) {
#pragma unroll
                for (int i = 0; i < HALF / 2; ++i) acc[i] = make_float2(0.0f, 0.0f);
                if (SCALE == SCALE_BLOCK_B) {
                    // out-of-range rows / columns read 1.0 (their products are zero anyway)
                    for (int i = lane; i < C::kRingFloatsPerWarp; i += 32) ring[i] = 1.0f;
                    __syncwarp();
                    prefetch_group(0);
                    prefetch_group(1);
                }
            }
            // Block mode: the reciprocal factors 1/(S_a*S_b) of the four chunks of group gn, from its slot (which must
            // have landed and been made visible to the warp), into a register queue that the chunk loop shifts.
            float fq[kBlocksPerWarp][4];
            auto load_factors = [&](int gn) {
                const float *sl = ring + (gn & 1) * C::kGroupFloats;
                const float4 b0 = *reinterpret_cast<const float4 *>(sl + 128);
                const float sb0[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float sa = sl[j * 32 + lane];
                    fq[0][j] = rcp_approx(sa * sb0[j]);
                    if (kBlocksPerWarp == 2) fq[1][j] = rcp_approx(sa * sl[132 + j]);
                }
            };
            if (SCALE == SCALE_BLOCK_B) {
                cp_async_wait<1>();   // group 0
                __syncwarp();
                load_factors(0);
            }
            for (int c = 0; c < nacc; ++c, ++cc) {
                const uint32_t a = cc & 1u;
                float f[G];
                // vector mode: this chunk's slot of the CTA's factor ring (filled by warps 2 and 3), taken over a block at a time
                const uint32_t vd = cc % C::kVecDepth;
                const float *vslot = scale_ring + vd * C::kVecSlotFloats;
                const float *slot = vslot + 128 + h * HALF;   // this warp's column reciprocals
                if (SCALE == SCALE_VEC_B && (cc % C::kVecBlock) == 0) {
                    const bool got = mbar_wait(vfull_bar(vd / C::kVecBlock), (cc / C::kVecDepth) & 1u, abort_flag, g.wait_limit_ns);
                    if (!__all_sync(0xFFFFFFFFu, got)) { ok = false; break; }
                }
#pragma unroll
                for (int gi = 0; gi < G; ++gi) {
                    if (SCALE == SCALE_BLOCK_B) f[gi] = (kBlocksPerWarp == 1 || ((col0 + 32 * gi) >> 7) == blk0) ? fq[0][0] : fq[kBlocksPerWarp - 1][0];
                    else f[gi] = vslot[q * 32 + lane];
                }
                if (SCALE == SCALE_BLOCK_B) {
#pragma unroll
                    for (int b = 0; b < kBlocksPerWarp; ++b) { fq[b][0] = fq[b][1]; fq[b][1] = fq[b][2]; fq[b][2] = fq[b][3]; }
                }
                // barrier that announces this chunk's partial sums (see the MMA issuer)
                const uint32_t done_bar = (KIND == MmaKind::F8F6F4) ? empty_bar(cc % S) : tfull_bar(a);
                const uint32_t done_par = (KIND == MmaKind::F8F6F4) ? ((cc / S) & 1u) : ((cc >> 1) & 1u);
                {
                    const bool got = mbar_wait(done_bar, done_par, abort_flag, g.wait_limit_ns);
                    if (!__all_sync(0xFFFFFFFFu, got)) { ok = false; break; }
                }
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN + h * HALF;
                // two 32-column groups in registers next to the accumulators
                uint32_t v[2][GC];
                tmem_ld_cols(taddr, v[0]);
                if (G > 1) tmem_ld_cols(taddr + GC, v[1]);
                if (SCALE != SCALE_NONE) {
                    // In the shadow of the first load.  Block mode: with the last chunk of a group of four the register
                    // queue is empty; the next group's slot (requested four chunks ago) is turned into the next four
                    // factors and the slot of the group just finished is refilled two groups ahead.  One warp barrier
                    // per four chunks: between the copies of all lanes and the reads of all lanes.
                    if (SCALE == SCALE_BLOCK_B) {
                        if ((c & 3) == 3) {
                            cp_async_wait<0>();
                            __syncwarp();
                            load_factors((c >> 2) + 1);
                            prefetch_group((c >> 2) + 2);
                        }
                    }
                }
                // all of this warp's reads of buffer `a` are done: hand it back to the MMA warp
                auto release_buffer = [&]() {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(a));
                };
                auto consume_group = [&](int gi, const uint32_t (&cur)[GC]) {
                    if (SCALE == SCALE_NONE) {
                        float o[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(cur[i]);
                        if (row_ok) store32<OUT_F32>(g, row, col0 + 32 * gi, o);
                    } else if (SCALE == SCALE_BLOCK_B) {
                        const float2 ff = make_float2(f[gi], f[gi]);
#pragma unroll
                        for (int i = 0; i < GC / 2; ++i)
                            acc[(GC / 2) * gi + i] = __ffma2_rn(make_float2(__uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1])), ff, acc[(GC / 2) * gi + i]);
                    } else {
                        const float2 ff = make_float2(f[0], f[0]);
                        const float4 *sbv = reinterpret_cast<const float4 *>(slot + GC * gi);
#pragma unroll
                        for (int i = 0; i < GC / 4; ++i) {
                            const float4 s4 = sbv[i];   // reciprocal column scales, broadcast read
                            const float2 r0 = make_float2(s4.x, s4.y);
                            const float2 r1 = make_float2(s4.z, s4.w);
                            const float2 p0 = __fmul2_rn(make_float2(__uint_as_float(cur[4 * i]), __uint_as_float(cur[4 * i + 1])), r0);
                            const float2 p1 = __fmul2_rn(make_float2(__uint_as_float(cur[4 * i + 2]), __uint_as_float(cur[4 * i + 3])), r1);
                            acc[(GC / 2) * gi + 2 * i] = __ffma2_rn(p0, ff, acc[(GC / 2) * gi + 2 * i]);
                            acc[(GC / 2) * gi + 2 * i + 1] = __ffma2_rn(p1, ff, acc[(GC / 2) * gi + 2 * i + 1]);
                        }
                    }
                };
                // Two loads are in flight from the start; each group's FMAs free its registers for the load two groups
                // on.  A load is waited for one group after it was issued, before the next one is issued (the wait covers
                // every outstanding load of the thread), so that its latency lies under that group's FMAs and no group is
                // consumed before its load has been waited for.  The buffer goes back to the MMA warp when the last load
                // has landed; the last group follows the release.
                tmem_ld_wait();
                if (G <= 2) release_buffer();
#pragma unroll
                for (int gi = 0; gi < G; ++gi) {
                    consume_group(gi, v[gi & 1]);
                    if (gi >= 1 && gi + 1 < G) tmem_ld_wait();                   // group gi+1 has landed
                    if (gi + 2 < G) tmem_ld_cols(taddr + GC * (gi + 2), v[gi & 1]);
                    if (G > 2 && gi + 2 == G) release_buffer();                  // ... and it was the chunk's last load
                }
                if (SCALE == SCALE_VEC_B && (cc % C::kVecBlock) == C::kVecBlock - 1) {
                    __syncwarp();                        // every lane has read the block's slots
                    if (lane == 0) mbar_arrive(vempty_bar(vd / C::kVecBlock));
                }
            }
            if (SCALE != SCALE_NONE) {
                cp_async_wait<0>();
                if (ok) {
                    if (C::kTmaOut && !g.accumulate) {
                        // round, stage 32 rows x 64 bytes in shared memory (16-byte chunks XOR-swizzled the way
                        // the output tensor map's 64-byte swizzle expects) and let the TMA unit write each box;
                        // rows and columns outside the matrix are clipped by the hardware
                        constexpr int kPerBox = OUT_F32 ? 16 : 32;   // output columns per 64-byte box row
#pragma unroll
                        for (int b = 0; b < HALF / kPerBox; ++b) {
                            if (lane == 0) bulk_wait_read0();     // the previous box has left the staging tile
                            __syncwarp();
                            const float *src = reinterpret_cast<const float *>(acc) + b * kPerBox;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                uint4 o;
                                if (OUT_F32) o = make_uint4(__float_as_uint(src[4 * j]), __float_as_uint(src[4 * j + 1]), __float_as_uint(src[4 * j + 2]), __float_as_uint(src[4 * j + 3]));
                                else o = make_uint4(pack_bf16x2(src[8 * j], src[8 * j + 1]), pack_bf16x2(src[8 * j + 2], src[8 * j + 3]),
                                                    pack_bf16x2(src[8 * j + 4], src[8 * j + 5]), pack_bf16x2(src[8 * j + 6], src[8 * j + 7]));
                                st_shared_v4(stage_u32 + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4), o);
                            }
                            fence_proxy_async();
                            __syncwarp();
                            const int col = col0 + b * kPerBox;
                            if (lane == 0 && col < g.No && row0 < g.Mo) { tma_store_2d(&tmO, stage_u32, col, row0); bulk_commit(); }
                        }
                    } else {
                        bool write_out = true;
                        if (SCALE == SCALE_VEC_B && wi.nsl > 1) {
                            // A slice of a sliced tile: this warp's 32 x HALF sums go to the slice's slot (512 contiguous bytes
                            // per store instruction); the warp that delivers a sub-tile's last slice adds all slices in slice
                            // order, whoever came last, so the result does not depend on the order of arrival.
                            float *av = reinterpret_cast<float *>(acc);
                            constexpr size_t kWarpFloats = 32 * HALF;
                            float *first = g.partials + (size_t)(wi.tail * wi.nsl) * kNumEpiWarps * kWarpFloats + e * kWarpFloats + lane * 4;
                            float *mine = first + (size_t)wi.slice * kNumEpiWarps * kWarpFloats;
#pragma unroll
                            for (int j4 = 0; j4 < HALF / 4; ++j4)
                                __stcg(reinterpret_cast<float4 *>(mine + j4 * 128), make_float4(av[4 * j4], av[4 * j4 + 1], av[4 * j4 + 2], av[4 * j4 + 3]));
                            __threadfence();
                            __syncwarp();
                            uint32_t old = 0;
                            if (lane == 0) old = atomicAdd(g.counters + wi.tail * kNumEpiWarps + e, 1u);
                            old = __shfl_sync(0xFFFFFFFFu, old, 0);
                            write_out = (old == (uint32_t)wi.nsl - 1u);
                            if (write_out) {
                                __threadfence();
#pragma unroll
                                for (int j4 = 0; j4 < HALF / 4; ++j4) {
                                    float4 v = __ldcg(reinterpret_cast<const float4 *>(first + j4 * 128));
                                    for (int sl = 1; sl < wi.nsl; ++sl) {
                                        const float4 u = __ldcg(reinterpret_cast<const float4 *>(first + (size_t)sl * kNumEpiWarps * kWarpFloats + j4 * 128));
                                        v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
                                    }
                                    av[4 * j4] = v.x; av[4 * j4 + 1] = v.y; av[4 * j4 + 2] = v.z; av[4 * j4 + 3] = v.w;
                                }
                            }
                        }
                        if (write_out && row_ok) {
#pragma unroll
                            for (int gi = 0; gi < HALF / 32; ++gi) store32<OUT_F32>(g, row, col0 + 32 * gi, reinterpret_cast<const float *>(acc) + 32 * gi);
                        }
                    }
                }
                __syncwarp();
            }
        }
        if (lane == 0) bulk_wait_all0();   // outstanding output stores have read their staging tiles
    }

    // ---- teardown: every role ends here, tensor memory is always released ------------------
    __syncwarp();
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before the CTA's resources go away
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        if (threadIdx.x == 0) atomicExch(g.status, (uint32_t)SNIP_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc<false>(tmem_base, C::kTmemCols);
    }
}

// Simple bf16 transpose (used only for BF16-tagged dgrad / wgrad operands).
__global__ void transpose_bf16_kernel(const uint16_t *__restrict__ in, uint16_t *__restrict__ out, int64_t rows, int64_t cols)
{
    __shared__ uint16_t tile[64][66];
    const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;
    for (int i = threadIdx.y; i < 64; i += blockDim.y) {
        const int64_t r = r0 + i, c = c0 + threadIdx.x * 2;
        if (r < rows && c < cols) {
            const uint32_t v = *reinterpret_cast<const uint32_t *>(in + r * cols + c);
            tile[i][threadIdx.x * 2] = (uint16_t)(v & 0xFFFFu);
            tile[i][threadIdx.x * 2 + 1] = (uint16_t)(v >> 16);
        }
    }
    __syncthreads();
    for (int i = threadIdx.y; i < 64; i += blockDim.y) {
        const int64_t c = c0 + i, r = r0 + threadIdx.x * 2;
        if (c < cols && r < rows) {
            const uint32_t v = (uint32_t)tile[threadIdx.x * 2][i] | ((uint32_t)tile[threadIdx.x * 2 + 1][i] << 16);
            *reinterpret_cast<uint32_t *>(out + c * rows + r) = v;
        }
    }
}

// ---- host side ---------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map over a row-major [rows][kc] operand whose rows are `row_bytes` apart, fetched in
// boxes of (128 bytes of K) x box_rows with the 128-byte swizzle.
int make_operand_map(CUtensorMap *map, const void *ptr, CUtensorMapDataType dt, int64_t rows, int64_t kc_elems,
                     int64_t row_bytes, int box_x_elems, int box_rows, CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) { snprintf(last_error_buffer(), 256, "cuTensorMapEncodeTiled entry point not found"); return SNIP_ERR_CUDA; }
    cuuint64_t dims[2] = {(cuuint64_t)kc_elems, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    cuuint32_t box[2] = {(cuuint32_t)box_x_elems, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(last_error_buffer(), 256, "cuTensorMapEncodeTiled failed: CUresult %d (rows %lld, k %lld, row bytes %lld, dtype %d)",
                 (int)r, (long long)rows, (long long)kc_elems, (long long)row_bytes, (int)dt);
        return SNIP_ERR_CUDA;
    }
    return SNIP_OK;
}

int sm_count()
{
    static thread_local int dev_cached = -1, n = 0;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev != dev_cached) { cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev); dev_cached = dev; }
    return n;
}

template <MmaKind KIND, int BN, int SCALE, bool OUT_F32>
int launch_gemm(const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmO, const GemmArgs &g, uint32_t idesc, cudaStream_t st)
{
    using C = Cfg<KIND, BN, SCALE>;
    auto kern = gemm_kernel<KIND, BN, SCALE, OUT_F32>;
    // a per-function, per-device attribute; setting it on every launch is cheap and correct on any device
    SNIP_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
    const int num_tiles = (int)(ceil_div(g.Mo, BM) * ceil_div(g.No, BN));
    const int sms = sm_count();
    GemmArgs ga = g;
    ga.split_first = num_tiles; ga.nsplit = 1; ga.num_items = num_tiles;
    if (SCALE == SCALE_VEC_B && g.partials && sms > 0) {
        // The tiles of the last, partial wave (all tiles, if there are fewer than SMs) are cut along the contraction into as
        // many slices as there are SMs to take them: at most kMaxSlices, none shorter than kMinSliceStages stages.
        const int full = (num_tiles / sms) * sms, rest = num_tiles - full;
        const int num_kstages = (int)ceil_div(g.Kc, C::kStageK);
        int ns = rest > 0 ? sms / rest : 1;
        if (ns > kMaxSlices) ns = kMaxSlices;
        while (ns > 1 && (num_kstages / ns < kMinSliceStages || rest * ns > kMaxSlicedItems)) --ns;
        if (ns > 1) {
            ga.split_first = full; ga.nsplit = ns; ga.num_items = full + rest * ns;
            SNIP_CUDA_TRY(cudaMemsetAsync(g.counters, 0, (size_t)rest * kNumEpiWarps * sizeof(uint32_t), st));
        }
    }
    const int grid = ga.num_items < sms ? ga.num_items : sms;
    kern<<<grid, kGemmThreads, C::kSmemBytes, st>>>(tmA, tmB, tmO, ga, idesc);
    SNIP_CUDA_TRY(cudaGetLastError());
    return SNIP_OK;
}

template <MmaKind KIND, int BN>
int launch_gemm_scale(int scale, bool out_f32, const CUtensorMap &tmA, const CUtensorMap &tmB, const CUtensorMap &tmO, const GemmArgs &g,
                      uint32_t idesc, cudaStream_t st)
{
    if (scale == SCALE_BLOCK_B)
        return out_f32 ? launch_gemm<KIND, BN, SCALE_BLOCK_B, true>(tmA, tmB, tmO, g, idesc, st)
                       : launch_gemm<KIND, BN, SCALE_BLOCK_B, false>(tmA, tmB, tmO, g, idesc, st);
    return out_f32 ? launch_gemm<KIND, BN, SCALE_VEC_B, true>(tmA, tmB, tmO, g, idesc, st)
                   : launch_gemm<KIND, BN, SCALE_VEC_B, false>(tmA, tmB, tmO, g, idesc, st);
}

}  // namespace

size_t gemm_ws_bytes() { return 256; }
// Workspace with which the weight-gradient product may slice the tiles of its last wave along the contraction:
// status word, arrival counters, one FP32 tile per slice.
size_t gemm_ws_bytes_sliced() { return kSliceCountersOffset + kSliceCountersBytes + (size_t)kMaxSlicedItems * BM * 256 * sizeof(float); }

// Testing hooks (snip_debug_set): process-wide, off by default.
namespace {
std::atomic<long long> g_wait_limit_ns{2000000000ll};   // bound of every device-side wait of the GEMM kernels
std::atomic<int> g_tx_skew{0};                           // bytes added to what a stage's barrier expects (a wait that cannot complete)
std::atomic<int> g_slicing{1};                           // 0: the weight-gradient product never slices its last wave
std::atomic<int> g_kernel_choice{0};                     // 0, 1 = single-CTA kernels, 2 = CTA-pair kernels for quantized operands
}  // namespace

// The hooks' current values, for the other GEMM families (gemm_mx.cu).
void gemm_debug_hooks(uint64_t *wait_limit_ns, int *tx_skew)
{
    *wait_limit_ns = (uint64_t)g_wait_limit_ns.load();
    *tx_skew = g_tx_skew.load();
}

int gemm_pair_impl(int fmt_a, int fmt_b, const void *a_codes, const void *b_codes, int64_t Mo, int64_t No, int64_t Kc, const float *sa,
                   int64_t sa_chunk_stride, const float *sb, int64_t sb_chunk_stride, int64_t sb_blk_stride, int scale_mode, void *out,
                   int out_dtype, int accumulate, uint32_t *status, uint64_t wait_limit_ns, int tx_skew, cudaStream_t st);

// Zeroes the status word of a GEMM workspace (enqueued; allocates nothing).
int gemm_clear_status(void *ws, cudaStream_t st)
{
    SNIP_CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(uint32_t), st));
    return SNIP_OK;
}

// Shared with the power-of-two-scale GEMMs: 2-D tiled tensor map over a row-major matrix.
int make_tiled_map_2d(CUtensorMap *map, const void *ptr, int dtype, int64_t rows, int64_t inner_elems, int64_t row_bytes, int box_x_elems,
                      int box_rows, int swizzle)
{
    return make_operand_map(map, ptr, static_cast<CUtensorMapDataType>(dtype), rows, inner_elems, row_bytes, box_x_elems, box_rows,
                            static_cast<CUtensorMapSwizzle>(swizzle));
}
int gemm_sm_count() { return sm_count(); }

int transpose_bf16(const void *in, void *out, int64_t rows, int64_t cols, cudaStream_t st)
{
    dim3 grid((unsigned)ceil_div(cols, 64), (unsigned)ceil_div(rows, 64)), block(32, 8);
    transpose_bf16_kernel<<<grid, block, 0, st>>>(static_cast<const uint16_t *>(in), static_cast<uint16_t *>(out), rows, cols);
    SNIP_CUDA_TRY(cudaGetLastError());
    return SNIP_OK;
}

// Core GEMM over stored operands.  a_codes: [Mo][Kc] and b_codes: [No][Kc], contraction-major.
// scale_mode: SCALE_NONE for BF16, SCALE_BLOCK_B (fwd / dgrad), SCALE_VEC_B (wgrad).
int gemm_impl(int fmt_a, int fmt_b, const void *a_codes, const void *b_codes, int64_t Mo, int64_t No, int64_t Kc, const float *sa,
              int64_t sa_chunk_stride, const float *sb, int64_t sb_chunk_stride, int64_t sb_blk_stride, int scale_mode, void *out,
              int out_dtype, int accumulate, void *ws, size_t ws_bytes, cudaStream_t st, bool clear_status)
{
    if (!a_codes || !b_codes || !out) return SNIP_ERR_ARG;
    if (!valid_dim(Mo) || !valid_dim(No) || !valid_dim(Kc) || Mo > INT32_MAX || No > INT32_MAX || Kc > INT32_MAX) return SNIP_ERR_SHAPE;
    if (out_dtype != SNIP_OUT_BF16 && out_dtype != SNIP_OUT_FP32) return SNIP_ERR_ARG;
    if (accumulate && out_dtype != SNIP_OUT_FP32) return SNIP_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < gemm_ws_bytes()) return SNIP_ERR_WORKSPACE;
    if (!aligned16(a_codes) || !aligned16(b_codes) || !aligned16(out) || !aligned16(ws)) return SNIP_ERR_ALIGN;
    const bool a16 = fmt_a == SNIP_FMT_BF16, b16 = fmt_b == SNIP_FMT_BF16;
    if (a16 != b16) return SNIP_ERR_UNSUPPORTED;
    if (!a16 && (!sa || !sb)) return SNIP_ERR_ARG;
    if (!a16 && (!aligned16(sa) || !aligned16(sb))) return SNIP_ERR_ALIGN;   // scale factors are fetched 16 bytes at a time
    int rc = require_sm100();
    if (rc != SNIP_OK) return rc;
    // The status word starts at zero for this call unless the caller runs several GEMMs against one word
    // and has cleared it itself (an earlier GEMM's timeout must survive the later ones).
    if (clear_status) { rc = gemm_clear_status(ws, st); if (rc) return rc; }

    GemmArgs g;
    g.Mo = (int32_t)Mo; g.No = (int32_t)No; g.Kc = (int32_t)Kc;
    g.sa = sa; g.sa_chunk_stride = sa_chunk_stride;
    g.sb = sb; g.sb_chunk_stride = sb_chunk_stride; g.sb_blk_stride = sb_blk_stride;
    g.out = out; g.ldo = No; g.accumulate = accumulate;
    g.status = static_cast<uint32_t *>(ws);
    g.split_first = 0; g.nsplit = 1; g.num_items = 0;   // set per launch
    g.partials = nullptr; g.counters = nullptr;
    if (!a16 && scale_mode == SCALE_VEC_B && ws_bytes >= gemm_ws_bytes_sliced() && g_slicing.load()) {
        g.counters = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(ws) + kSliceCountersOffset);
        g.partials = reinterpret_cast<float *>(static_cast<uint8_t *>(ws) + kSliceCountersOffset + kSliceCountersBytes);
    }
    g.stage_tx_bytes = 0;
    g.wait_limit_ns = (uint64_t)g_wait_limit_ns.load();
    const int tx_skew = g_tx_skew.load();
    const bool f32 = out_dtype == SNIP_OUT_FP32;

    // The CTA-pair kernels (gemm_pair.cu) are an alternative form of the same product, kept for comparison: they
    // run only when asked for through snip_debug_set (on the 7B shapes they are slower than the kernels below).
    const int choice = g_kernel_choice.load();
    if (!a16 && choice == 2)
        return gemm_pair_impl(fmt_a, fmt_b, a_codes, b_codes, Mo, No, Kc, sa, sa_chunk_stride, sb, sb_chunk_stride, sb_blk_stride, scale_mode,
                              out, out_dtype, accumulate, g.status, g.wait_limit_ns, tx_skew, st);

    CUtensorMap tmA, tmB, tmO;
    // output boxes of 32 rows x 64 bytes for the TMA stores of the block-mode epilogue
    rc = f32 ? make_operand_map(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Mo, No, No * 4, 16, 32, CU_TENSOR_MAP_SWIZZLE_64B)
             : make_operand_map(&tmO, out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Mo, No, No * 2, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
    if (rc) return rc;
    if (a16) {
        rc = make_operand_map(&tmA, a_codes, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, Mo, Kc, Kc * 2, 64, BM);
        if (rc) return rc;
        rc = make_operand_map(&tmB, b_codes, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, No, Kc, Kc * 2, 64, 256);
        if (rc) return rc;
        const uint32_t idesc = make_idesc(1, 1, BM, 256);
        g.stage_tx_bytes = (BM + 256) * 128 + tx_skew;
        return f32 ? launch_gemm<MmaKind::F16, 256, SCALE_NONE, true>(tmA, tmB, tmO, g, idesc, st)
                   : launch_gemm<MmaKind::F16, 256, SCALE_NONE, false>(tmA, tmB, tmO, g, idesc, st);
    }
    if (fmt_a == SNIP_FMT_FP4_E2M1 && fmt_b == SNIP_FMT_FP4_E2M1 && (Kc % 128) != 0) {
        // Packed FP4 on both sides, contraction length ending in a 64-wide tile: kind::mxf4 on the packed bytes
        // (fetched as plain u8, exact extents).  Whole chunks take the path below instead: the per-chunk
        // promotion, not the tensor pipe, sets the pace of these kernels, and there a 128x256 tile of
        // kind::f8f6f4 (FP4 codes expanded by the TMA unit, still fetched packed from L2) does a third more
        // columns per hand-off than the 128x192 tile that tensor memory allows next to kind::mxf4's scale
        // factors: measured 10-20 % faster on the 7B shapes.
        constexpr int BN = 192;
        rc = make_operand_map(&tmA, a_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, Kc / 2, Kc / 2, 128, BM);
        if (rc) return rc;
        rc = make_operand_map(&tmB, b_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, No, Kc / 2, Kc / 2, 128, BN);
        if (rc) return rc;
        const uint32_t idesc = make_idesc_block_scaled(1, 1, BM, BN);
        g.stage_tx_bytes = (BM + BN) * 128 + tx_skew;
        return launch_gemm_scale<MmaKind::MXF4, BN>(scale_mode, f32, tmA, tmB, tmO, g, idesc, st);
    }
    // FP8 x FP8, the mixed pairs and FP4 x FP4 over whole chunks: kind::f8f6f4; FP4 operands are expanded by
    // the TMA unit to one 16-byte-aligned group per 16 elements, which is the layout this MMA kind reads
    constexpr int BN = 256;
    const bool a4 = fmt_a == SNIP_FMT_FP4_E2M1, b4 = fmt_b == SNIP_FMT_FP4_E2M1;
    // The expanding 4-bit tensor-map type only accepts an inner extent that is a multiple of 128
    // elements.  A contraction length ending in a 64-wide tile is therefore declared rounded up: the
    // extra 64 codes of each row are the first codes of the next row (for the last row, 32 bytes of
    // the slack that snip_quantize_sizes reserves); they meet zero-filled FP8 codes of the other
    // operand, whose map has the exact extent, so they contribute nothing.  (Two FP4 operands with such a
    // length never get here: both maps would be padded.)
    const int64_t kpad = ceil_div(Kc, 128) * 128;
    rc = make_operand_map(&tmA, a_codes, a4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, Mo, a4 ? kpad : Kc,
                          a4 ? Kc / 2 : Kc, 128, BM);
    if (rc) return rc;
    rc = make_operand_map(&tmB, b_codes, b4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, No, b4 ? kpad : Kc,
                          b4 ? Kc / 2 : Kc, 128, BN);
    if (rc) return rc;
    const uint32_t idesc = make_idesc(a4 ? 5 : 0, b4 ? 5 : 0, BM, BN);
    // an FP4 operand expanded by the TMA unit occupies 128 B per row in shared memory but reports
    // only its 64 packed source bytes to the barrier
    g.stage_tx_bytes = BM * (a4 ? 64 : 128) + BN * (b4 ? 64 : 128) + tx_skew;
    return launch_gemm_scale<MmaKind::F8F6F4, BN>(scale_mode, f32, tmA, tmB, tmO, g, idesc, st);
}

}  // namespace snip

extern "C" int snip_gemm_quantized(int op, const snip_qtensor_t *a, const snip_qtensor_t *b, void *out, int out_dtype,
                                   int accumulate, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!a || !b || op < SNIP_OP_FWD || op > SNIP_OP_WGRAD) return SNIP_ERR_ARG;
    if (!valid_fmt(a->fmt) || !valid_fmt(b->fmt)) return SNIP_ERR_ARG;
    const bool q = a->fmt != SNIP_FMT_BF16;
    int64_t Mo, No, Kc;
    const float *sa = a->scales, *sb = b->scales;
    int64_t sa_cs, sb_cs, sb_bs;
    int mode;
    if (op == SNIP_OP_FWD) {
        // A = X[M,K] ROW tiles, B = W[N,K] blocks
        if (a->cols != b->cols || a->transposed || b->transposed) return SNIP_ERR_SHAPE;
        if (q && (a->block != SNIP_BLOCK_ROW_1x128 || b->block != SNIP_BLOCK_BLK_128x128)) return SNIP_ERR_UNSUPPORTED;
        Mo = a->rows; No = b->rows; Kc = a->cols;
        sa_cs = Mo; sb_bs = ceil_div(Kc, 128); sb_cs = 1; mode = SCALE_BLOCK_B;
    } else if (op == SNIP_OP_DGRAD) {
        // A = dY[M,N] ROW tiles, B = W[N,K] blocks stored transposed ([K,N])
        if (a->cols != b->rows || a->transposed || !b->transposed) return SNIP_ERR_SHAPE;
        if (q && (a->block != SNIP_BLOCK_ROW_1x128 || b->block != SNIP_BLOCK_BLK_128x128)) return SNIP_ERR_UNSUPPORTED;
        Mo = a->rows; No = b->cols; Kc = a->cols;
        sa_cs = Mo; sb_bs = 1; sb_cs = ceil_div(No, 128); mode = SCALE_BLOCK_B;
    } else {
        // A = dY[M,N] COL tiles stored transposed ([N,M]), B = X[M,K] COL tiles stored transposed ([K,M])
        if (a->rows != b->rows || !a->transposed || !b->transposed) return SNIP_ERR_SHAPE;
        if (q && (a->block != SNIP_BLOCK_COL_128x1 || b->block != SNIP_BLOCK_COL_128x1)) return SNIP_ERR_UNSUPPORTED;
        Mo = a->cols; No = b->cols; Kc = a->rows;
        sa_cs = Mo; sb_cs = No; sb_bs = 0; mode = SCALE_VEC_B;
    }
    if (!q) mode = SCALE_NONE;
    return gemm_impl(a->fmt, b->fmt, a->codes, b->codes, Mo, No, Kc, sa, sa_cs, sb, sb_cs, sb_bs, mode, out, out_dtype, accumulate,
                     ws, ws_bytes, static_cast<cudaStream_t>(stream), true);
}

extern "C" int snip_debug_set(int key, long long value)
{
    using namespace snip;
    switch (key) {
        case SNIP_DEBUG_WAIT_LIMIT_NS: if (value <= 0) return SNIP_ERR_ARG; g_wait_limit_ns.store(value); return SNIP_OK;
        case SNIP_DEBUG_TX_SKEW_BYTES: if (value < 0 || value > 4096 || (value % 16) != 0) return SNIP_ERR_ARG; g_tx_skew.store((int)value); return SNIP_OK;
        case SNIP_DEBUG_GEMM_KERNEL: if (value < 0 || value > 2) return SNIP_ERR_ARG; g_kernel_choice.store((int)value); return SNIP_OK;
        case SNIP_DEBUG_GEMM_SLICING: if (value < 0 || value > 1) return SNIP_ERR_ARG; g_slicing.store((int)value); return SNIP_OK;
        default: return SNIP_ERR_ARG;
    }
}

extern "C" int snip_poll_status(const void *ws, int *status_host)
{
    using namespace snip;
    if (!ws || !status_host) return SNIP_ERR_ARG;
    uint32_t v = 0;
    SNIP_CUDA_TRY(cudaMemcpy(&v, ws, sizeof(v), cudaMemcpyDeviceToHost));
    *status_host = (int)v;
    return SNIP_OK;
}
