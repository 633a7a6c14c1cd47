// Per-block-scaled quantizers BF16 -> FP8 E4M3 / FP4 E2M1 with fused error-norm statistics.
//
// Computes, per tile (paper Sec. 2.3):  amax = max|x|,  S = FPX_MAX / amax,
// code = RNE_fmt(x * S);  and per tensor (Sec. 3.1, Step 1)  sum x^2 and sum (x - code/S)^2.
// Tile kinds: 1x128 along the columns (ROW), 128x1 along the rows (COL), 128x128 (BLK).
//
// Memory-bound design: one CTA owns a 128x128 bf16 tile; each of its 256 threads holds an
// 8x8 sub-block in registers (eight 128-bit loads in flight per thread), so every element is
// read from HBM exactly once and the three tile kinds differ only in how the block-amax is
// reduced (16-lane shuffles for ROW, a small shared-memory exchange for COL, both for BLK).
// Codes are written with 64/128-bit stores; transposed outputs are staged through an
// XOR-swizzled shared-memory tile so that the global stores stay fully coalesced.
#include <cuda_bf16.h>
#include <float.h>

#include "common.cuh"
#include "quant_device.cuh"

namespace snip {

int gemm_sm_count();  // gemm.cu: SM count of the current device (cached per device)

namespace {

constexpr int kTile = 128;
constexpr int kThreads = 256;

struct CtaPartial {  // one per CTA, reduced in fixed order by stats_reduce_kernel
    double sumsq_x;
    double sumsq_err;
    float amax;
    float pad[3];
};

struct QuantArgs {
    const uint16_t *x;
    int64_t rows, cols, ld;
    uint8_t *codes;       // may be null (NO_CODES)
    float *scales;        // may be null (NO_CODES)
    CtaPartial *partials; // may be null (no stats)
    float2 *row_partials; // [col tiles][rows] {sum x^2, sum err^2}; may be null
    int64_t tiles_r, tiles_c, ntiles;
    int pow2;             // 1: power-of-two scale rule (largest 2^e with amax * 2^e <= FPX_MAX)
    uint32_t *sf;         // optional: UE8M0 bytes of 1/S in 512-byte atoms for hardware block scaling; null if unused
};

// Shared memory of one CTA (one 128x128 tile).
struct QuantShared {
    __align__(16) uint8_t stage[kTile * kTile];  // transposed codes of the tile (FP8 uses all 16 KB)
    uint32_t col_amax[8][kTile / 2];              // packed bf16 pairs, one row per warp
    float col_scale[kTile];
    float col_ninv[kTile];
    float red_f[8][3];
};

// Tile (r, c) of an nr x nc grid of 128x128 tiles.
struct Tile {
    int r, c, nr, nc;
};
// Running sums of one CTA over the tiles it processes (held by thread 0).
struct StatsAcc {
    double x = 0.0, e = 0.0;
    float m = 0.0f;
};

// The kernels are persistent: a CTA walks over tiles t = blockIdx.x, blockIdx.x + gridDim.x, ... (row-major
// tile order).  Each thread fetches its own 8x8 sub-block (eight 16-byte cp.async) into a private slot of
// shared memory and reads it back itself, so the hand-off needs no barrier: cp.async.wait_group is the
// only wait.  The next tile's fetch is issued as soon as the current one has been encoded, so it is in
// flight during the write-out and while the other resident CTAs compute.
constexpr int kStageBytes = kTile * kTile * 2;

__device__ __forceinline__ void prefetch_tile(const QuantArgs &a, int tr, int tc, uint8_t *stage_base)
{
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t rbase = (int64_t)tr * kTile + 8 * ty, cbase = (int64_t)tc * kTile + 8 * tx;
    const bool ok = cbase < a.cols && rbase < a.rows;       // dims are multiples of 64: all 64 elements or none
    const uint16_t *xb = a.x + (ok ? rbase * a.ld + cbase : 0);
    const uint32_t ld32 = (uint32_t)a.ld;
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(stage_base) + tid * 16;
    const int nbytes = ok ? 16 : 0;                          // 0: the slot is zero-filled, nothing is read
#pragma unroll
    for (int p = 0; p < 8; ++p)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + p * (kThreads * 16)), "l"(xb + (ok ? p * ld32 : 0)), "r"(nbytes) : "memory");
}
__device__ __forceinline__ void prefetch_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void prefetch_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// One output of the tile whose 8x8 sub-block of this thread sits in slot[p * kThreads], p = 0..7 (shared memory;
// re-read where needed instead of held in registers, which keeps four CTAs resident per SM).
// FMT: target format (BF16 = statistics only).  BLOCK: tile kind.  TRANSPOSED: codes stored as
// the transpose.  CODES: write codes and scales.  STATS: accumulate sums.  ROWSTATS: per-row sums.
template <int FMT, int BLOCK, bool TRANSPOSED, bool CODES, bool STATS, bool ROWSTATS>
__device__ __forceinline__ void quantize_tile(const QuantArgs &a, const Tile &tl, const uint4 *slot, QuantShared &sh, StatsAcc &acc)
{
    constexpr bool kQuant = (FMT != SNIP_FMT_BF16);
    constexpr int kCodeBytes8 = (FMT == SNIP_FMT_FP8_E4M3) ? 8 : 4;  // bytes per 8 elements
    constexpr int kRowBytes = kTile * kCodeBytes8 / 8;               // staged bytes per line
    uint8_t *const stage = sh.stage;
    auto &col_amax = sh.col_amax;
    auto &col_scale = sh.col_scale;
    auto &col_ninv = sh.col_ninv;
    auto &red_f = sh.red_f;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t r0 = (int64_t)tl.r * kTile, c0 = (int64_t)tl.c * kTile;
    const int64_t rbase = r0 + 8 * ty, cbase = c0 + 8 * tx;
    const bool col_ok = cbase < a.cols;  // cols is a multiple of 64, so 8-groups never straddle

    // ---- block amax -> scales --------------------------------------------------------
    float s_row[8], s_col[8];  // scale per row p (ROW) / per column j (COL); BLK uses s_row[0]
    float n_row[8], n_col[8];  // matching -1/S for the error term
    (void)s_row; (void)s_col; (void)n_row; (void)n_col;
    float my_amax = 0.0f;      // this thread's amax, for the tensor-wide statistic
    if (kQuant || STATS) {
        uint32_t rmax[8];      // per row: packed max over the 8 columns (as 4 pairs folded)
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const uint4 vp = slot[p * kThreads];
            uint32_t m = absmax2(0u, vp.x);
            m = absmax2(m, vp.y);
            m = absmax2(m, vp.z);
            m = absmax2(m, vp.w);
            rmax[p] = m;
        }
        if (BLOCK == SNIP_BLOCK_ROW_1x128 && kQuant) {
            // fold pairs, pack two rows per register, reduce across the 16 lanes of the row
            uint32_t pk[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t m0 = rmax[2 * q], m1 = rmax[2 * q + 1];
                m0 = max2(m0, m0 >> 16);  // low half = row 2q
                m1 = max2(m1, m1 << 16);  // high half = row 2q+1
                pk[q] = (m0 & 0xFFFFu) | (m1 & 0xFFFF0000u);
            }
#pragma unroll
            for (int off = 1; off < 16; off <<= 1)
#pragma unroll
                for (int q = 0; q < 4; ++q) pk[q] = max2(pk[q], __shfl_xor_sync(0xFFFFFFFFu, pk[q], off));
            // lane (tx & 7) derives the scale of row p = tx & 7, then the 8 scales are shared
            const int myp = tx & 7;
            uint32_t sel = pk[0];
#pragma unroll
            for (int q = 1; q < 4; ++q) sel = ((myp >> 1) == q) ? pk[q] : sel;
            float am = (myp & 1) ? bf16hi(sel) : bf16lo(sel);
            float mine = tile_scale<FMT>(am, a.pow2);
            float mine_ninv = neg_inv_scale<FMT>(am, mine, a.pow2);
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                s_row[p] = __shfl_sync(0xFFFFFFFFu, mine, (lane & 16) | p);
                if (STATS) n_row[p] = __shfl_sync(0xFFFFFFFFu, mine_ninv, (lane & 16) | p);
            }
            if (STATS) {
#pragma unroll
                for (int q = 0; q < 4; ++q) my_amax = fmaxf(my_amax, fmaxf(bf16lo(pk[q]), bf16hi(pk[q])));
            }
            if (CODES && tx == 0 && a.sf) {
                // atom [row tile][column tile]: word (r % 32) * 4 + r / 32 holds row r's byte four times
                uint32_t *atom = a.sf + ((int64_t)tl.r * tl.nc + tl.c) * 128;
#pragma unroll
                for (int p = 0; p < 8; ++p) {
                    const int r = 8 * ty + p;
                    atom[(r & 31) * 4 + (r >> 5)] = (rbase + p < a.rows) ? sf_word(s_row[p]) : 0x7F7F7F7Fu;
                }
            }
            if (CODES && tx == 0) {
                // scales[tile j][row]: eight consecutive rows per thread
                float *dst = a.scales + (int64_t)tl.c * a.rows + rbase;
                if (rbase < a.rows) {
                    *reinterpret_cast<float4 *>(dst) = make_float4(s_row[0], s_row[1], s_row[2], s_row[3]);
                    *reinterpret_cast<float4 *>(dst + 4) = make_float4(s_row[4], s_row[5], s_row[6], s_row[7]);
                }
            }
        } else {
            // column maxima over this thread's 8 rows (4 packed registers = 8 columns)
            uint32_t cm[4] = {0, 0, 0, 0};
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                const uint4 vp = slot[p * kThreads];
                cm[0] = absmax2(cm[0], vp.x);
                cm[1] = absmax2(cm[1], vp.y);
                cm[2] = absmax2(cm[2], vp.z);
                cm[3] = absmax2(cm[3], vp.w);
            }
            if (BLOCK == SNIP_BLOCK_COL_128x1 && kQuant) {
                // the two row groups of a warp, then the 8 warps through shared memory
#pragma unroll
                for (int q = 0; q < 4; ++q) cm[q] = max2(cm[q], __shfl_xor_sync(0xFFFFFFFFu, cm[q], 16));
                if (lane < 16)
                    *reinterpret_cast<uint4 *>(&col_amax[warp][4 * tx]) = make_uint4(cm[0], cm[1], cm[2], cm[3]);
                __syncthreads();
                if (tid < kTile) {
                    const uint16_t *h = reinterpret_cast<const uint16_t *>(&col_amax[0][0]);
                    uint32_t m = 0;
#pragma unroll
                    for (int w = 0; w < 8; ++w) m = max(m, (uint32_t)h[w * kTile + tid]);  // non-negative bf16: integer order
                    float am = __uint_as_float(m << 16);
                    float s = tile_scale<FMT>(am, a.pow2);
                    col_scale[tid] = s;
                    col_ninv[tid] = neg_inv_scale<FMT>(am, s, a.pow2);
                    // atom [column tile][row tile] (the operand is consumed transposed): one word per column
                    if (CODES && a.sf) a.sf[((int64_t)tl.c * tl.nr + tl.r) * 128 + (tid & 31) * 4 + (tid >> 5)] = (c0 + tid < a.cols) ? sf_word(s) : 0x7F7F7F7Fu;
                    if (CODES && c0 + tid < a.cols) a.scales[(int64_t)tl.r * a.cols + c0 + tid] = s;
                    if (STATS) my_amax = am;
                }
                __syncthreads();
                const float4 s0 = *reinterpret_cast<const float4 *>(&col_scale[8 * tx]);
                const float4 s1 = *reinterpret_cast<const float4 *>(&col_scale[8 * tx + 4]);
                s_col[0] = s0.x; s_col[1] = s0.y; s_col[2] = s0.z; s_col[3] = s0.w;
                s_col[4] = s1.x; s_col[5] = s1.y; s_col[6] = s1.z; s_col[7] = s1.w;
                if (STATS) {
                    const float4 n0 = *reinterpret_cast<const float4 *>(&col_ninv[8 * tx]);
                    const float4 n1 = *reinterpret_cast<const float4 *>(&col_ninv[8 * tx + 4]);
                    n_col[0] = n0.x; n_col[1] = n0.y; n_col[2] = n0.z; n_col[3] = n0.w;
                    n_col[4] = n1.x; n_col[5] = n1.y; n_col[6] = n1.z; n_col[7] = n1.w;
                }
            } else {
                // BLK (or statistics-only): one amax for the whole CTA tile
                uint32_t m = max2(max2(cm[0], cm[1]), max2(cm[2], cm[3]));
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) m = max2(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
                float am = fmaxf(bf16lo(m), bf16hi(m));
                if (lane == 0) red_f[warp][2] = am;
                __syncthreads();
                float bm = red_f[0][2];
#pragma unroll
                for (int w = 1; w < 8; ++w) bm = fmaxf(bm, red_f[w][2]);
                my_amax = bm;
                if (kQuant) {
                    s_row[0] = tile_scale<FMT == SNIP_FMT_BF16 ? SNIP_FMT_FP8_E4M3 : FMT>(bm, a.pow2);
                    n_row[0] = neg_inv_scale<FMT == SNIP_FMT_BF16 ? SNIP_FMT_FP8_E4M3 : FMT>(bm, s_row[0], a.pow2);
                    if (CODES && a.sf && tid < kTile) {
                        const int64_t atom = TRANSPOSED ? (int64_t)tl.c * tl.nr + tl.r : (int64_t)tl.r * tl.nc + tl.c;
                        a.sf[atom * 128 + tid] = sf_word(s_row[0]);
                    }
                    if (CODES && tid == 0) a.scales[(int64_t)tl.r * tl.nc + tl.c] = s_row[0];
                }
                __syncthreads();  // red_f is reused below
            }
        }
    }

    // ---- encode, statistics, store ------------------------------------------------------
    float sx = 0.0f, se = 0.0f;
    float rsx[8], rse[8];
    (void)rsx; (void)rse;
    if (kQuant) {
        float2 sc[4], ni[4];
        if (BLOCK == SNIP_BLOCK_COL_128x1) {
#pragma unroll
            for (int j = 0; j < 4; ++j) { sc[j] = make_float2(s_col[2 * j], s_col[2 * j + 1]); ni[j] = make_float2(n_col[2 * j], n_col[2 * j + 1]); }
        } else if (BLOCK == SNIP_BLOCK_BLK_128x128) {
#pragma unroll
            for (int j = 0; j < 4; ++j) { sc[j] = make_float2(s_row[0], s_row[0]); ni[j] = make_float2(n_row[0], n_row[0]); }
        }
        uint32_t codes[8][2];
        float2 sx2 = make_float2(0.0f, 0.0f), se2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            if (BLOCK == SNIP_BLOCK_ROW_1x128) {
#pragma unroll
                for (int j = 0; j < 4; ++j) { sc[j] = make_float2(s_row[p], s_row[p]); ni[j] = make_float2(n_row[p], n_row[p]); }
            }
            if (ROWSTATS) {
                float2 px = make_float2(0.0f, 0.0f), pe = make_float2(0.0f, 0.0f);
                quant8<FMT, STATS>(slot[p * kThreads], sc, ni, codes[p], px, pe);
                rsx[p] = px.x + px.y; rse[p] = pe.x + pe.y;
                sx += rsx[p]; se += rse[p];
            } else {
                quant8<FMT, STATS>(slot[p * kThreads], sc, ni, codes[p], sx2, se2);
            }
        }
        if (STATS && !ROWSTATS) { sx = sx2.x + sx2.y; se = se2.x + se2.y; }
        if (CODES) {
            if (!TRANSPOSED) {
                const int64_t out_ld = a.cols * kCodeBytes8 / 8;  // bytes per output row
                if (col_ok && rbase < a.rows) {
                    uint8_t *dst = a.codes + rbase * out_ld + cbase * kCodeBytes8 / 8;
                    const uint32_t ld32 = (uint32_t)out_ld;
#pragma unroll
                    for (int p = 0; p < 8; ++p) {
                        if (FMT == SNIP_FMT_FP8_E4M3)
                            *reinterpret_cast<uint2 *>(dst + p * ld32) = make_uint2(codes[p][0], codes[p][1]);
                        else
                            *reinterpret_cast<uint32_t *>(dst + p * ld32) = codes[p][0];
                    }
                }
            } else {
                // Transpose the 8x8 sub-block of codes in registers: for column j collect the
                // codes of rows p = 0..7, then stage line (8*tx + j) of the transposed tile.
                // Chunk index ty is XOR-ed with tx so that the 16 lanes of a row group hit
                // distinct banks.
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t lo = 0, hi = 0;
                    if (FMT == SNIP_FMT_FP8_E4M3) {
#pragma unroll
                        for (int p = 0; p < 8; ++p) {
                            uint32_t b = (codes[p][j >> 2] >> (8 * (j & 3))) & 0xFFu;
                            if (p < 4) lo |= b << (8 * p); else hi |= b << (8 * (p - 4));
                        }
                        uint2 *dst = reinterpret_cast<uint2 *>(stage + (8 * tx + j) * kRowBytes) + (ty ^ tx);
                        *dst = make_uint2(lo, hi);
                    } else {
#pragma unroll
                        for (int p = 0; p < 8; ++p) {
                            uint32_t b = (codes[p][0] >> (4 * j)) & 0xFu;
                            lo |= b << (4 * p);
                        }
                        uint32_t *dst = reinterpret_cast<uint32_t *>(stage + (8 * tx + j) * kRowBytes) + (ty ^ tx);
                        *dst = lo;
                    }
                }
                __syncthreads();
                // write out: line c of the staged tile holds rows r0..r0+127 of column c0+c
                const int64_t out_ld = a.rows * kCodeBytes8 / 8;  // bytes per transposed row
                constexpr int kChunks = kRowBytes / 16;            // 16-byte chunks per line
                const int valid_rows = (int)min((int64_t)kTile, a.rows - r0);
                for (int idx = tid; idx < kTile * kChunks; idx += kThreads) {
                    const int c = idx / kChunks, q = idx % kChunks;
                    if (c0 + c >= a.cols) continue;
                    const int key = (c >> 3) & 15;
                    uint4 o;
                    if (FMT == SNIP_FMT_FP8_E4M3) {
                        const uint2 *src = reinterpret_cast<const uint2 *>(stage + c * kRowBytes);
                        uint2 h0 = src[(2 * q) ^ key], h1 = src[(2 * q + 1) ^ key];
                        o = make_uint4(h0.x, h0.y, h1.x, h1.y);
                        if (16 * q >= valid_rows) continue;  // rows is a multiple of 64
                    } else {
                        const uint32_t *src = reinterpret_cast<const uint32_t *>(stage + c * kRowBytes);
                        o = make_uint4(src[(4 * q) ^ key], src[(4 * q + 1) ^ key], src[(4 * q + 2) ^ key],
                                       src[(4 * q + 3) ^ key]);
                        if (32 * q >= valid_rows) continue;
                    }
                    uint8_t *dst = a.codes + (c0 + c) * out_ld + r0 * kCodeBytes8 / 8 + 16 * q;
                    *reinterpret_cast<uint4 *>(dst) = o;
                }
            }
        }
    } else if (STATS) {
        // BF16: identity, only sum x^2
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const uint4 vp = slot[p * kThreads];
            const uint32_t w[4] = {vp.x, vp.y, vp.z, vp.w};
            float px = 0.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float x0 = bf16lo(w[i]), x1 = bf16hi(w[i]);
                px = fmaf(x0, x0, px);
                px = fmaf(x1, x1, px);
            }
            sx += px;
            if (ROWSTATS) { rsx[p] = px; rse[p] = 0.0f; }
        }
    }

    // ---- statistics: warp -> CTA -> one partial per CTA ------------------------------------
    if (ROWSTATS) {
        // per row: add the 16 lanes that share the row, lane tx==0 writes {sum x^2, sum err^2}
#pragma unroll
        for (int p = 0; p < 8; ++p) {
#pragma unroll
            for (int off = 1; off < 16; off <<= 1) {
                rsx[p] += __shfl_xor_sync(0xFFFFFFFFu, rsx[p], off);
                rse[p] += __shfl_xor_sync(0xFFFFFFFFu, rse[p], off);
            }
        }
        if (tx == 0 && rbase < a.rows) {
            float2 *dst = a.row_partials + (int64_t)tl.c * a.rows + rbase;
#pragma unroll
            for (int p = 0; p < 8; ++p) dst[p] = make_float2(rsx[p], rse[p]);
        }
    }
    if (STATS) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            sx += __shfl_xor_sync(0xFFFFFFFFu, sx, off);
            se += __shfl_xor_sync(0xFFFFFFFFu, se, off);
            my_amax = fmaxf(my_amax, __shfl_xor_sync(0xFFFFFFFFu, my_amax, off));
        }
        if (lane == 0) { red_f[warp][0] = sx; red_f[warp][1] = se; red_f[warp][2] = my_amax; }
        __syncthreads();
        if (tid == 0) {
            double dx = 0.0, de = 0.0;
            float am = 0.0f;
#pragma unroll
            for (int w = 0; w < 8; ++w) { dx += (double)red_f[w][0]; de += (double)red_f[w][1]; am = fmaxf(am, red_f[w][2]); }
            acc.x += dx;
            acc.e += de;
            acc.m = fmaxf(acc.m, am);
        }
    }
}

// Dynamic shared memory of the kernels: the tile slot, then the QuantShared scratch.
constexpr size_t kSmemBytes = (size_t)kStageBytes + sizeof(QuantShared);
constexpr int kCtasPerSm = 4;

__device__ __forceinline__ void write_partial(CtaPartial *partials, const StatsAcc &acc)
{
    if (threadIdx.x == 0) {
        CtaPartial *dst = partials + blockIdx.x;
        dst->sumsq_x = acc.x;
        dst->sumsq_err = acc.e;
        dst->amax = acc.m;
    }
}

// Walk of one CTA over its tiles without divisions in the loop.
struct TileWalk {
    int r, c, step_r, step_c, nr, nc;
    __device__ __forceinline__ TileWalk(int nr_, int nc_) : nr(nr_), nc(nc_)
    {
        r = (int)blockIdx.x / nc_; c = (int)blockIdx.x % nc_;
        step_r = (int)gridDim.x / nc_; step_c = (int)gridDim.x % nc_;
    }
    __device__ __forceinline__ bool valid() const { return r < nr; }
    __device__ __forceinline__ void next()
    {
        r += step_r; c += step_c;
        if (c >= nc) { c -= nc; ++r; }
    }
};

template <int FMT, int BLOCK, bool TRANSPOSED, bool CODES, bool STATS, bool ROWSTATS>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) quantize_kernel(const QuantArgs a)
{
    extern __shared__ __align__(128) uint8_t smem[];
    QuantShared &sh = *reinterpret_cast<QuantShared *>(smem + kStageBytes);
    const uint4 *slot = reinterpret_cast<const uint4 *>(smem) + threadIdx.x;
    // the statistics reduction that follows on the stream may be scheduled now; it waits for this
    // grid to finish before it reads anything (programmatic dependent launch)
    if (STATS) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    StatsAcc acc;
    TileWalk w((int)a.tiles_r, (int)a.tiles_c);
    if (w.valid()) prefetch_tile(a, w.r, w.c, smem);
    prefetch_commit();
    while (w.valid()) {
        prefetch_wait<0>();
        const Tile tl = {w.r, w.c, w.nr, w.nc};
        quantize_tile<FMT, BLOCK, TRANSPOSED, CODES, STATS, ROWSTATS>(a, tl, slot, sh, acc);
        w.next();
        if (w.valid()) prefetch_tile(a, w.r, w.c, smem);   // this thread's reads of its slot are done
        prefetch_commit();
        __syncthreads();  // the scratch arrays are reused by the next tile
    }
    if (STATS) write_partial(a.partials, acc);
}

// Two outputs from one read (the tile kinds a tensor is consumed with, paper Fig. 5): `a` as stored
// (1x128 tiles along the columns, or 128x128 blocks) and `b` transposed (128x1 tiles along the rows, or
// the same 128x128 blocks), each with its own format, scales and statistics.
struct DualArgs {
    QuantArgs a, b;
};
template <int FMT_A, int FMT_B, bool BLK, bool STATS>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) quantize_dual_kernel(const DualArgs d)
{
    extern __shared__ __align__(128) uint8_t smem[];
    QuantShared &sh = *reinterpret_cast<QuantShared *>(smem + kStageBytes);
    const uint4 *slot = reinterpret_cast<const uint4 *>(smem) + threadIdx.x;
    if (STATS) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    StatsAcc acc_a, acc_b;
    TileWalk w((int)d.a.tiles_r, (int)d.a.tiles_c);
    if (w.valid()) prefetch_tile(d.a, w.r, w.c, smem);
    prefetch_commit();
    while (w.valid()) {
        prefetch_wait<0>();
        const Tile tl = {w.r, w.c, w.nr, w.nc};
        quantize_tile<FMT_A, BLK ? SNIP_BLOCK_BLK_128x128 : SNIP_BLOCK_ROW_1x128, false, true, STATS, false>(d.a, tl, slot, sh, acc_a);
        __syncthreads();  // the scratch arrays are reused by the second output
        quantize_tile<FMT_B, BLK ? SNIP_BLOCK_BLK_128x128 : SNIP_BLOCK_COL_128x1, true, true, STATS, false>(d.b, tl, slot, sh, acc_b);
        w.next();
        if (w.valid()) prefetch_tile(d.a, w.r, w.c, smem);
        prefetch_commit();
        __syncthreads();
    }
    if (STATS) { write_partial(d.a.partials, acc_a); write_partial(d.b.partials, acc_b); }
}

// Fixed-order reduction of the per-CTA partials into one snip_stats_t (deterministic: every thread
// owns a fixed strided subset, warps combine with shuffles, warp results are added in warp order).
// Launched with programmatic stream serialization: it may start while the quantizer still runs and
// blocks in griddepcontrol.wait until that grid has completed and its writes are visible.
struct ReduceSets {
    const CtaPartial *partials[2];
    snip_stats_t *out[2];
};
__global__ void __launch_bounds__(1024) stats_reduce_kernel(const ReduceSets sets, int64_t n)
{
    __shared__ double sh_x[32], sh_e[32];
    __shared__ float sh_m[32];
    const CtaPartial *partials = sets.partials[blockIdx.x];
    snip_stats_t *out = sets.out[blockIdx.x];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    double dx = 0.0, de = 0.0;
    float am = 0.0f;
    for (int64_t i = threadIdx.x; i < n; i += 1024) {
        const double2 p = *reinterpret_cast<const double2 *>(&partials[i]);
        dx += p.x;
        de += p.y;
        am = fmaxf(am, partials[i].amax);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        dx += __shfl_xor_sync(0xFFFFFFFFu, dx, off);
        de += __shfl_xor_sync(0xFFFFFFFFu, de, off);
        am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, off));
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { sh_x[warp] = dx; sh_e[warp] = de; sh_m[warp] = am; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double tx = 0.0, te = 0.0;
        float tm = 0.0f;
        for (int w = 0; w < 32; ++w) { tx += sh_x[w]; te += sh_e[w]; tm = fmaxf(tm, sh_m[w]); }
        out->sumsq_x = tx;
        out->sumsq_err = te;
        out->amax = tm;
        out->reserved = 0;
    }
}

// Per-row sums: add the column-tile partials of each row in ascending tile order.
__global__ void row_stats_reduce_kernel(const float2 *row_partials, int64_t rows, int64_t col_tiles, double *row_stats)
{
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    double dx = 0.0, de = 0.0;
    for (int64_t j = 0; j < col_tiles; ++j) {
        float2 p = row_partials[j * rows + r];
        dx += (double)p.x;
        de += (double)p.y;
    }
    row_stats[2 * r] = dx;
    row_stats[2 * r + 1] = de;
}

// Launch of a persistent kernel: its dynamic shared memory exceeds the default limit, so the limit is
// raised first (a per-function, per-device attribute; setting it again is cheap).
template <typename Kernel, typename Args>
void launch_persistent(Kernel kernel, const Args &args, dim3 grid, cudaStream_t st)
{
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess) return;  // left in cudaGetLastError
    kernel<<<grid, kThreads, kSmemBytes, st>>>(args);
}

template <int FMT, int BLOCK, bool TRANSPOSED>
void launch_variant(const QuantArgs &a, bool codes, bool stats, bool rowstats, dim3 grid, cudaStream_t st)
{
    if (codes && stats && rowstats) launch_persistent(quantize_kernel<FMT, BLOCK, TRANSPOSED, true, true, true>, a, grid, st);
    else if (codes && stats) launch_persistent(quantize_kernel<FMT, BLOCK, TRANSPOSED, true, true, false>, a, grid, st);
    else if (codes) launch_persistent(quantize_kernel<FMT, BLOCK, TRANSPOSED, true, false, false>, a, grid, st);
    else if (rowstats) launch_persistent(quantize_kernel<FMT, BLOCK, false, false, true, true>, a, grid, st);
    else launch_persistent(quantize_kernel<FMT, BLOCK, false, false, true, false>, a, grid, st);
}

template <int FMT>
void launch_fmt(const QuantArgs &a, int block, bool transposed, bool codes, bool stats, bool rowstats, dim3 grid, cudaStream_t st)
{
    if (block == SNIP_BLOCK_ROW_1x128) {
        if (transposed) launch_variant<FMT, SNIP_BLOCK_ROW_1x128, true>(a, codes, stats, rowstats, grid, st);
        else launch_variant<FMT, SNIP_BLOCK_ROW_1x128, false>(a, codes, stats, rowstats, grid, st);
    } else if (block == SNIP_BLOCK_COL_128x1) {
        if (transposed) launch_variant<FMT, SNIP_BLOCK_COL_128x1, true>(a, codes, stats, rowstats, grid, st);
        else launch_variant<FMT, SNIP_BLOCK_COL_128x1, false>(a, codes, stats, rowstats, grid, st);
    } else {
        if (transposed) launch_variant<FMT, SNIP_BLOCK_BLK_128x128, true>(a, codes, stats, rowstats, grid, st);
        else launch_variant<FMT, SNIP_BLOCK_BLK_128x128, false>(a, codes, stats, rowstats, grid, st);
    }
}

// CTAs of a persistent launch over ntiles tiles: kCtasPerSm per SM (what the kernels' shared memory and
// registers allow), never more than there are tiles.
int64_t persistent_ctas(int64_t ntiles)
{
    const int64_t cap = kCtasPerSm * (int64_t)gemm_sm_count();
    return ntiles < cap ? ntiles : cap;
}

size_t stats_ws_bytes(int64_t rows, int64_t cols, bool rowstats)
{
    const int64_t tr = ceil_div(rows, kTile), tc = ceil_div(cols, kTile);
    size_t b = align_up((size_t)(tr * tc) * sizeof(CtaPartial), 256);
    if (rowstats) b += align_up((size_t)(tc * rows) * sizeof(float2), 256);
    return b;
}

}  // namespace

// Internal entry used by snip_quantize and by the linear-layer calls.
int quantize_impl_ex(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, int pow2, void *sf,
                     void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes, cudaStream_t st);

int quantize_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags,
                  void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes,
                  cudaStream_t st)
{
    return quantize_impl_ex(x, rows, cols, ld, fmt, block, flags, 0, nullptr, codes, scales, stats, row_stats, ws, ws_bytes, st);
}

// pow2 = 1 selects the power-of-two scale rule; sf (optional, needs pow2) receives the UE8M0 atoms.
int quantize_impl_ex(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, int pow2, void *sf,
                     void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (sf) {
        const bool tr = (flags & SNIP_Q_TRANSPOSED) != 0;
        // atoms follow the orientation the GEMM consumes: row tiles as stored, column tiles transposed
        if (!pow2 || !aligned16(sf) || (block == SNIP_BLOCK_ROW_1x128 && tr) || (block == SNIP_BLOCK_COL_128x1 && !tr)) return SNIP_ERR_UNSUPPORTED;
    }
    if (!x || !valid_fmt(fmt) || !valid_block(block)) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols) || ld < cols || (ld % 8) != 0) return SNIP_ERR_SHAPE;
    const bool want_stats = (flags & SNIP_Q_STATS) != 0;
    const bool want_rows = row_stats != nullptr;
    const bool want_codes = fmt != SNIP_FMT_BF16 && !(flags & SNIP_Q_NO_CODES);
    const bool transposed = (flags & SNIP_Q_TRANSPOSED) != 0;
    if (want_stats && !stats) return SNIP_ERR_ARG;
    if (want_codes && (!codes || !scales)) return SNIP_ERR_ARG;
    if (!want_codes && !want_stats && !want_rows) return SNIP_ERR_ARG;  // nothing to do
    if (!aligned16(x) || (want_codes && (!aligned16(codes) || !aligned16(scales))) || (stats && !aligned16(stats)) ||
        (row_stats && !aligned16(row_stats)))
        return SNIP_ERR_ALIGN;
    const bool any_stats = want_stats || want_rows;
    const size_t need = any_stats ? stats_ws_bytes(rows, cols, want_rows) : 0;
    if (need > 0 && (!ws || ws_bytes < need)) return SNIP_ERR_WORKSPACE;
    if (need > 0 && !aligned16(ws)) return SNIP_ERR_ALIGN;
    int rc = require_sm100();
    if (rc != SNIP_OK) return rc;

    const int64_t tr = ceil_div(rows, kTile), tc = ceil_div(cols, kTile);
    QuantArgs a;
    a.x = static_cast<const uint16_t *>(x);
    a.rows = rows; a.cols = cols; a.ld = ld;
    a.pow2 = pow2; a.sf = static_cast<uint32_t *>(sf);
    a.codes = want_codes ? static_cast<uint8_t *>(codes) : nullptr;
    a.scales = want_codes ? scales : nullptr;
    a.partials = any_stats ? static_cast<CtaPartial *>(ws) : nullptr;
    a.row_partials = want_rows ? reinterpret_cast<float2 *>(static_cast<uint8_t *>(ws) + align_up((size_t)(tr * tc) * sizeof(CtaPartial), 256)) : nullptr;
    a.tiles_r = tr; a.tiles_c = tc; a.ntiles = tr * tc;
    const int64_t nparts = persistent_ctas(tr * tc);
    dim3 grid((unsigned)nparts);
    if (fmt == SNIP_FMT_FP8_E4M3) launch_fmt<SNIP_FMT_FP8_E4M3>(a, block, transposed, want_codes, any_stats, want_rows, grid, st);
    else if (fmt == SNIP_FMT_FP4_E2M1) launch_fmt<SNIP_FMT_FP4_E2M1>(a, block, transposed, want_codes, any_stats, want_rows, grid, st);
    else launch_variant<SNIP_FMT_BF16, SNIP_BLOCK_BLK_128x128, false>(a, false, true, want_rows, grid, st);
    SNIP_CUDA_TRY(cudaGetLastError());
    if (want_stats) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1);
        cfg.blockDim = dim3(1024);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const ReduceSets sets = {{a.partials, nullptr}, {stats, nullptr}};
        SNIP_CUDA_TRY(cudaLaunchKernelEx(&cfg, stats_reduce_kernel, sets, nparts));
    }
    if (want_rows) {
        row_stats_reduce_kernel<<<(unsigned)ceil_div(rows, 256), 256, 0, st>>>(a.row_partials, rows, tc, row_stats);
        SNIP_CUDA_TRY(cudaGetLastError());
    }
    return SNIP_OK;
}

// One read, two outputs.  blk = false: a = 1x128 tiles as stored, b = 128x1 tiles transposed;
// blk = true: a = 128x128 blocks as stored, b = the same blocks transposed.
template <int FMT_A, int FMT_B>
static void launch_dual(const DualArgs &d, bool blk, bool stats, dim3 grid, cudaStream_t st)
{
    if (blk && stats) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, true, true>, d, grid, st);
    else if (blk) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, true, false>, d, grid, st);
    else if (stats) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, true>, d, grid, st);
    else launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, false>, d, grid, st);
}

int quantize_dual_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, bool blk, int pow2, const DualOut &oa, const DualOut &ob,
                       void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (!x) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols) || ld < cols || (ld % 8) != 0) return SNIP_ERR_SHAPE;
    const DualOut *o[2] = {&oa, &ob};
    for (int i = 0; i < 2; ++i) {
        if (o[i]->fmt != SNIP_FMT_FP8_E4M3 && o[i]->fmt != SNIP_FMT_FP4_E2M1) return SNIP_ERR_UNSUPPORTED;
        if (!o[i]->codes || !o[i]->scales) return SNIP_ERR_ARG;
        if (o[i]->sf && !pow2) return SNIP_ERR_UNSUPPORTED;
        if (!aligned16(o[i]->codes) || !aligned16(o[i]->scales) || (o[i]->sf && !aligned16(o[i]->sf)) ||
            (o[i]->stats && (reinterpret_cast<uintptr_t>(o[i]->stats) & 7u)))
            return SNIP_ERR_ALIGN;
    }
    if ((oa.stats == nullptr) != (ob.stats == nullptr)) return SNIP_ERR_ARG;
    if (!aligned16(x)) return SNIP_ERR_ALIGN;
    const bool stats = oa.stats != nullptr;
    const size_t one = stats_ws_bytes(rows, cols, false);
    if (stats && (!ws || ws_bytes < 2 * one)) return SNIP_ERR_WORKSPACE;
    if (stats && !aligned16(ws)) return SNIP_ERR_ALIGN;
    int rc = require_sm100();
    if (rc != SNIP_OK) return rc;
    const int64_t tr = ceil_div(rows, kTile), tc = ceil_div(cols, kTile);
    DualArgs d;
    for (int i = 0; i < 2; ++i) {
        QuantArgs &q = i ? d.b : d.a;
        q.x = static_cast<const uint16_t *>(x);
        q.rows = rows; q.cols = cols; q.ld = ld;
        q.codes = static_cast<uint8_t *>(o[i]->codes);
        q.scales = o[i]->scales;
        q.partials = stats ? reinterpret_cast<CtaPartial *>(static_cast<uint8_t *>(ws) + i * one) : nullptr;
        q.row_partials = nullptr;
        q.pow2 = pow2;
        q.sf = static_cast<uint32_t *>(o[i]->sf);
        q.tiles_r = tr; q.tiles_c = tc; q.ntiles = tr * tc;
    }
    const int64_t nparts = persistent_ctas(tr * tc);
    dim3 grid((unsigned)nparts);
    const bool a8 = oa.fmt == SNIP_FMT_FP8_E4M3, b8 = ob.fmt == SNIP_FMT_FP8_E4M3;
    if (a8 && b8) launch_dual<SNIP_FMT_FP8_E4M3, SNIP_FMT_FP8_E4M3>(d, blk, stats, grid, st);
    else if (a8) launch_dual<SNIP_FMT_FP8_E4M3, SNIP_FMT_FP4_E2M1>(d, blk, stats, grid, st);
    else if (b8) launch_dual<SNIP_FMT_FP4_E2M1, SNIP_FMT_FP8_E4M3>(d, blk, stats, grid, st);
    else launch_dual<SNIP_FMT_FP4_E2M1, SNIP_FMT_FP4_E2M1>(d, blk, stats, grid, st);
    SNIP_CUDA_TRY(cudaGetLastError());
    if (stats) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2);
        cfg.blockDim = dim3(1024);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const ReduceSets sets = {{d.a.partials, d.b.partials}, {oa.stats, ob.stats}};
        SNIP_CUDA_TRY(cudaLaunchKernelEx(&cfg, stats_reduce_kernel, sets, nparts));
    }
    return SNIP_OK;
}

}  // namespace snip

extern "C" int snip_quantize_sizes(int64_t rows, int64_t cols, int fmt, int block, uint32_t flags,
                                   size_t *codes_bytes, size_t *scales_bytes, size_t *ws_bytes)
{
    using namespace snip;
    if (!valid_fmt(fmt) || !valid_block(block)) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols)) return SNIP_ERR_SHAPE;
    const bool want_codes = fmt != SNIP_FMT_BF16 && !(flags & SNIP_Q_NO_CODES);
    size_t cb = 0, sb = 0;
    if (want_codes) {
        cb = (size_t)(rows * cols) / (fmt == SNIP_FMT_FP4_E2M1 ? 2 : 1);
        // 64 bytes of tail slack after FP4 codes: the GEMM's 4-bit tensor map may read (and ignore)
        // up to 32 bytes past the last row when the contraction length ends in a 64-wide tile
        if (fmt == SNIP_FMT_FP4_E2M1 && ((rows % 128) || (cols % 128))) cb += 64;
        const int64_t tr = ceil_div(rows, 128), tc = ceil_div(cols, 128);
        int64_t n = block == SNIP_BLOCK_ROW_1x128 ? tc * rows : block == SNIP_BLOCK_COL_128x1 ? tr * cols : tr * tc;
        sb = (size_t)n * sizeof(float);
    }
    if (codes_bytes) *codes_bytes = cb;
    if (scales_bytes) *scales_bytes = sb;
    if (ws_bytes) *ws_bytes = stats_ws_bytes(rows, cols, true);
    return SNIP_OK;
}

extern "C" int snip_quantize(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block,
                             uint32_t flags, void *codes, float *scales, snip_stats_t *stats, double *row_stats,
                             void *ws, size_t ws_bytes, void *stream)
{
    return snip::quantize_impl(x, rows, cols, ld, fmt, block, flags, codes, scales, stats, row_stats, ws, ws_bytes,
                               static_cast<cudaStream_t>(stream));
}

// ---- variant for callers that cannot allocate ------------------------------------------------
//
// Some users of this library cannot obtain scratch memory for us: a plug-in that runs inside a
// host application's fixed memory budget, or a service whose steady-state loop must never reach
// the CUDA allocator (cudaMalloc synchronizes the whole device and can fail under fragmentation).
// For them the statistics scratch lives in a fixed array inside the library's device image: every
// GPU that loads the library holds these kStaticScratchBytes until the process exits.
namespace snip {
namespace {

constexpr size_t kStaticScratchTiles = 16384;                                 // 128x128 tiles, e.g. 16384 x 16384 elements
constexpr size_t kStaticScratchBytes = kStaticScratchTiles * sizeof(CtaPartial);  // 512 KiB

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, not an address a kernel could use, so the address is looked up once per
// device (with that device current) and cached.
int static_scratch_address(void **out)
{
    constexpr int kMaxDevices = 64;
    static void *cached[kMaxDevices] = {nullptr};
    int dev = 0;
    SNIP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SNIP_ERR_UNSUPPORTED;
    void *p = __atomic_load_n(&cached[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        SNIP_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return SNIP_ERR_CUDA;
        __atomic_store_n(&cached[dev], p, __ATOMIC_RELEASE);   // every thread computes the same value
    }
    *out = p;
    return SNIP_OK;
}

}  // namespace
}  // namespace snip

extern "C" int snip_quantize_noalloc(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags,
                                     void *codes, float *scales, snip_stats_t *stats, void *stream)
{
    using namespace snip;
    if (!valid_dim(rows) || !valid_dim(cols)) return SNIP_ERR_SHAPE;
    const size_t need = stats_ws_bytes(rows, cols, false);
    if (need > kStaticScratchBytes) {
        snprintf(last_error_buffer(), 256, "snip_quantize_noalloc: %lld x %lld needs %zu bytes of scratch, the built-in array holds %zu",
                 (long long)rows, (long long)cols, need, kStaticScratchBytes);
        return SNIP_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != SNIP_OK) return rc;
    // Nothing in the scratch has to start at zero: every CTA overwrites its own partial before the
    // reduction kernel reads it, so stale contents of an earlier call are never observed.
    return quantize_impl(x, rows, cols, ld, fmt, block, flags, codes, scales, stats, nullptr, scratch, kStaticScratchBytes,
                         static_cast<cudaStream_t>(stream));
}

// ---- power-of-two ("MX-style") option -------------------------------------------------------

extern "C" int snip_quantize_mx_sizes(int64_t rows, int64_t cols, size_t *sf_bytes)
{
    using namespace snip;
    if (!sf_bytes) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols)) return SNIP_ERR_SHAPE;
    *sf_bytes = (size_t)(ceil_div(rows, 128) * ceil_div(cols, 128)) * 512;
    return SNIP_OK;
}

extern "C" int snip_quantize_mx(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags,
                                void *codes, float *scales, void *sf, snip_stats_t *stats, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (fmt == SNIP_FMT_BF16) return SNIP_ERR_UNSUPPORTED;
    return quantize_impl_ex(x, rows, cols, ld, fmt, block, flags, 1, sf, codes, scales, stats, nullptr, ws, ws_bytes,
                            static_cast<cudaStream_t>(stream));
}


// ---- one read, two outputs -------------------------------------------------------------------

extern "C" int snip_quantize_dual_workspace(int64_t rows, int64_t cols, size_t *ws_bytes)
{
    using namespace snip;
    if (!ws_bytes) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols)) return SNIP_ERR_SHAPE;
    *ws_bytes = 2 * stats_ws_bytes(rows, cols, false);
    return SNIP_OK;
}

extern "C" int snip_quantize_dual(const void *x, int64_t rows, int64_t cols, int64_t ld, int kind, int pow2_scale,
                                  const snip_qout_t *as_stored, const snip_qout_t *transposed, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    if (!as_stored || !transposed) return SNIP_ERR_ARG;
    if (kind != SNIP_DUAL_ROW_COLT && kind != SNIP_DUAL_BLK_BLKT) return SNIP_ERR_ARG;
    const DualOut oa = {as_stored->fmt, as_stored->codes, as_stored->scales, as_stored->sf, as_stored->stats};
    const DualOut ob = {transposed->fmt, transposed->codes, transposed->scales, transposed->sf, transposed->stats};
    return quantize_dual_impl(x, rows, cols, ld, kind == SNIP_DUAL_BLK_BLKT, pow2_scale ? 1 : 0, oa, ob, ws, ws_bytes,
                              static_cast<cudaStream_t>(stream));
}
