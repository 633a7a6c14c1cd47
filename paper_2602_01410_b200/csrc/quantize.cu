// Per-block-scaled quantizers BF16 -> FP8 E4M3 / FP4 E2M1 with fused error-norm statistics.
//
// Computes, per tile (paper Sec. 2.3):  amax = max|x|,  S = FPX_MAX / amax,
// code = RNE_fmt(x * S);  and per tensor (Sec. 3.1, Step 1)  sum x^2 and sum (x - code/S)^2.
// Tile kinds: 1x128 along the columns (ROW), 128x1 along the rows (COL), 128x128 (BLK).
//
// Design: persistent kernels, 256 threads per CTA, several CTAs per SM; a CTA walks over 128x128 bf16 tiles.
// Every thread fetches its own 8x8 sub-block with eight 16-byte cp.async copies into a private slot of a
// shared-memory tile and reads it back itself (the only wait is cp.async.wait_group); the next tile's fetch is
// in flight while this one is encoded, so every element is read from HBM exactly once.  The three tile kinds
// differ only in how the tile maxima are reduced (16-lane exchange for ROW, a small shared-memory exchange
// for COL, both for BLK).  Codes as stored leave straight from registers; transposed codes go through
// byte-permute 8x8 transposes and an XOR-swizzled shared-memory tile so that the global stores stay coalesced.
// The two-output form (quantize_dual_kernel) encodes each element under two scales in the same pass.
//
// Added options (paper Sec. 3.2 lets further quantization methods join the per-layer choices): the power-of-two scale
// rule on the same tiles or on 32-long tiles (ROW_1x32 / COL_32x1: the maxima are combined over 4 lanes / 2 warps
// instead of 16 lanes / 8 warps), with the scale exponents also written as the 512-byte atoms the block-scaled MMA
// reads; and the two-level form in the style of NVFP4 (quantize_nvfp4_dual_kernel: 16-long tiles = two neighbouring
// lanes / the two row groups of a warp, an E4M3 scale byte per tile, a per-tensor factor from a caller-supplied bound).
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
    int32_t rows, cols, ld;   // 32-bit (checked on the host): index products are 32 x 32 -> 64-bit multiplies
    uint8_t *codes;       // may be null (NO_CODES)
    float *scales;        // may be null (NO_CODES)
    CtaPartial *partials; // may be null (no stats)
    float2 *row_partials; // [col tiles][rows] {sum x^2, sum err^2}; may be null
    int32_t tiles_r, tiles_c;
    int64_t ntiles;
    uint64_t seed;        // stochastic rounding: key of the generator
    int pow2;             // 1: power-of-two scale rule (largest 2^e with amax * 2^e <= FPX_MAX)
    uint32_t *sf;         // optional: UE8M0 bytes of 1/S in 512-byte atoms for hardware block scaling; null if unused
                          // (two-level option: the E4M3 scale bytes, two atoms per 128x128 tile)
    const float *tensor_amax;   // two-level option: bound of the tensor's magnitudes (device); else unused
};

// Scratch shared memory of one CTA (next to the tile slot).
struct QuantShared {
    __align__(16) uint8_t stage[kTile * kTile];  // transposed codes of the tile (FP8 uses all 16 KB)
    uint32_t col_amax[8][kTile / 2];              // packed bf16 pairs, one row per warp
    float col_scale[kTile];
    float col_ninv[kTile];
    float row_scale[kTile];
    float row_ninv[kTile];
    uint32_t red_m[8];
    double red_d[8][4];
};

// Scratch of the 32-long tile kinds (kernels that use them ask for this much more shared memory): the scale of every
// 1x32 / 32x1 tile of the 128x128 tile, [32-block][line].
struct QuantShared32 {
    __align__(16) float row_scale[4][kTile];
    __align__(16) float col_scale[4][kTile];
};

// Scratch of the 16-long tile kinds (two-level option): the scale byte of every 1x16 / 16x1 tile of the 128x128 tile,
// [line][tile along the contraction], so that a line's four bytes of a half are one word.
struct QuantShared16 {
    __align__(16) uint8_t row_sf[kTile][8];
    __align__(16) uint8_t col_sf[kTile][8];
};
// Per-tensor factors of the two-level option: enc = 2688 / bound and its reciprocal.
struct TwoLevel {
    float enc = 1.0f, inv_enc = 1.0f;
};

// Tile (r, c) of an nr x nc grid of 128x128 tiles.
struct Tile {
    int r, c, nr, nc;
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
    const uint16_t *xb = a.x + (ok ? (int64_t)(int32_t)rbase * a.ld + cbase : 0);
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
// Compile-time description of one output of a tile pass.
template <int FMT_, int BLOCK_, bool TRANSPOSED_, bool CODES_, bool SR_ = false>
struct Out {
    static constexpr int FMT = FMT_, BLOCK = BLOCK_;
    static constexpr bool TRANSPOSED = TRANSPOSED_, CODES = CODES_, kQuant = (FMT_ != SNIP_FMT_BF16), SR = SR_;
    static_assert(!SR_ || FMT_ == SNIP_FMT_FP4_E2M1, "stochastic rounding is offered for FP4 E2M1 only");
};
struct NoOut {
    static constexpr int FMT = SNIP_FMT_BF16, BLOCK = SNIP_BLOCK_BLK_128x128;
    static constexpr bool TRANSPOSED = false, CODES = false, kQuant = false, SR = false;
};

// Per-thread running sums over the tiles of a CTA (binary64: one add per tile and sum).
struct ThreadStats {
    double x = 0.0, ea = 0.0, eb = 0.0;
    float amax = 0.0f;
};

// -1/S for the error term x - value(code)/S = x + value(code) * (-1/S).  Paper's rule: amax/FPX_MAX equals
// 1/S to within one rounding, which the statistics (1e-4) do not see; power-of-two rule: exact, from the
// exponent field.  For an empty tile the value is irrelevant (all codes are zero).
template <int FMT>
__device__ __forceinline__ float neg_inv(float amax, float s, int pow2)
{
    constexpr float kInvMax = (FMT == SNIP_FMT_FP8_E4M3) ? (1.0f / 448.0f) : (1.0f / 6.0f);
    return pow2 ? __uint_as_float(0x80000000u | ((254u << 23) - __float_as_uint(s))) : -amax * kInvMax;
}

// Two binary32 products -> packed codes of an element pair (FP8: 16 bits, FP4: 8 bits) and, with STATS,
// the squared error added to se2.
template <int FMT, bool STATS>
__device__ __forceinline__ uint32_t encode_pair(const float2 x, const float2 s, const float2 n, float2 &se2)
{
    const float2 t = __fmul2_rn(x, s);   // IEEE binary32 products, as the scalar definition asks for
    uint32_t c;
    if (FMT == SNIP_FMT_FP8_E4M3) c = cvt_e4m3x2(t.x, t.y);
    else c = cvt_e2m1x2(t.x, t.y);
    if (STATS) {
        const float2 d = (FMT == SNIP_FMT_FP8_E4M3) ? dec_e4m3x2(c) : dec_e2m1x2(c);
        const float2 e = __ffma2_rn(d, n, x);
        se2 = __ffma2_rn(e, e, se2);
    }
    return c;
}

// Stochastic-rounding form for FP4: u2 holds the two 16-bit uniforms of the pair (first element low).
// The rounded values are at hand in binary32, so the error term needs no decode.
template <bool STATS>
__device__ __forceinline__ uint32_t encode_pair_sr_fp4(const float2 x, const float2 s, const float2 n, uint32_t u2, float2 &se2)
{
    const float2 t = __fmul2_rn(x, s);
    const float2 v = make_float2(sr_e2m1_value(t.x, u2 & 0xFFFFu), sr_e2m1_value(t.y, u2 >> 16));
    if (STATS) {
        const float2 e = __ffma2_rn(v, n, x);
        se2 = __ffma2_rn(e, e, se2);
    }
    return cvt_e2m1x2(v.x, v.y);   // exact: v is representable
}

// Packs the four pair codes of 8 consecutive elements: FP8 -> two words, FP4 -> one word.
template <int FMT>
__device__ __forceinline__ void pack8(const uint32_t (&c)[4], uint32_t (&out)[2])
{
    if (FMT == SNIP_FMT_FP8_E4M3) {
        out[0] = c[0] | (c[1] << 16);
        out[1] = c[2] | (c[3] << 16);
    } else {
        out[0] = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
        out[1] = 0;
    }
}

// Address of this thread's codes of row rbase in the as-stored (row-major) output; row p follows p * out_ld bytes later.
template <int FMT>
__device__ __forceinline__ uint8_t *row_store_base(const QuantArgs &a, int64_t rbase, int64_t cbase, uint32_t &out_ld)
{
    constexpr int kCodeBytes8 = (FMT == SNIP_FMT_FP8_E4M3) ? 8 : 4;
    out_ld = (uint32_t)(a.cols * kCodeBytes8 / 8);
    return a.codes + (uint64_t)(uint32_t)rbase * out_ld + (uint32_t)cbase * kCodeBytes8 / 8;
}
// One 8-byte (FP8) or 4-byte (FP4) store per row.
template <int FMT>
__device__ __forceinline__ void store_row(uint8_t *dst, const uint32_t (&code)[2])
{
    if (FMT == SNIP_FMT_FP8_E4M3) *reinterpret_cast<uint2 *>(dst) = make_uint2(code[0], code[1]);
    else *reinterpret_cast<uint32_t *>(dst) = code[0];
}

// 4x4 byte transpose: t[j] byte i = a[i] byte j (eight byte permutes).
__device__ __forceinline__ void transpose4x4_bytes(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t (&t)[4])
{
    const uint32_t x0 = __byte_perm(a0, a1, 0x5140), x1 = __byte_perm(a0, a1, 0x7362);
    const uint32_t y0 = __byte_perm(a2, a3, 0x5140), y1 = __byte_perm(a2, a3, 0x7362);
    t[0] = __byte_perm(x0, y0, 0x5410);
    t[1] = __byte_perm(x0, y0, 0x7632);
    t[2] = __byte_perm(x1, y1, 0x5410);
    t[3] = __byte_perm(x1, y1, 0x7632);
}

// Transposes this thread's 8x8 codes in registers and stages them: line (8*tx + j) of the transposed tile
// gets the codes of rows 8*ty .. 8*ty+7 of column 8*tx + j.  The chunk index ty is XOR-ed with tx so that
// the 16 lanes of a row group hit distinct banks.
template <int FMT>
__device__ __forceinline__ void stage_transposed(uint8_t *stage, int tx, int ty, const uint32_t (&codes)[8][2])
{
    constexpr int kRowBytes = (FMT == SNIP_FMT_FP8_E4M3) ? kTile : kTile / 2;
    if (FMT == SNIP_FMT_FP8_E4M3) {
        // codes[p][h]: bytes of columns 4h .. 4h+3 of row p; four 4x4 byte transposes
        uint32_t lo[2][4], hi[2][4];   // [h][j]: rows 0-3 / rows 4-7 of column 4h + j
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            transpose4x4_bytes(codes[0][h], codes[1][h], codes[2][h], codes[3][h], lo[h]);
            transpose4x4_bytes(codes[4][h], codes[5][h], codes[6][h], codes[7][h], hi[h]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            reinterpret_cast<uint2 *>(stage + (8 * tx + j) * kRowBytes)[ty ^ tx] = make_uint2(lo[j >> 2][j & 3], hi[j >> 2][j & 3]);
    } else {
        // codes[p][0]: eight nibbles (columns 0..7) of row p.  Pair rows (2q, 2q+1) into bytes, even and odd
        // columns apart: ev[q] byte k = column 2k, od[q] byte k = column 2k+1 (low nibble = row 2q); a 4x4
        // byte transpose of each then gives the eight-row word of every column.
        uint32_t ev[4], od[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t r0 = codes[2 * q][0], r1 = codes[2 * q + 1][0];
            ev[q] = (r0 & 0x0F0F0F0Fu) | ((r1 << 4) & 0xF0F0F0F0u);
            od[q] = ((r0 >> 4) & 0x0F0F0F0Fu) | (r1 & 0xF0F0F0F0u);
        }
        uint32_t te[4], to[4];
        transpose4x4_bytes(ev[0], ev[1], ev[2], ev[3], te);
        transpose4x4_bytes(od[0], od[1], od[2], od[3], to);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            reinterpret_cast<uint32_t *>(stage + (8 * tx + 2 * k) * kRowBytes)[ty ^ tx] = te[k];
            reinterpret_cast<uint32_t *>(stage + (8 * tx + 2 * k + 1) * kRowBytes)[ty ^ tx] = to[k];
        }
    }
}

// Writes the staged transposed tile: line c holds rows r0 .. r0+127 of column c0 + c; 16-byte stores.
template <int FMT>
__device__ __forceinline__ void write_transposed(const QuantArgs &a, const uint8_t *stage, int64_t r0, int64_t c0)
{
    constexpr int kCodeBytes8 = (FMT == SNIP_FMT_FP8_E4M3) ? 8 : 4;
    constexpr int kRowBytes = kTile * kCodeBytes8 / 8;
    constexpr int kChunks = kRowBytes / 16;
    const uint32_t out_ld = (uint32_t)a.rows * kCodeBytes8 / 8;
    const int valid_rows = (int)min((int64_t)kTile, a.rows - r0);   // rows is a multiple of 64
    const int valid_cols = (int)min((int64_t)kTile, a.cols - c0);
    uint8_t *base = a.codes + (uint64_t)(uint32_t)c0 * out_ld + (uint32_t)r0 * kCodeBytes8 / 8;
#pragma unroll
    for (int idx = threadIdx.x; idx < kTile * kChunks; idx += kThreads) {
        const int c = idx / kChunks, q = idx % kChunks;
        const int key = (c >> 3) & 15;
        uint4 o;
        bool ok = c < valid_cols;
        if (FMT == SNIP_FMT_FP8_E4M3) {
            const uint2 *src = reinterpret_cast<const uint2 *>(stage + c * kRowBytes);
            const uint2 h0 = src[(2 * q) ^ key], h1 = src[(2 * q + 1) ^ key];
            o = make_uint4(h0.x, h0.y, h1.x, h1.y);
            ok = ok && 16 * q < valid_rows;
        } else {
            const uint32_t *src = reinterpret_cast<const uint32_t *>(stage + c * kRowBytes);
            o = make_uint4(src[(4 * q) ^ key], src[(4 * q + 1) ^ key], src[(4 * q + 2) ^ key], src[(4 * q + 3) ^ key]);
            ok = ok && 32 * q < valid_rows;
        }
        if (ok) *reinterpret_cast<uint4 *>(base + (uint64_t)(uint32_t)c * out_ld + 16 * q) = o;
    }
}

// Scales of one output for this thread's 8x8 sub-block.
struct SubScales {
    float s_row[8], n_row[8];   // 1x128 tiles: one per row p
    float s_col[8], n_col[8];   // 128x1 tiles: one per column j
    float s_blk, n_blk;         // 128x128 block
};

template <class O>
__device__ __forceinline__ float2 scale_pair(const SubScales &sc, int p, int i)
{
    if (O::BLOCK == SNIP_BLOCK_ROW_1x128 || O::BLOCK == SNIP_BLOCK_ROW_1x32 || O::BLOCK == SNIP_BLOCK_ROW_1x16) return make_float2(sc.s_row[p], sc.s_row[p]);
    if (O::BLOCK == SNIP_BLOCK_COL_128x1 || O::BLOCK == SNIP_BLOCK_COL_32x1 || O::BLOCK == SNIP_BLOCK_COL_16x1) return make_float2(sc.s_col[2 * i], sc.s_col[2 * i + 1]);
    return make_float2(sc.s_blk, sc.s_blk);
}
template <class O>
__device__ __forceinline__ float2 ninv_pair(const SubScales &sc, int p, int i)
{
    if (O::BLOCK == SNIP_BLOCK_ROW_1x128 || O::BLOCK == SNIP_BLOCK_ROW_1x32 || O::BLOCK == SNIP_BLOCK_ROW_1x16) return make_float2(sc.n_row[p], sc.n_row[p]);
    if (O::BLOCK == SNIP_BLOCK_COL_128x1 || O::BLOCK == SNIP_BLOCK_COL_32x1 || O::BLOCK == SNIP_BLOCK_COL_16x1) return make_float2(sc.n_col[2 * i], sc.n_col[2 * i + 1]);
    return make_float2(sc.n_blk, sc.n_blk);
}

// Row scales.  rmax[p]: this thread's packed partial maxima of row p (sign bits meaningless).  The 16 lanes
// of a row group combine them with an exchange-halving butterfly (5 shuffles instead of 16): after it, lane
// tx holds the maxima of rows 2q and 2q+1, q = 2*bit3(tx) + bit2(tx).  Lane tx with bit1 = 0 then owns row
// 2q + bit0: it derives the scale (one division per lane), writes the global scale / atom word and
// publishes scale and -1/S through shared memory; every lane reads back its eight rows after a warp barrier.
template <class O>
__device__ __forceinline__ void row_scales(const QuantArgs &a, const Tile &tl, QuantShared &sh, const uint32_t (&rmax)[8], int tx, int ty,
                                           int64_t rbase, SubScales &sc, float &amax_acc)
{
    uint32_t pk[4];   // rows 2q (low half) and 2q+1 (high half)
#pragma unroll
    for (int q = 0; q < 4; ++q)
        pk[q] = max2(__byte_perm(rmax[2 * q], rmax[2 * q + 1], 0x5410) & 0x7FFF7FFFu, __byte_perm(rmax[2 * q], rmax[2 * q + 1], 0x7632) & 0x7FFF7FFFu);
    const bool b3 = (tx & 8) != 0, b2 = (tx & 4) != 0;
    uint32_t k0 = b3 ? pk[2] : pk[0], k1 = b3 ? pk[3] : pk[1];
    const uint32_t g0 = b3 ? pk[0] : pk[2], g1 = b3 ? pk[1] : pk[3];
    k0 = max2(k0, __shfl_xor_sync(0xFFFFFFFFu, g0, 8));
    k1 = max2(k1, __shfl_xor_sync(0xFFFFFFFFu, g1, 8));
    uint32_t k = b2 ? k1 : k0;
    const uint32_t g = b2 ? k0 : k1;
    k = max2(k, __shfl_xor_sync(0xFFFFFFFFu, g, 4));
    k = max2(k, __shfl_xor_sync(0xFFFFFFFFu, k, 2));
    k = max2(k, __shfl_xor_sync(0xFFFFFFFFu, k, 1));
    const int myrow = ((tx >> 3) & 1) * 4 + ((tx >> 2) & 1) * 2 + (tx & 1);
    const float am = (tx & 1) ? bf16hi(k) : bf16lo(k);
    amax_acc = fmaxf(amax_acc, am);
    const float s = tile_scale<O::FMT>(am, a.pow2);
    if (!(tx & 2)) {
        const int r = 8 * ty + myrow;
        sh.row_scale[r] = s;
        sh.row_ninv[r] = neg_inv<O::FMT>(am, s, a.pow2);
        if (O::CODES) {
            // atom [row tile][column tile]: word (r % 32) * 4 + r / 32 holds row r's byte four times
            if (a.sf) a.sf[((int64_t)tl.r * tl.nc + tl.c) * 128 + (r & 31) * 4 + (r >> 5)] = (rbase + myrow < a.rows) ? sf_word(s) : 0x7F7F7F7Fu;
            if (rbase + myrow < a.rows) a.scales[(int64_t)tl.c * a.rows + rbase + myrow] = s;   // scales[tile j][row]
        }
    }
    __syncwarp();
    const float4 s0 = *reinterpret_cast<const float4 *>(&sh.row_scale[8 * ty]);
    const float4 s1 = *reinterpret_cast<const float4 *>(&sh.row_scale[8 * ty + 4]);
    const float4 n0 = *reinterpret_cast<const float4 *>(&sh.row_ninv[8 * ty]);
    const float4 n1 = *reinterpret_cast<const float4 *>(&sh.row_ninv[8 * ty + 4]);
    sc.s_row[0] = s0.x; sc.s_row[1] = s0.y; sc.s_row[2] = s0.z; sc.s_row[3] = s0.w;
    sc.s_row[4] = s1.x; sc.s_row[5] = s1.y; sc.s_row[6] = s1.z; sc.s_row[7] = s1.w;
    sc.n_row[0] = n0.x; sc.n_row[1] = n0.y; sc.n_row[2] = n0.z; sc.n_row[3] = n0.w;
    sc.n_row[4] = n1.x; sc.n_row[5] = n1.y; sc.n_row[6] = n1.z; sc.n_row[7] = n1.w;
}

// Column scales: thread tid < 128 owns column tid of the tile (its maximum is in sh.col_amax), publishes
// scale and -1/S through shared memory and writes the global scale / atom word.  Two barriers inside.
template <class O>
__device__ __forceinline__ void col_scales(const QuantArgs &a, const Tile &tl, QuantShared &sh, int tid, int tx, int64_t c0, SubScales &sc)
{
    __syncthreads();   // sh.col_amax complete
    if (tid < kTile) {
        const uint16_t *h = reinterpret_cast<const uint16_t *>(&sh.col_amax[0][0]);
        uint32_t m = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) m = max(m, (uint32_t)h[w * kTile + tid] & 0x7FFFu);  // non-negative bf16: integer order
        const float am = __uint_as_float(m << 16);
        const float s = tile_scale<O::FMT>(am, a.pow2);
        sh.col_scale[tid] = s;
        sh.col_ninv[tid] = neg_inv<O::FMT>(am, s, a.pow2);
        // atom [column tile][row tile] (the operand is consumed transposed): one word per column
        if (O::CODES && a.sf) a.sf[((int64_t)tl.c * tl.nr + tl.r) * 128 + (tid & 31) * 4 + (tid >> 5)] = (c0 + tid < a.cols) ? sf_word(s) : 0x7F7F7F7Fu;
        if (O::CODES && c0 + tid < a.cols) a.scales[(int64_t)tl.r * a.cols + c0 + tid] = s;
    }
    __syncthreads();
    const float4 s0 = *reinterpret_cast<const float4 *>(&sh.col_scale[8 * tx]);
    const float4 s1 = *reinterpret_cast<const float4 *>(&sh.col_scale[8 * tx + 4]);
    const float4 n0 = *reinterpret_cast<const float4 *>(&sh.col_ninv[8 * tx]);
    const float4 n1 = *reinterpret_cast<const float4 *>(&sh.col_ninv[8 * tx + 4]);
    sc.s_col[0] = s0.x; sc.s_col[1] = s0.y; sc.s_col[2] = s0.z; sc.s_col[3] = s0.w;
    sc.s_col[4] = s1.x; sc.s_col[5] = s1.y; sc.s_col[6] = s1.z; sc.s_col[7] = s1.w;
    sc.n_col[0] = n0.x; sc.n_col[1] = n0.y; sc.n_col[2] = n0.z; sc.n_col[3] = n0.w;
    sc.n_col[4] = n1.x; sc.n_col[5] = n1.y; sc.n_col[6] = n1.z; sc.n_col[7] = n1.w;
}

// -1/S of a power-of-two S, from its exponent field (exact).
__device__ __forceinline__ float neg_inv_pow2(float s) { return __uint_as_float(0x80000000u | ((254u << 23) - __float_as_uint(s))); }

// 1x32 tiles (power-of-two scales only).  The four lanes that share a 32-column piece of a row group combine their
// maxima with an exchange-halving butterfly (2 shuffles): lane tx then holds rows 4*bit1(tx) + 2*bit0(tx) and the next
// one of piece tx / 4.  It derives both scales, writes them out and publishes them; after a warp barrier every lane
// reads the eight scales of its own piece, and lanes 0..7 of the row group assemble the atom words of rows 8*ty + tx
// (the bytes of the row's four pieces in order).
template <class O>
__device__ __forceinline__ void row32_scales(const QuantArgs &a, const Tile &tl, QuantShared32 &s32, const uint32_t (&rmax)[8], int tx, int ty,
                                             int64_t rbase, SubScales &sc, float &amax_acc)
{
    uint32_t pk[4];   // rows 2q (low half) and 2q+1 (high half)
#pragma unroll
    for (int q = 0; q < 4; ++q)
        pk[q] = max2(__byte_perm(rmax[2 * q], rmax[2 * q + 1], 0x5410) & 0x7FFF7FFFu, __byte_perm(rmax[2 * q], rmax[2 * q + 1], 0x7632) & 0x7FFF7FFFu);
    const bool b1 = (tx & 2) != 0, b0 = (tx & 1) != 0;
    uint32_t k0 = b1 ? pk[2] : pk[0], k1 = b1 ? pk[3] : pk[1];
    const uint32_t g0 = b1 ? pk[0] : pk[2], g1 = b1 ? pk[1] : pk[3];
    k0 = max2(k0, __shfl_xor_sync(0xFFFFFFFFu, g0, 2));
    k1 = max2(k1, __shfl_xor_sync(0xFFFFFFFFu, g1, 2));
    uint32_t k = b0 ? k1 : k0;
    const uint32_t g = b0 ? k0 : k1;
    k = max2(k, __shfl_xor_sync(0xFFFFFFFFu, g, 1));
    const int piece = tx >> 2, r2 = (b1 ? 4 : 0) + (b0 ? 2 : 0);
    const float am0 = bf16lo(k), am1 = bf16hi(k);
    amax_acc = fmaxf(amax_acc, fmaxf(am0, am1));
    const float s0 = tile_scale<O::FMT>(am0, 1), s1 = tile_scale<O::FMT>(am1, 1);
    *reinterpret_cast<float2 *>(&s32.row_scale[piece][8 * ty + r2]) = make_float2(s0, s1);
    if (O::CODES && (int64_t)tl.c * kTile + 32 * piece < a.cols) {
        float *dst = a.scales + ((int64_t)tl.c * 4 + piece) * a.rows + rbase + r2;   // scales[32-piece j][row]
        if (rbase + r2 < a.rows) dst[0] = s0;
        if (rbase + r2 + 1 < a.rows) dst[1] = s1;
    }
    __syncwarp();
    const float4 v0 = *reinterpret_cast<const float4 *>(&s32.row_scale[piece][8 * ty]);
    const float4 v1 = *reinterpret_cast<const float4 *>(&s32.row_scale[piece][8 * ty + 4]);
    sc.s_row[0] = v0.x; sc.s_row[1] = v0.y; sc.s_row[2] = v0.z; sc.s_row[3] = v0.w;
    sc.s_row[4] = v1.x; sc.s_row[5] = v1.y; sc.s_row[6] = v1.z; sc.s_row[7] = v1.w;
#pragma unroll
    for (int p = 0; p < 8; ++p) sc.n_row[p] = neg_inv_pow2(sc.s_row[p]);
    if (O::CODES && a.sf && tx < 8) {
        const int r = 8 * ty + tx;
        uint32_t word = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) word |= ((254u - (__float_as_uint(s32.row_scale[b][r]) >> 23)) & 0xFFu) << (8 * b);
        a.sf[((int64_t)tl.r * tl.nc + tl.c) * 128 + (r & 31) * 4 + (r >> 5)] = (rbase + tx < a.rows) ? word : 0x7F7F7F7Fu;
    }
}

// 32x1 tiles (power-of-two scales only).  sh.col_amax holds each warp's maxima of its 16 rows; a 32-row piece is two
// warps.  Thread tid owns column tid % 128 and the pieces 2*(tid / 128) and the next one; after the second barrier
// every thread reads the eight scales of its columns in its own piece, and threads 0..127 assemble the atom word of
// their column.
template <class O>
__device__ __forceinline__ void col32_scales(const QuantArgs &a, const Tile &tl, QuantShared &sh, QuantShared32 &s32, int tid, int tx, int ty,
                                             int64_t r0, int64_t c0, SubScales &sc)
{
    __syncthreads();   // sh.col_amax complete
    {
        const uint16_t *h = reinterpret_cast<const uint16_t *>(&sh.col_amax[0][0]);
        const int col = tid & (kTile - 1);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int piece = 2 * (tid >> 7) + j;
            const uint32_t m = max((uint32_t)h[(2 * piece) * kTile + col] & 0x7FFFu, (uint32_t)h[(2 * piece + 1) * kTile + col] & 0x7FFFu);
            const float s = tile_scale<O::FMT>(__uint_as_float(m << 16), 1);
            s32.col_scale[piece][col] = s;
            if (O::CODES && c0 + col < a.cols && r0 + 32 * piece < a.rows) a.scales[((int64_t)tl.r * 4 + piece) * a.cols + c0 + col] = s;
        }
    }
    __syncthreads();
    const int piece = ty >> 2;
    const float4 v0 = *reinterpret_cast<const float4 *>(&s32.col_scale[piece][8 * tx]);
    const float4 v1 = *reinterpret_cast<const float4 *>(&s32.col_scale[piece][8 * tx + 4]);
    sc.s_col[0] = v0.x; sc.s_col[1] = v0.y; sc.s_col[2] = v0.z; sc.s_col[3] = v0.w;
    sc.s_col[4] = v1.x; sc.s_col[5] = v1.y; sc.s_col[6] = v1.z; sc.s_col[7] = v1.w;
#pragma unroll
    for (int j = 0; j < 8; ++j) sc.n_col[j] = neg_inv_pow2(sc.s_col[j]);
    if (O::CODES && a.sf && tid < kTile) {
        uint32_t word = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) word |= ((254u - (__float_as_uint(s32.col_scale[b][tid]) >> 23)) & 0xFFu) << (8 * b);
        // atom [column tile][row tile] (the operand is consumed transposed): one word per column
        a.sf[((int64_t)tl.c * tl.nr + tl.r) * 128 + (tid & 31) * 4 + (tid >> 5)] = (c0 + tid < a.cols) ? word : 0x7F7F7F7Fu;
    }
}

// Two-level option: scale byte, encode factor and (negated) decode factor of two tiles from their maxima.
//   d = (amax / 6) * enc in binary32;  sf = E4M3(d), nearest even, saturating;  E = enc / value(sf);  -value(sf) / enc
__device__ __forceinline__ uint32_t two_level_pair(float am0, float am1, const TwoLevel &tw, float &e0, float &e1, float &n0, float &n1)
{
    const float d0 = __fmul_rn(__fdiv_rn(am0, 6.0f), tw.enc), d1 = __fmul_rn(__fdiv_rn(am1, 6.0f), tw.enc);
    const uint32_t c = cvt_e4m3x2(d0, d1);          // low byte: first tile
    const float2 sv = dec_e4m3x2(c);
    e0 = sv.x == 0.0f ? 0.0f : __fdiv_rn(tw.enc, sv.x);
    e1 = sv.y == 0.0f ? 0.0f : __fdiv_rn(tw.enc, sv.y);
    n0 = -sv.x * tw.inv_enc;
    n1 = -sv.y * tw.inv_enc;
    return c;
}

// 1x16 tiles of the two-level option: a tile is the 8 columns of this lane and of its neighbour (lane ^ 1).  The two
// share the work (four IEEE divisions per pair of tiles): the even lane derives the factors of rows 0..3, the odd lane
// those of rows 4..7, each stages its scale bytes, and they swap the factors.  After a warp barrier lane tx of the row
// group writes the atom word of row 8*ty + tx%8, half tx/8 (the bytes of that half's four tiles in order).
template <class O>
__device__ __forceinline__ void row16_scales(const QuantArgs &a, const Tile &tl, QuantShared16 &s16, const TwoLevel &tw, const uint32_t (&rmax)[8],
                                             int tx, int ty, int64_t rbase, SubScales &sc, float &amax_acc)
{
    float am[8];
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        const uint32_t m = rmax[p] & 0x7FFF7FFFu;
        uint32_t mm = max(m & 0xFFFFu, m >> 16);                 // non-negative bf16: integer order
        mm = max(mm, __shfl_xor_sync(0xFFFFFFFFu, mm, 1));
        am[p] = __uint_as_float(mm << 16);
        amax_acc = fmaxf(amax_acc, am[p]);
    }
    const bool odd = (tx & 1) != 0;
    float e[4], n[4];
#pragma unroll
    for (int i = 0; i < 4; i += 2) {
        const uint32_t c = two_level_pair(odd ? am[4 + i] : am[i], odd ? am[5 + i] : am[i + 1], tw, e[i], e[i + 1], n[i], n[i + 1]);
        if (O::CODES && a.sf) {
            const int r = 8 * ty + (odd ? 4 : 0) + i;
            s16.row_sf[r][tx >> 1] = (uint8_t)(c & 0xFFu);
            s16.row_sf[r + 1][tx >> 1] = (uint8_t)(c >> 8);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float eo = __shfl_xor_sync(0xFFFFFFFFu, e[i], 1), no = __shfl_xor_sync(0xFFFFFFFFu, n[i], 1);
        sc.s_row[i] = odd ? eo : e[i];      sc.n_row[i] = odd ? no : n[i];
        sc.s_row[4 + i] = odd ? e[i] : eo;  sc.n_row[4 + i] = odd ? n[i] : no;
    }
    if (O::CODES && a.sf) {
        __syncwarp();
        const int r = 8 * ty + (tx & 7), half = tx >> 3;
        const uint32_t word = *reinterpret_cast<const uint32_t *>(&s16.row_sf[r][4 * half]);
        a.sf[(((int64_t)tl.r * tl.nc + tl.c) * 2 + half) * 128 + (r & 31) * 4 + (r >> 5)] = (rbase + (tx & 7) < a.rows) ? word : 0u;
    }
}

// 16x1 tiles of the two-level option: a warp holds 16 rows, so after the exchange with lane ^ 16 (done by the caller)
// cm holds the tile maxima of this lane's eight columns; the tile's index along the contraction is the warp's.
// The two lanes share the work: lanes 0..15 derive the factors of columns 0..3, lanes 16..31 those of columns 4..7, and
// they swap.  The scale bytes are staged for write_col16_atoms, which runs after the CTA barrier of the transposed output.
template <class O>
__device__ __forceinline__ void col16_scales(const QuantArgs &a, QuantShared16 &s16, const TwoLevel &tw, const uint32_t (&cm)[4], int lane, int tx,
                                             int warp, SubScales &sc)
{
    const bool upper = lane >= 16;
    float e[4], n[4];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const uint32_t m = (upper ? cm[2 + q] : cm[q]) & 0x7FFF7FFFu;
        const uint32_t c = two_level_pair(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u), tw, e[2 * q], e[2 * q + 1], n[2 * q], n[2 * q + 1]);
        if (O::CODES && a.sf) {
            const int col = 8 * tx + (upper ? 4 : 0) + 2 * q;
            s16.col_sf[col][warp] = (uint8_t)(c & 0xFFu);
            s16.col_sf[col + 1][warp] = (uint8_t)(c >> 8);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float eo = __shfl_xor_sync(0xFFFFFFFFu, e[i], 16), no = __shfl_xor_sync(0xFFFFFFFFu, n[i], 16);
        sc.s_col[i] = upper ? eo : e[i];      sc.n_col[i] = upper ? no : n[i];
        sc.s_col[4 + i] = upper ? e[i] : eo;  sc.n_col[4 + i] = upper ? n[i] : no;
    }
}
template <class O>
__device__ __forceinline__ void write_col16_atoms(const QuantArgs &a, const Tile &tl, const QuantShared16 &s16, int tid, int64_t c0)
{
    if (O::CODES && a.sf) {
        const int col = tid & (kTile - 1), half = tid >> 7;
        const uint32_t word = *reinterpret_cast<const uint32_t *>(&s16.col_sf[col][4 * half]);
        // atoms [column tile][row tile][half] (the operand is consumed transposed): one word per column and half
        a.sf[(((int64_t)tl.c * tl.nr + tl.r) * 2 + half) * 128 + (col & 31) * 4 + (col >> 5)] = (c0 + col < a.cols) ? word : 0u;
    }
}

template <class O>
__device__ __forceinline__ void blk_scales(const QuantArgs &a, const Tile &tl, float blk_am, int tid, SubScales &sc)
{
    sc.s_blk = tile_scale<O::FMT>(blk_am, a.pow2);
    sc.n_blk = neg_inv<O::FMT>(blk_am, sc.s_blk, a.pow2);
    if (O::CODES && a.sf && tid < kTile) {
        const int64_t atom = O::TRANSPOSED ? (int64_t)tl.c * tl.nr + tl.r : (int64_t)tl.r * tl.nc + tl.c;
        a.sf[atom * 128 + tid] = sf_word(sc.s_blk);
    }
    if (O::CODES && tid == 0) a.scales[(int64_t)tl.r * tl.nc + tl.c] = sc.s_blk;
}

// One tile, up to two outputs (A, B), everything from the thread's 8x8 sub-block in slot[p * kThreads].
// A and B: Out<...> or NoOut.  ROWSTATS (per-row sums) refers to output A.  after_reads() is called once
// the last read of the slot has been issued (the caller starts the next tile's fetch there).
template <class A, class B, bool STATS, bool ROWSTATS, class AfterReads>
__device__ __forceinline__ void process_tile(const QuantArgs &qa, const QuantArgs &qb, const Tile &tl, const uint4 *slot, QuantShared &sh,
                                             QuantShared32 *s32, ThreadStats &ts, AfterReads after_reads, const TwoLevel &tw = TwoLevel())
{
    QuantShared16 *s16 = reinterpret_cast<QuantShared16 *>(s32);   // the same place: a kernel uses one of the two
    static_assert(!(A::TRANSPOSED && B::TRANSPOSED), "one transposed output per pass");
    constexpr bool kRow = (A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x128) || (B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x128);
    constexpr bool kCol = (A::kQuant && A::BLOCK == SNIP_BLOCK_COL_128x1) || (B::kQuant && B::BLOCK == SNIP_BLOCK_COL_128x1);
    constexpr bool kRow32 = (A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x32) || (B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x32);
    constexpr bool kCol32 = (A::kQuant && A::BLOCK == SNIP_BLOCK_COL_32x1) || (B::kQuant && B::BLOCK == SNIP_BLOCK_COL_32x1);
    constexpr bool kRow16 = (A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x16) || (B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x16);
    constexpr bool kCol16 = (A::kQuant && A::BLOCK == SNIP_BLOCK_COL_16x1) || (B::kQuant && B::BLOCK == SNIP_BLOCK_COL_16x1);
    static_assert(!((kRow && kRow32) || (kCol && kCol32)), "one row-tiled and one column-tiled output per pass");
    static_assert(!(kRow16 && (kRow || kRow32)) && !(kCol16 && (kCol || kCol32)), "one row-tiled and one column-tiled output per pass");
    constexpr bool kBlk = (A::kQuant && A::BLOCK == SNIP_BLOCK_BLK_128x128) || (B::kQuant && B::BLOCK == SNIP_BLOCK_BLK_128x128);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t r0 = (int64_t)tl.r * kTile, c0 = (int64_t)tl.c * kTile;
    const int64_t rbase = r0 + 8 * ty, cbase = c0 + 8 * tx;
    const bool in_range = cbase < qa.cols && rbase < qa.rows;   // dims are multiples of 64: all 64 elements or none

    // ---- maxima (signs are garbage until masked: max.xorsign.abs keeps magnitudes only) -----------
    SubScales sa, sb;
    {
        uint32_t rmax[8], cm[4] = {0, 0, 0, 0};
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const uint4 vp = slot[p * kThreads];
            if (kRow || kRow32 || kRow16) rmax[p] = absmax2x(absmax2x(vp.x, vp.y), absmax2x(vp.z, vp.w));
            if (kCol || kCol32 || kCol16 || kBlk || !(kRow || kRow32 || kRow16)) {
                cm[0] = absmax2x(cm[0], vp.x);
                cm[1] = absmax2x(cm[1], vp.y);
                cm[2] = absmax2x(cm[2], vp.z);
                cm[3] = absmax2x(cm[3], vp.w);
            }
        }
        if (kRow16) {
            float am = 0.0f;
            if (A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x16) row16_scales<A>(qa, tl, *s16, tw, rmax, tx, ty, rbase, sa, am);
            if (B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x16) row16_scales<B>(qb, tl, *s16, tw, rmax, tx, ty, rbase, sb, am);
            if (STATS) ts.amax = fmaxf(ts.amax, am);
        }
        if (kCol16) {
#pragma unroll
            for (int q = 0; q < 4; ++q) cm[q] = absmax2x(cm[q], __shfl_xor_sync(0xFFFFFFFFu, cm[q], 16));
            if (A::kQuant && A::BLOCK == SNIP_BLOCK_COL_16x1) col16_scales<A>(qa, *s16, tw, cm, lane, tx, warp, sa);
            if (B::kQuant && B::BLOCK == SNIP_BLOCK_COL_16x1) col16_scales<B>(qb, *s16, tw, cm, lane, tx, warp, sb);
        }
        if (kRow || kRow32) {
            static_assert(!(A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x128 && B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x128), "one row-tiled output per pass");
            static_assert(!(A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x32 && B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x32), "one row-tiled output per pass");
            float am = 0.0f;
            if (A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x128) row_scales<A>(qa, tl, sh, rmax, tx, ty, rbase, sa, am);
            if (B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x128) row_scales<B>(qb, tl, sh, rmax, tx, ty, rbase, sb, am);
            if (A::kQuant && A::BLOCK == SNIP_BLOCK_ROW_1x32) row32_scales<A>(qa, tl, *s32, rmax, tx, ty, rbase, sa, am);
            if (B::kQuant && B::BLOCK == SNIP_BLOCK_ROW_1x32) row32_scales<B>(qb, tl, *s32, rmax, tx, ty, rbase, sb, am);
            if (STATS) ts.amax = fmaxf(ts.amax, am);
        }
        if (kCol || kCol32) {
            // the two row groups of a warp, then the 8 warps through shared memory
#pragma unroll
            for (int q = 0; q < 4; ++q) cm[q] = absmax2x(cm[q], __shfl_xor_sync(0xFFFFFFFFu, cm[q], 16));
            if (lane < 16) *reinterpret_cast<uint4 *>(&sh.col_amax[warp][4 * tx]) = make_uint4(cm[0], cm[1], cm[2], cm[3]);
            if (A::kQuant && A::BLOCK == SNIP_BLOCK_COL_128x1) col_scales<A>(qa, tl, sh, tid, tx, c0, sa);
            if (B::kQuant && B::BLOCK == SNIP_BLOCK_COL_128x1) col_scales<B>(qb, tl, sh, tid, tx, c0, sb);
            if (A::kQuant && A::BLOCK == SNIP_BLOCK_COL_32x1) col32_scales<A>(qa, tl, sh, *s32, tid, tx, ty, r0, c0, sa);
            if (B::kQuant && B::BLOCK == SNIP_BLOCK_COL_32x1) col32_scales<B>(qb, tl, sh, *s32, tid, tx, ty, r0, c0, sb);
        }
        if (kBlk || (!(kRow || kRow32 || kRow16) && STATS)) {
            uint32_t m = absmax2x(absmax2x(cm[0], cm[1]), absmax2x(cm[2], cm[3])) & 0x7FFF7FFFu;
            m = max(m & 0xFFFFu, m >> 16);
            if (!(kRow || kRow32 || kRow16) && STATS) ts.amax = fmaxf(ts.amax, __uint_as_float(m << 16));
            if (kBlk) {
                m = __reduce_max_sync(0xFFFFFFFFu, m);
                if (lane == 0) sh.red_m[warp] = m;
                __syncthreads();
                uint32_t bm = sh.red_m[0];
#pragma unroll
                for (int w = 1; w < 8; ++w) bm = max(bm, sh.red_m[w]);
                const float blk_am = __uint_as_float(bm << 16);
                if (A::kQuant && A::BLOCK == SNIP_BLOCK_BLK_128x128) blk_scales<A>(qa, tl, blk_am, tid, sa);
                if (B::kQuant && B::BLOCK == SNIP_BLOCK_BLK_128x128) blk_scales<B>(qb, tl, blk_am, tid, sb);
            }
        }
    }

    // ---- encode, statistics, as-stored codes ------------------------------------------------------
    uint32_t keep[8][2];   // codes of the transposed output, held until the sub-block is complete
    (void)keep;
    uint32_t ld_a = 0, ld_b = 0;
    uint8_t *dst_a = (A::kQuant && A::CODES && !A::TRANSPOSED) ? row_store_base<A::FMT>(qa, rbase, cbase, ld_a) : nullptr;
    uint8_t *dst_b = (B::kQuant && B::CODES && !B::TRANSPOSED) ? row_store_base<B::FMT>(qb, rbase, cbase, ld_b) : nullptr;
    (void)dst_a; (void)dst_b;
    float2 sx2 = make_float2(0.0f, 0.0f), sea2 = make_float2(0.0f, 0.0f), seb2 = make_float2(0.0f, 0.0f);
    float rsx[8], rse[8];
    (void)rsx; (void)rse;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        const uint4 vp = slot[p * kThreads];
        const uint32_t w[4] = {vp.x, vp.y, vp.z, vp.w};
        uint32_t ca[4], cb[4];
        uint32_t ua[4], ub[4];   // stochastic rounding: the eight 16-bit uniforms of this row segment
        (void)ua; (void)ub;
        if (A::SR || B::SR) {
            // element index r * cols + c, eight consecutive columns per generator call
            const uint64_t blk = ((uint64_t)(rbase + p) * (uint64_t)qa.cols + (uint64_t)cbase) >> 3;
            if (A::SR) philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)qa.seed, (uint32_t)(qa.seed >> 32), ua);
            if (B::SR) philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)qb.seed, (uint32_t)(qb.seed >> 32), ub);
        }
        float2 px = make_float2(0.0f, 0.0f), pe = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 x = make_float2(bf16lo(w[i]), bf16hi(w[i]));
            if (STATS) { if (ROWSTATS) px = __ffma2_rn(x, x, px); else sx2 = __ffma2_rn(x, x, sx2); }
            if (A::kQuant) {
                if (A::SR) ca[i] = encode_pair_sr_fp4<STATS>(x, scale_pair<A>(sa, p, i), ninv_pair<A>(sa, p, i), ua[i], ROWSTATS ? pe : sea2);
                else ca[i] = encode_pair<A::FMT, STATS>(x, scale_pair<A>(sa, p, i), ninv_pair<A>(sa, p, i), ROWSTATS ? pe : sea2);
            }
            if (B::kQuant) {
                if (B::SR) cb[i] = encode_pair_sr_fp4<STATS>(x, scale_pair<B>(sb, p, i), ninv_pair<B>(sb, p, i), ub[i], seb2);
                else cb[i] = encode_pair<B::FMT, STATS>(x, scale_pair<B>(sb, p, i), ninv_pair<B>(sb, p, i), seb2);
            }
        }
        if (ROWSTATS) {
            rsx[p] = px.x + px.y; rse[p] = pe.x + pe.y;
            sx2.x += rsx[p]; sea2.x += rse[p];
        }
        if (A::kQuant && A::CODES) {
            uint32_t code[2];
            pack8<A::FMT>(ca, code);
            if (A::TRANSPOSED) { keep[p][0] = code[0]; keep[p][1] = code[1]; }
            else if (in_range) store_row<A::FMT>(dst_a + p * ld_a, code);
        }
        if (B::kQuant && B::CODES) {
            uint32_t code[2];
            pack8<B::FMT>(cb, code);
            if (B::TRANSPOSED) { keep[p][0] = code[0]; keep[p][1] = code[1]; }
            else if (in_range) store_row<B::FMT>(dst_b + p * ld_b, code);
        }
    }
    after_reads();

    if (STATS) {
        ts.x += (double)(sx2.x + sx2.y);
        if (A::kQuant) ts.ea += (double)(sea2.x + sea2.y);
        if (B::kQuant) ts.eb += (double)(seb2.x + seb2.y);
    }
    if (ROWSTATS) {
        // per row: add the 16 lanes that share the row, lane tx == 0 writes {sum x^2, sum err^2}
#pragma unroll
        for (int p = 0; p < 8; ++p) {
#pragma unroll
            for (int off = 1; off < 16; off <<= 1) {
                rsx[p] += __shfl_xor_sync(0xFFFFFFFFu, rsx[p], off);
                rse[p] += __shfl_xor_sync(0xFFFFFFFFu, rse[p], off);
            }
        }
        if (tx == 0 && rbase < qa.rows) {
            float2 *dst = qa.row_partials + (int64_t)tl.c * qa.rows + rbase;
#pragma unroll
            for (int p = 0; p < 8; ++p) dst[p] = make_float2(rsx[p], rse[p]);
        }
    }

    // ---- transposed codes: registers -> swizzled shared tile -> coalesced 16-byte stores ------------
    if (A::kQuant && A::CODES && A::TRANSPOSED) {
        stage_transposed<A::FMT>(sh.stage, tx, ty, keep);
        __syncthreads();
        write_transposed<A::FMT>(qa, sh.stage, r0, c0);
    }
    if (B::kQuant && B::CODES && B::TRANSPOSED) {
        stage_transposed<B::FMT>(sh.stage, tx, ty, keep);
        __syncthreads();
        write_transposed<B::FMT>(qb, sh.stage, r0, c0);
        if (B::BLOCK == SNIP_BLOCK_COL_16x1) write_col16_atoms<B>(qb, tl, *s16, tid, c0);
    }
}

// End of a CTA's walk: its threads' sums -> one CtaPartial per output (warp shuffles, then warp order).
template <bool HAS_B>
__device__ __forceinline__ void finish_stats(const ThreadStats &ts, QuantShared &sh, CtaPartial *pa, CtaPartial *pb)
{
    double x = ts.x, ea = ts.ea, eb = ts.eb;
    float am = ts.amax;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        x += __shfl_xor_sync(0xFFFFFFFFu, x, off);
        ea += __shfl_xor_sync(0xFFFFFFFFu, ea, off);
        if (HAS_B) eb += __shfl_xor_sync(0xFFFFFFFFu, eb, off);
        am = fmaxf(am, __shfl_xor_sync(0xFFFFFFFFu, am, off));
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();   // the scratch of the last tile is no longer in use
    if (lane == 0) { sh.red_d[warp][0] = x; sh.red_d[warp][1] = ea; sh.red_d[warp][2] = eb; sh.red_d[warp][3] = (double)am; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double tx_ = 0.0, ta = 0.0, tb = 0.0, tm = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) { tx_ += sh.red_d[w][0]; ta += sh.red_d[w][1]; tb += sh.red_d[w][2]; tm = fmax(tm, sh.red_d[w][3]); }
        CtaPartial *d = pa + blockIdx.x;
        d->sumsq_x = tx_; d->sumsq_err = ta; d->amax = (float)tm;
        if (HAS_B) {
            d = pb + blockIdx.x;
            d->sumsq_x = tx_; d->sumsq_err = tb; d->amax = (float)tm;
        }
    }
}

// Dynamic shared memory of the kernels: the tile slot, then the QuantShared scratch.
constexpr size_t kSmemBytes = (size_t)kStageBytes + sizeof(QuantShared);
#ifndef SNIP_DUAL_CTAS
#define SNIP_DUAL_CTAS 3
#endif
constexpr int kCtasPerSm = 4;
constexpr int kDualCtasPerSm = SNIP_DUAL_CTAS;

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

template <int FMT, int BLOCK, bool TRANSPOSED, bool CODES, bool STATS, bool ROWSTATS, bool SR = false>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) quantize_kernel(const QuantArgs a)
{
    extern __shared__ __align__(128) uint8_t smem[];
    QuantShared &sh = *reinterpret_cast<QuantShared *>(smem + kStageBytes);
    QuantShared32 *s32 = reinterpret_cast<QuantShared32 *>(smem + kSmemBytes);   // present only for the 32-long tile kinds
    const uint4 *slot = reinterpret_cast<const uint4 *>(smem) + threadIdx.x;
    // this grid may have been scheduled before the kernel ahead of it on the stream has finished (see
    // launch_persistent): nothing is read or written before that kernel is complete
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the statistics reduction that follows on the stream may be scheduled now; it waits for this
    // grid to finish before it reads anything (programmatic dependent launch)
    if (STATS) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    ThreadStats ts;
    TileWalk w((int)a.tiles_r, (int)a.tiles_c);
    if (w.valid()) prefetch_tile(a, w.r, w.c, smem);
    prefetch_commit();
    while (w.valid()) {
        prefetch_wait<0>();
        const Tile tl = {w.r, w.c, w.nr, w.nc};
        w.next();
        process_tile<Out<FMT, BLOCK, TRANSPOSED, CODES, SR>, NoOut, STATS, ROWSTATS>(a, a, tl, slot, sh, s32, ts, [&] {
            if (w.valid()) prefetch_tile(a, w.r, w.c, smem);   // this thread's reads of its slot are done
            prefetch_commit();
        });
        __syncthreads();  // the scratch arrays are reused by the next tile
    }
    if (STATS) finish_stats<false>(ts, sh, a.partials, nullptr);
}

// Two outputs from one read (the tile kinds a tensor is consumed with, paper Fig. 5): `a` as stored
// (1x128 tiles along the columns, or 128x128 blocks) and `b` transposed (128x1 tiles along the rows, or
// the same 128x128 blocks), each with its own format, scales and statistics.
struct DualArgs {
    QuantArgs a, b;
};
template <int FMT_A, int FMT_B, bool BLK, bool STATS, bool SR_A = false, bool SR_B = false, bool SUB32 = false>
__global__ void __launch_bounds__(kThreads, kDualCtasPerSm) quantize_dual_kernel(const DualArgs d)
{
    extern __shared__ __align__(128) uint8_t smem[];
    QuantShared &sh = *reinterpret_cast<QuantShared *>(smem + kStageBytes);
    QuantShared32 *s32 = reinterpret_cast<QuantShared32 *>(smem + kSmemBytes);   // present only with SUB32
    const uint4 *slot = reinterpret_cast<const uint4 *>(smem) + threadIdx.x;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (STATS) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    ThreadStats ts;
    TileWalk w((int)d.a.tiles_r, (int)d.a.tiles_c);
    if (w.valid()) prefetch_tile(d.a, w.r, w.c, smem);
    prefetch_commit();
    while (w.valid()) {
        prefetch_wait<0>();
        const Tile tl = {w.r, w.c, w.nr, w.nc};
        w.next();
        using A = Out<FMT_A, SUB32 ? SNIP_BLOCK_ROW_1x32 : BLK ? SNIP_BLOCK_BLK_128x128 : SNIP_BLOCK_ROW_1x128, false, true, SR_A>;
        using B = Out<FMT_B, SUB32 ? SNIP_BLOCK_COL_32x1 : BLK ? SNIP_BLOCK_BLK_128x128 : SNIP_BLOCK_COL_128x1, true, true, SR_B>;
        process_tile<A, B, STATS, false>(d.a, d.b, tl, slot, sh, s32, ts, [&] {
            if (w.valid()) prefetch_tile(d.a, w.r, w.c, smem);
            prefetch_commit();
        });
        __syncthreads();
    }
    if (STATS) finish_stats<true>(ts, sh, d.a.partials, d.b.partials);
}

// Two-level option, both copies from one read: a = 1x16 tiles as stored, b = 16x1 tiles transposed, E2M1 codes.
template <bool STATS, bool SR = false>
__global__ void __launch_bounds__(kThreads, kDualCtasPerSm) quantize_nvfp4_dual_kernel(const DualArgs d)
{
    extern __shared__ __align__(128) uint8_t smem[];
    QuantShared &sh = *reinterpret_cast<QuantShared *>(smem + kStageBytes);
    QuantShared32 *s32 = reinterpret_cast<QuantShared32 *>(smem + kSmemBytes);   // holds this kernel's QuantShared16
    const uint4 *slot = reinterpret_cast<const uint4 *>(smem) + threadIdx.x;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (STATS) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    TwoLevel tw;
    {
        const float bound = *d.a.tensor_amax;
        tw.enc = bound == 0.0f ? 1.0f : fminf(__fdiv_rn(2688.0f, bound), FLT_MAX);
        tw.inv_enc = __fdiv_rn(1.0f, tw.enc);
    }
    ThreadStats ts;
    TileWalk w((int)d.a.tiles_r, (int)d.a.tiles_c);
    if (w.valid()) prefetch_tile(d.a, w.r, w.c, smem);
    prefetch_commit();
    while (w.valid()) {
        prefetch_wait<0>();
        const Tile tl = {w.r, w.c, w.nr, w.nc};
        w.next();
        using A = Out<SNIP_FMT_FP4_E2M1, SNIP_BLOCK_ROW_1x16, false, true, SR>;
        using B = Out<SNIP_FMT_FP4_E2M1, SNIP_BLOCK_COL_16x1, true, true, SR>;
        process_tile<A, B, STATS, false>(d.a, d.b, tl, slot, sh, s32, ts, [&] {
            if (w.valid()) prefetch_tile(d.a, w.r, w.c, smem);
            prefetch_commit();
        }, tw);
        __syncthreads();
    }
    if (STATS) finish_stats<true>(ts, sh, d.a.partials, d.b.partials);
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
    // a quantizer launched behind this reduction may take the SMs the previous quantizer is leaving; it waits
    // for this grid before it reads or writes anything
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
void launch_persistent(Kernel kernel, const Args &args, dim3 grid, cudaStream_t st, size_t smem_bytes = kSmemBytes)
{
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess) return;  // left in cudaGetLastError
    // Programmatic stream serialization: when the kernel before it on the stream signals its dependents early (the
    // statistics reduction of the previous call does), this grid's CTAs may take their places while that kernel
    // drains; they block in griddepcontrol.wait until it has completed, before they touch global memory.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, args);   // an error stays in cudaGetLastError for the caller
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

constexpr size_t kSmemBytes32 = kSmemBytes + sizeof(QuantShared32);
constexpr int kCtasPerSm32 = 3;   // what the larger shared-memory footprint allows

// 32-long tile kinds: 1x32 tiles as stored, 32x1 tiles transposed.
template <int FMT>
void launch_fmt32(const QuantArgs &a, int block, bool codes, bool stats, dim3 grid, cudaStream_t st)
{
    if (block == SNIP_BLOCK_ROW_1x32) {
        if (codes && stats) launch_persistent(quantize_kernel<FMT, SNIP_BLOCK_ROW_1x32, false, true, true, false>, a, grid, st, kSmemBytes32);
        else if (codes) launch_persistent(quantize_kernel<FMT, SNIP_BLOCK_ROW_1x32, false, true, false, false>, a, grid, st, kSmemBytes32);
        else launch_persistent(quantize_kernel<FMT, SNIP_BLOCK_ROW_1x32, false, false, true, false>, a, grid, st, kSmemBytes32);
    } else {
        if (codes && stats) launch_persistent(quantize_kernel<FMT, SNIP_BLOCK_COL_32x1, true, true, true, false>, a, grid, st, kSmemBytes32);
        else if (codes) launch_persistent(quantize_kernel<FMT, SNIP_BLOCK_COL_32x1, true, true, false, false>, a, grid, st, kSmemBytes32);
        else launch_persistent(quantize_kernel<FMT, SNIP_BLOCK_COL_32x1, false, false, true, false>, a, grid, st, kSmemBytes32);
    }
}

// CTAs of a persistent launch over ntiles tiles: kCtasPerSm per SM (what the kernels' shared memory and
// registers allow), never more than there are tiles.
int64_t persistent_ctas(int64_t ntiles, int per_sm = kCtasPerSm)
{
    const int64_t cap = per_sm * (int64_t)gemm_sm_count();
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

int quantize_impl_full(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, int pow2, void *sf, int sr,
                       uint64_t seed, void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes,
                       cudaStream_t st);

// pow2 = 1 selects the power-of-two scale rule; sf (optional, needs pow2) receives the UE8M0 atoms.
int quantize_impl_ex(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, int pow2, void *sf,
                     void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes, cudaStream_t st)
{
    return quantize_impl_full(x, rows, cols, ld, fmt, block, flags, pow2, sf, 0, 0, codes, scales, stats, row_stats, ws, ws_bytes, st);
}

// sr = 1: stochastic rounding with `seed` (FP4 codes, 1x128 tiles as stored or 128x1 tiles transposed, no per-row sums).
int quantize_impl_full(const void *x, int64_t rows, int64_t cols, int64_t ld, int fmt, int block, uint32_t flags, int pow2, void *sf, int sr,
                       uint64_t seed, void *codes, float *scales, snip_stats_t *stats, double *row_stats, void *ws, size_t ws_bytes,
                       cudaStream_t st)
{
    if (sf) {
        const bool tr = (flags & SNIP_Q_TRANSPOSED) != 0;
        // atoms follow the orientation the GEMM consumes: row tiles as stored, column tiles transposed
        if (!pow2 || !aligned16(sf) || (block == SNIP_BLOCK_ROW_1x128 && tr) || (block == SNIP_BLOCK_COL_128x1 && !tr)) return SNIP_ERR_UNSUPPORTED;
    }
    const bool b32 = block == SNIP_BLOCK_ROW_1x32 || block == SNIP_BLOCK_COL_32x1;
    if (b32) {
        // 32-long tiles: power-of-two scales of a quantized format, 1x32 as stored or 32x1 transposed, no per-row sums, RNE
        const bool tr = (flags & SNIP_Q_TRANSPOSED) != 0;
        if (!pow2 || sr || row_stats || fmt == SNIP_FMT_BF16 || (block == SNIP_BLOCK_ROW_1x32) == tr) return SNIP_ERR_UNSUPPORTED;
    }
    if (!x || !valid_fmt(fmt) || !(valid_block(block) || b32)) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols) || ld < cols || (ld % 8) != 0 || rows > INT32_MAX || ld > INT32_MAX) return SNIP_ERR_SHAPE;
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
    a.rows = (int32_t)rows; a.cols = (int32_t)cols; a.ld = (int32_t)ld;
    a.pow2 = pow2; a.sf = static_cast<uint32_t *>(sf);
    a.seed = seed;
    a.codes = want_codes ? static_cast<uint8_t *>(codes) : nullptr;
    a.scales = want_codes ? scales : nullptr;
    a.partials = any_stats ? static_cast<CtaPartial *>(ws) : nullptr;
    a.row_partials = want_rows ? reinterpret_cast<float2 *>(static_cast<uint8_t *>(ws) + align_up((size_t)(tr * tc) * sizeof(CtaPartial), 256)) : nullptr;
    a.tiles_r = (int32_t)tr; a.tiles_c = (int32_t)tc; a.ntiles = tr * tc;
    const int64_t nparts = persistent_ctas(tr * tc, b32 ? kCtasPerSm32 : kCtasPerSm);
    dim3 grid((unsigned)nparts);
    if (b32) {
        if (fmt == SNIP_FMT_FP8_E4M3) launch_fmt32<SNIP_FMT_FP8_E4M3>(a, block, want_codes, any_stats, grid, st);
        else launch_fmt32<SNIP_FMT_FP4_E2M1>(a, block, want_codes, any_stats, grid, st);
    } else
    if (sr) {
        const bool row = block == SNIP_BLOCK_ROW_1x128 && !transposed, colt = block == SNIP_BLOCK_COL_128x1 && transposed;
        if (fmt != SNIP_FMT_FP4_E2M1 || !want_codes || want_rows || !(row || colt)) return SNIP_ERR_UNSUPPORTED;
        constexpr int F4 = SNIP_FMT_FP4_E2M1;
        if (row && any_stats) launch_persistent(quantize_kernel<F4, SNIP_BLOCK_ROW_1x128, false, true, true, false, true>, a, grid, st);
        else if (row) launch_persistent(quantize_kernel<F4, SNIP_BLOCK_ROW_1x128, false, true, false, false, true>, a, grid, st);
        else if (any_stats) launch_persistent(quantize_kernel<F4, SNIP_BLOCK_COL_128x1, true, true, true, false, true>, a, grid, st);
        else launch_persistent(quantize_kernel<F4, SNIP_BLOCK_COL_128x1, true, true, false, false, true>, a, grid, st);
    } else
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
// Two-output launch with stochastic rounding on the FP4 outputs that ask for it (row/column kinds only).
template <int FMT_A, int FMT_B, bool SR_A, bool SR_B>
static void launch_dual_sr(const DualArgs &d, bool stats, dim3 grid, cudaStream_t st)
{
    if (stats) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, true, SR_A, SR_B>, d, grid, st);
    else launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, false, SR_A, SR_B>, d, grid, st);
}

template <int FMT_A, int FMT_B>
static void launch_dual(const DualArgs &d, bool blk, bool stats, dim3 grid, cudaStream_t st)
{
    if (blk && stats) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, true, true>, d, grid, st);
    else if (blk) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, true, false>, d, grid, st);
    else if (stats) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, true>, d, grid, st);
    else launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, false>, d, grid, st);
}

template <int FMT_A, int FMT_B, bool SR_A = false, bool SR_B = false>
static void launch_dual32(const DualArgs &d, bool stats, dim3 grid, cudaStream_t st)
{
    if (stats) launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, true, SR_A, SR_B, true>, d, grid, st, kSmemBytes32);
    else launch_persistent(quantize_dual_kernel<FMT_A, FMT_B, false, false, SR_A, SR_B, true>, d, grid, st, kSmemBytes32);
}

// kind: SNIP_DUAL_ROW_COLT, SNIP_DUAL_BLK_BLKT or SNIP_DUAL_ROW32_COL32T (power-of-two scales only).
int quantize_dual_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, int kind, int pow2, const DualOut &oa, const DualOut &ob,
                       void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (!x) return SNIP_ERR_ARG;
    const bool blk = kind == SNIP_DUAL_BLK_BLKT, sub32 = kind == SNIP_DUAL_ROW32_COL32T;
    if (sub32 && !pow2) return SNIP_ERR_UNSUPPORTED;
    if (!valid_dim(rows) || !valid_dim(cols) || ld < cols || (ld % 8) != 0 || rows > INT32_MAX || ld > INT32_MAX) return SNIP_ERR_SHAPE;
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
        q.rows = (int32_t)rows; q.cols = (int32_t)cols; q.ld = (int32_t)ld;
        q.codes = static_cast<uint8_t *>(o[i]->codes);
        q.scales = o[i]->scales;
        q.partials = stats ? reinterpret_cast<CtaPartial *>(static_cast<uint8_t *>(ws) + i * one) : nullptr;
        q.row_partials = nullptr;
        q.pow2 = pow2;
        q.seed = o[i]->seed;
        q.sf = static_cast<uint32_t *>(o[i]->sf);
        q.tiles_r = (int32_t)tr; q.tiles_c = (int32_t)tc; q.ntiles = tr * tc;
    }
    const int64_t nparts = persistent_ctas(tr * tc, kDualCtasPerSm);
    dim3 grid((unsigned)nparts);
    const bool a8 = oa.fmt == SNIP_FMT_FP8_E4M3, b8 = ob.fmt == SNIP_FMT_FP8_E4M3;
    constexpr int F8 = SNIP_FMT_FP8_E4M3, F4 = SNIP_FMT_FP4_E2M1;
    if (sub32 && (oa.sr || ob.sr)) {
        if ((oa.sr && a8) || (ob.sr && b8)) return SNIP_ERR_UNSUPPORTED;   // stochastic rounding is offered for FP4 codes
        if (oa.sr && ob.sr) launch_dual32<F4, F4, true, true>(d, stats, grid, st);
        else if (oa.sr && b8) launch_dual32<F4, F8, true, false>(d, stats, grid, st);
        else if (oa.sr) launch_dual32<F4, F4, true, false>(d, stats, grid, st);
        else if (a8) launch_dual32<F8, F4, false, true>(d, stats, grid, st);
        else launch_dual32<F4, F4, false, true>(d, stats, grid, st);
    } else if (sub32) {
        if (a8 && b8) launch_dual32<F8, F8>(d, stats, grid, st);
        else if (a8) launch_dual32<F8, F4>(d, stats, grid, st);
        else if (b8) launch_dual32<F4, F8>(d, stats, grid, st);
        else launch_dual32<F4, F4>(d, stats, grid, st);
    } else
    if (oa.sr || ob.sr) {
        if (blk || (oa.sr && a8) || (ob.sr && b8)) return SNIP_ERR_UNSUPPORTED;   // FP4 row / column tiles only
        if (oa.sr && ob.sr) launch_dual_sr<F4, F4, true, true>(d, stats, grid, st);
        else if (oa.sr && b8) launch_dual_sr<F4, F8, true, false>(d, stats, grid, st);
        else if (oa.sr) launch_dual_sr<F4, F4, true, false>(d, stats, grid, st);
        else if (a8) launch_dual_sr<F8, F4, false, true>(d, stats, grid, st);
        else launch_dual_sr<F4, F4, false, true>(d, stats, grid, st);
    } else
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

// Two-level option (see include/snip.h): both copies of a tensor from one read.
int quantize_nvfp4_dual_impl(const void *x, int64_t rows, int64_t cols, int64_t ld, const float *tensor_amax, void *codes_a, void *sf_a,
                             snip_stats_t *stats_a, void *codes_b, void *sf_b, snip_stats_t *stats_b, int rounding, uint64_t seed, void *ws,
                             size_t ws_bytes, cudaStream_t st)
{
    if (rounding != SNIP_ROUND_NEAREST_EVEN && rounding != SNIP_ROUND_STOCHASTIC) return SNIP_ERR_ARG;
    const bool sr = rounding == SNIP_ROUND_STOCHASTIC;
    if (!x || !tensor_amax || !codes_a || !sf_a || !codes_b || !sf_b) return SNIP_ERR_ARG;
    if (!valid_dim(rows) || !valid_dim(cols) || ld < cols || (ld % 8) != 0 || rows > INT32_MAX || ld > INT32_MAX) return SNIP_ERR_SHAPE;
    if ((stats_a == nullptr) != (stats_b == nullptr)) return SNIP_ERR_ARG;
    if (!aligned16(x) || !aligned16(codes_a) || !aligned16(sf_a) || !aligned16(codes_b) || !aligned16(sf_b) ||
        (reinterpret_cast<uintptr_t>(tensor_amax) & 3u) || (stats_a && ((reinterpret_cast<uintptr_t>(stats_a) | reinterpret_cast<uintptr_t>(stats_b)) & 7u)))
        return SNIP_ERR_ALIGN;
    const bool stats = stats_a != nullptr;
    const size_t one = stats_ws_bytes(rows, cols, false);
    if (stats && (!ws || ws_bytes < 2 * one)) return SNIP_ERR_WORKSPACE;
    if (stats && !aligned16(ws)) return SNIP_ERR_ALIGN;
    int rc = require_sm100();
    if (rc != SNIP_OK) return rc;
    const int64_t tr = ceil_div(rows, kTile), tc = ceil_div(cols, kTile);
    DualArgs d;
    void *codes[2] = {codes_a, codes_b}, *sf[2] = {sf_a, sf_b};
    for (int i = 0; i < 2; ++i) {
        QuantArgs &q = i ? d.b : d.a;
        q.x = static_cast<const uint16_t *>(x);
        q.rows = (int32_t)rows; q.cols = (int32_t)cols; q.ld = (int32_t)ld;
        q.codes = static_cast<uint8_t *>(codes[i]);
        q.scales = nullptr;
        q.partials = stats ? reinterpret_cast<CtaPartial *>(static_cast<uint8_t *>(ws) + i * one) : nullptr;
        q.row_partials = nullptr;
        q.pow2 = 0;
        q.seed = seed;
        q.sf = static_cast<uint32_t *>(sf[i]);
        q.tensor_amax = tensor_amax;
        q.tiles_r = (int32_t)tr; q.tiles_c = (int32_t)tc; q.ntiles = tr * tc;
    }
    const int64_t nparts = persistent_ctas(tr * tc, kDualCtasPerSm);
    dim3 grid((unsigned)nparts);
    if (stats && sr) launch_persistent(quantize_nvfp4_dual_kernel<true, true>, d, grid, st, kSmemBytes32);
    else if (stats) launch_persistent(quantize_nvfp4_dual_kernel<true, false>, d, grid, st, kSmemBytes32);
    else if (sr) launch_persistent(quantize_nvfp4_dual_kernel<false, true>, d, grid, st, kSmemBytes32);
    else launch_persistent(quantize_nvfp4_dual_kernel<false, false>, d, grid, st, kSmemBytes32);
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
        const ReduceSets sets = {{d.a.partials, d.b.partials}, {stats_a, stats_b}};
        SNIP_CUDA_TRY(cudaLaunchKernelEx(&cfg, stats_reduce_kernel, sets, nparts));
    }
    return SNIP_OK;
}

}  // namespace snip

extern "C" int snip_quantize_nvfp4_sizes(int64_t rows, int64_t cols, size_t *codes_bytes, size_t *sf_bytes)
{
    using namespace snip;
    if (!valid_dim(rows) || !valid_dim(cols)) return SNIP_ERR_SHAPE;
    // 64 bytes of tail slack after the codes of a ragged shape, as in snip_quantize_sizes
    if (codes_bytes) *codes_bytes = (size_t)(rows * cols) / 2 + (((rows % 128) || (cols % 128)) ? 64 : 0);
    if (sf_bytes) *sf_bytes = (size_t)(ceil_div(rows, 128) * ceil_div(cols, 128)) * 1024;
    return SNIP_OK;
}

extern "C" int snip_quantize_nvfp4_dual(const void *x, int64_t rows, int64_t cols, int64_t ld, const float *tensor_amax, void *codes_stored,
                                        void *sf_stored, snip_stats_t *stats_stored, void *codes_transposed, void *sf_transposed,
                                        snip_stats_t *stats_transposed, int rounding, uint64_t seed, void *ws, size_t ws_bytes, void *stream)
{
    return snip::quantize_nvfp4_dual_impl(x, rows, cols, ld, tensor_amax, codes_stored, sf_stored, stats_stored, codes_transposed, sf_transposed,
                                          stats_transposed, rounding, seed, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

extern "C" int snip_quantize_sizes(int64_t rows, int64_t cols, int fmt, int block, uint32_t flags,
                                   size_t *codes_bytes, size_t *scales_bytes, size_t *ws_bytes)
{
    using namespace snip;
    const bool b32 = block == SNIP_BLOCK_ROW_1x32 || block == SNIP_BLOCK_COL_32x1;
    if (!valid_fmt(fmt) || !(valid_block(block) || b32)) return SNIP_ERR_ARG;
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
        if (block == SNIP_BLOCK_ROW_1x32) n = ceil_div(cols, 32) * rows;
        if (block == SNIP_BLOCK_COL_32x1) n = ceil_div(rows, 32) * cols;
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
    // only the statistics use scratch: a call without SNIP_Q_STATS never touches the built-in array
    const size_t need = (flags & SNIP_Q_STATS) ? stats_ws_bytes(rows, cols, false) : 0;
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
    if (kind != SNIP_DUAL_ROW_COLT && kind != SNIP_DUAL_BLK_BLKT && kind != SNIP_DUAL_ROW32_COL32T) return SNIP_ERR_ARG;
    if ((as_stored->rounding & ~1) || (transposed->rounding & ~1)) return SNIP_ERR_ARG;
    const DualOut oa = {as_stored->fmt, as_stored->codes, as_stored->scales, as_stored->sf, as_stored->stats, as_stored->rounding, as_stored->seed};
    const DualOut ob = {transposed->fmt, transposed->codes, transposed->scales, transposed->sf, transposed->stats, transposed->rounding, transposed->seed};
    return quantize_dual_impl(x, rows, cols, ld, kind, pow2_scale ? 1 : 0, oa, ob, ws, ws_bytes,
                              static_cast<cudaStream_t>(stream));
}

// ---- stochastic rounding (paper Sec. 6.1) ------------------------------------------------------

extern "C" int snip_quantize_sr(const void *x, int64_t rows, int64_t cols, int64_t ld, int block, uint32_t flags, uint64_t seed, int pow2_scale,
                                void *codes, float *scales, void *sf, snip_stats_t *stats, void *ws, size_t ws_bytes, void *stream)
{
    using namespace snip;
    return quantize_impl_full(x, rows, cols, ld, SNIP_FMT_FP4_E2M1, block, flags, pow2_scale ? 1 : 0, sf, 1, seed, codes, scales, stats, nullptr, ws,
                              ws_bytes, static_cast<cudaStream_t>(stream));
}
