// Shared host-side helpers of the SNIP library: status handling and argument checks.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "snip.h"

namespace snip {

// Thread-local text of the last CUDA error observed inside the library.
char *last_error_buffer();
void set_last_error(const char *where, cudaError_t e);

#define SNIP_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t _e = (expr);                              \
        if (_e != cudaSuccess) {                              \
            ::snip::set_last_error(#expr, _e);                \
            return SNIP_ERR_CUDA;                             \
        }                                                     \
    } while (0)

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline bool valid_fmt(int f) { return f >= SNIP_FMT_BF16 && f <= SNIP_FMT_FP4_E2M1; }
static inline bool valid_block(int b) { return b >= SNIP_BLOCK_ROW_1x128 && b <= SNIP_BLOCK_BLK_128x128; }
static inline bool valid_dim(int64_t d) { return d > 0 && (d % 64) == 0; }

// One output of the two-output quantizer (quantize.cu: quantize_dual_impl).
struct DualOut {
    int fmt;
    void *codes;
    float *scales;
    void *sf;             // optional UE8M0 atoms (power-of-two rule only)
    snip_stats_t *stats;  // optional; both outputs or neither
    int sr = 0;           // 1: stochastic rounding (FP4 only)
    uint64_t seed = 0;
};

// Fails with SNIP_ERR_UNSUPPORTED unless the current device is compute capability 10.x.
int require_sm100();

}  // namespace snip
