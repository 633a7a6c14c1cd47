// Deliberately naive FP64 matrix products on the GPU, used ONLY by the tests as a bridge between the CPU oracle
// and full-matrix comparisons at sizes where the oracle's triple loop would take hours.  One thread per output
// element, one plain loop over the contraction, double-precision FMAs, no tensor cores, no shared memory, and no
// code in common with the library.  Its inputs are the oracle's dequantized operands (float64); it is itself
// compared with the oracle's GEMMs in full on small cases before anything is compared with it.
//
//   op 0 (forward)          C[M,N] = A[M,K] . B[N,K]^T
//   op 1 (input gradient)   C[M,K] = A[M,N] . B[N,K]
//   op 2 (weight gradient)  C[N,K] = A[M,N]^T . B[M,K]
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

// C[i,j] = sum_l A(i,l) * B(l,j) with element strides given, so that one kernel serves the three orientations.
__global__ void naive_matmul_f64(const double *__restrict__ a, const double *__restrict__ b, double *__restrict__ c, int64_t rows, int64_t cols,
                                 int64_t len, int64_t a_row, int64_t a_l, int64_t b_l, int64_t b_col)
{
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = (int64_t)blockIdx.y * blockDim.y + threadIdx.y;
    if (i >= rows || j >= cols) return;
    double acc = 0.0;
    for (int64_t l = 0; l < len; ++l) acc = fma(a[i * a_row + l * a_l], b[l * b_l + j * b_col], acc);
    c[i * cols + j] = acc;
}

}  // namespace

// All pointers are device pointers to float64.  Returns a cudaError_t as int (0 = success).  Synchronous.
extern "C" int naive_gemm_f64(int op, const double *a, const double *b, double *c, int64_t M, int64_t N, int64_t K)
{
    int64_t rows, cols, len, a_row, a_l, b_l, b_col;
    if (op == 0) { rows = M; cols = N; len = K; a_row = K; a_l = 1; b_l = 1; b_col = K; }          // B[N,K]: (l, j) -> j*K + l
    else if (op == 1) { rows = M; cols = K; len = N; a_row = N; a_l = 1; b_l = K; b_col = 1; }     // B[N,K]: (l, j) -> l*K + j
    else if (op == 2) { rows = N; cols = K; len = M; a_row = 1; a_l = N; b_l = K; b_col = 1; }     // A[M,N]: (i, l) -> l*N + i
    else return (int)cudaErrorInvalidValue;
    dim3 block(32, 8), grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 7) / 8));
    naive_matmul_f64<<<grid, block>>>(a, b, c, rows, cols, len, a_row, a_l, b_l, b_col);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    return (int)cudaDeviceSynchronize();
}
