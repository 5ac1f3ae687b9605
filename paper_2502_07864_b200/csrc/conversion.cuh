// GQA -> MLA conversion on calibration activations (Sec. 4.2, 4.3; App. B, C, D): launchers.
// Everything here is fp32 on the device (the orthonormalisation inside the subspace iteration runs in fp64):
// the conversion is a one-off whose results are eigenvectors, which bf16 would not resolve.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "transmla.h"

namespace transmla {
namespace conv {

// C[M,N] = alpha * op(A) op(B); op(A) is A [M,K] (ta = 0, row stride lda) or the transpose of A [K,M] (ta = 1), likewise
// op(B) from B [K,N] or B [N,K].  `batch` problems, strides in elements.  TOut = float or double (fp64 accumulation).
cudaError_t gemm_f32(int ta, int tb, int M, int N, int K, float alpha, const float* A, int lda, long long strideA,
                     const float* B, int ldb, long long strideB, float* C, int ldc, long long strideC, int batch,
                     cudaStream_t stream);
// seg[G][2n][g*fold]: rows 0..n-1 the real parts, n..2n-1 the imaginary parts of group G's dimensions (App. B, C)
cudaError_t gather_segments(const float* K, int n, int g, int d, int fold, float* seg, cudaStream_t stream);
// Symmetric eigendecomposition of `batch` matrices of order m <= 128 (parallel cyclic Jacobi, one block each).
cudaError_t sym_eig(float* a, int batch, int m, float* eigvals, float* eigvecs, int32_t* dev_status, cudaStream_t stream);
cudaError_t rorope_apply(const float* X, int C, const float* U, int g, int d, int fold, float* Y, cudaStream_t stream);
cudaError_t row_norm_ratio(const float* k_nope, int n, int mk, const float* v, int mv, float* scratch, float* alpha_out,
                           cudaStream_t stream);
cudaError_t balance_concat(const float* k_nope, int n, int mk, const float* v, int mv, const float* alpha, float* Z,
                           cudaStream_t stream);
// Cholesky QR: Q [m,r] = Y L^-T with Y^T Y = L L^T (Gram matrix G [r,r] and its factor in fp64; L32 [r,r] the factor
// in fp32 for the solve).  r <= 1024.  Q may alias Y.  Sets TRANSMLA_DEV_NUMERIC if the Gram matrix is not positive definite.
constexpr int kGramPartials = 8;  // partial Gram matrices [r,r] fp64 that `partial` must hold
cudaError_t cholesky_qr(const float* Y, int m, int r, double* partial, double* G, float* L32, float* Q, int32_t* dev_status,
                        cudaStream_t stream);

}  // namespace conv
}  // namespace transmla
