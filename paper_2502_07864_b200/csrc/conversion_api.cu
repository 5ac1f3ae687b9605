// C ABI of the conversion steps (Sec. 4.2, 4.3; App. B, C, D).  All matrices fp32, dense, row-major, on the device.
#include "conversion.cuh"

using namespace transmla;

namespace {
inline bool al16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline transmla_status_t done(cudaError_t e) { return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA; }
inline bool rorope_shape_ok(int g, int d, int fold) {
  return g >= 1 && d >= 2 && d % 2 == 0 && fold >= 1 && (d / 2) % fold == 0 && g * fold <= 128;
}
}  // namespace

extern "C" {

transmla_status_t transmla_conv_gemm(int ta, int tb, int M, int N, int K, float alpha, const float* A, int lda, const float* B,
                                     int ldb, float* C, int ldc, void* stream) {
  if (!A || !B || !C) return TRANSMLA_ERR_NULL;
  if (M < 1 || N < 1 || K < 1 || lda < (ta ? M : K) || ldb < (tb ? K : N) || ldc < N) return TRANSMLA_ERR_SHAPE;
  return done(conv::gemm_f32(ta, tb, M, N, K, alpha, A, lda, 0, B, ldb, 0, C, ldc, 0, 1, static_cast<cudaStream_t>(stream)));
}

size_t transmla_conv_rorope_scratch_bytes(int n, int g, int d, int fold) {
  if (n < 1 || !rorope_shape_ok(g, d, fold)) return 0;
  return static_cast<size_t>(d / 2 / fold) * 2 * n * g * fold * sizeof(float);
}

transmla_status_t transmla_conv_rorope_covariance(const float* K, int n, int g, int d, int fold, void* scratch,
                                                  size_t scratch_bytes, float* cov, void* stream) {
  if (!K || !scratch || !cov) return TRANSMLA_ERR_NULL;
  if (n < 1 || !rorope_shape_ok(g, d, fold)) return TRANSMLA_ERR_SHAPE;
  if (!al16(K) || !al16(scratch) || !al16(cov)) return TRANSMLA_ERR_ALIGN;
  if (scratch_bytes < transmla_conv_rorope_scratch_bytes(n, g, d, fold)) return TRANSMLA_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* seg = static_cast<float*>(scratch);
  const int m = g * fold, groups = d / 2 / fold;
  if (cudaError_t e = conv::gather_segments(K, n, g, d, fold, seg, s); e != cudaSuccess) return TRANSMLA_ERR_CUDA;
  // sigma_x + sigma_y = [K_x ; K_y]^T [K_x ; K_y] per group
  return done(conv::gemm_f32(1, 0, m, m, 2 * n, 1.f, seg, m, static_cast<long long>(2) * n * m, seg, m,
                             static_cast<long long>(2) * n * m, cov, m, static_cast<long long>(m) * m, groups, s));
}

transmla_status_t transmla_conv_sym_eig(float* a, int batch, int m, float* eigvals, float* eigvecs, int32_t* dev_status,
                                        void* stream) {
  if (!a || !eigvals || !eigvecs) return TRANSMLA_ERR_NULL;
  if (batch < 1 || m < 1 || m > 128) return TRANSMLA_ERR_SHAPE;
  return done(conv::sym_eig(a, batch, m, eigvals, eigvecs, dev_status, static_cast<cudaStream_t>(stream)));
}

transmla_status_t transmla_conv_rorope_apply(const float* X, int C, const float* U, int g, int d, int fold, float* Y, void* stream) {
  if (!X || !U || !Y) return TRANSMLA_ERR_NULL;
  if (C < 1 || !rorope_shape_ok(g, d, fold) || X == Y) return TRANSMLA_ERR_SHAPE;
  return done(conv::rorope_apply(X, C, U, g, d, fold, Y, static_cast<cudaStream_t>(stream)));
}

transmla_status_t transmla_conv_alpha(const float* k_nope, int n, int mk, const float* v, int mv, float* scratch, float* alpha_out,
                                      void* stream) {
  if (!k_nope || !v || !scratch || !alpha_out) return TRANSMLA_ERR_NULL;
  if (n < 1 || mk < 1 || mv < 1) return TRANSMLA_ERR_SHAPE;
  return done(conv::row_norm_ratio(k_nope, n, mk, v, mv, scratch, alpha_out, static_cast<cudaStream_t>(stream)));
}

transmla_status_t transmla_conv_balance_concat(const float* k_nope, int n, int mk, const float* v, int mv, const float* alpha,
                                               float* Z, void* stream) {
  if (!k_nope || !v || !alpha || !Z) return TRANSMLA_ERR_NULL;
  if (n < 1 || mk < 1 || mv < 1) return TRANSMLA_ERR_SHAPE;
  return done(conv::balance_concat(k_nope, n, mk, v, mv, alpha, Z, static_cast<cudaStream_t>(stream)));
}

size_t transmla_conv_subspace_scratch_bytes(int m, int r) {
  if (m < 1 || r < 1 || r > m || r > 1024) return 0;
  return static_cast<size_t>(m) * r * sizeof(float) + static_cast<size_t>(r) * r * ((conv::kGramPartials + 1) * sizeof(double) + sizeof(float)) + 512;
}

transmla_status_t transmla_conv_top_subspace(const float* Cmat, int m, int r, int iters, float* Q, void* scratch,
                                             size_t scratch_bytes, int32_t* dev_status, void* stream) {
  if (!Cmat || !Q || !scratch) return TRANSMLA_ERR_NULL;
  if (m < 1 || r < 1 || r > m || r > 1024 || iters < 1) return TRANSMLA_ERR_SHAPE;
  if (!al16(Cmat) || !al16(Q) || (reinterpret_cast<uintptr_t>(scratch) & 255)) return TRANSMLA_ERR_ALIGN;
  if (scratch_bytes < transmla_conv_subspace_scratch_bytes(m, r)) return TRANSMLA_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(scratch);
  double* partial = reinterpret_cast<double*>(w);
  double* G = partial + static_cast<size_t>(conv::kGramPartials) * r * r;
  float* L32 = reinterpret_cast<float*>(G + static_cast<size_t>(r) * r);
  float* Y = reinterpret_cast<float*>(
      w + ((static_cast<size_t>(r) * r * ((conv::kGramPartials + 1) * sizeof(double) + sizeof(float)) + 255) & ~size_t(255)));
  // Orthogonal iteration: Q <- orth(C Q).  One Cholesky QR per round keeps the columns independent; the basis is made
  // orthonormal to fp32 resolution by the two passes at the start and the extra pass at the end.
  auto orth = [&](float* y, float* q) { return conv::cholesky_qr(y, m, r, partial, G, L32, q, dev_status, s) == cudaSuccess; };
  if (!orth(Q, Q) || !orth(Q, Q)) return TRANSMLA_ERR_CUDA;
  for (int it = 0; it < iters; ++it) {
    if (conv::gemm_f32(0, 0, m, r, m, 1.f, Cmat, m, 0, Q, r, 0, Y, r, 0, 1, s) != cudaSuccess) return TRANSMLA_ERR_CUDA;
    if (!orth(Y, Q)) return TRANSMLA_ERR_CUDA;
  }
  return orth(Q, Q) ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

}  // extern "C"
