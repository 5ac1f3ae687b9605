// Kernels of the GQA -> MLA conversion on calibration activations (Sec. 4.2, 4.3; App. B, C, D).
// fp32 SIMT arithmetic (fp64 where the orthonormalisation needs it): the results are eigenvectors and low-rank
// bases, and the step is a one-off per model, bound by the two large contractions (the joint second moment and
// the subspace iteration's products).
#include "conversion.cuh"

namespace transmla {
namespace conv {

// ------------------------------------------------------------------------------------------------ GEMM
// 128 x 128 tile, 256 threads x (8 x 8) outputs, k in steps of 16 through two shared-memory buffers: the next
// tile's global loads (16 bytes each where the storage allows, element by element at ragged edges or odd strides)
// are in flight while the current tile is multiplied.  Any of the four storage combinations, no shape restriction.
constexpr int BM = 128, BN = 128, BK = 16;

// One operand tile [128 x BK] as two float4 per thread.  `rows_major`: the operand is stored [rows, K] (k contiguous),
// otherwise [K, rows] (rows contiguous).  r0 = first row of the tile, R = row count, ld = storage stride.
struct TileRegs { float4 v[2]; };
__device__ __forceinline__ void fetch_tile(TileRegs& t, const float* P, bool rows_major, bool vec, int ld, int r0, int R, int k0,
                                           int K, int tid) {
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int f = tid + 256 * u;
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    if (rows_major) {
      const int rr = r0 + f / 4, k = k0 + (f % 4) * 4;
      if (rr < R) {
        const float* src = P + static_cast<size_t>(rr) * ld + k;
        if (vec && k + 3 < K) { const float4 q = *reinterpret_cast<const float4*>(src); x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w; }
        else {
#pragma unroll
          for (int c = 0; c < 4; ++c) if (k + c < K) x[c] = src[c];
        }
      }
    } else {
      const int k = k0 + f / 32, rr = r0 + (f % 32) * 4;
      if (k < K) {
        const float* src = P + static_cast<size_t>(k) * ld + rr;
        if (vec && rr + 3 < R) { const float4 q = *reinterpret_cast<const float4*>(src); x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w; }
        else {
#pragma unroll
          for (int c = 0; c < 4; ++c) if (rr + c < R) x[c] = src[c];
        }
      }
    }
    t.v[u] = make_float4(x[0], x[1], x[2], x[3]);
  }
}
__device__ __forceinline__ void stash_tile(const TileRegs& t, float (*S)[BM + 4], bool rows_major, int tid) {
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int f = tid + 256 * u;
    if (rows_major) {
      const int rr = f / 4, kq = (f % 4) * 4;
      S[kq][rr] = t.v[u].x; S[kq + 1][rr] = t.v[u].y; S[kq + 2][rr] = t.v[u].z; S[kq + 3][rr] = t.v[u].w;
    } else {
      *reinterpret_cast<float4*>(&S[f / 32][(f % 32) * 4]) = t.v[u];
    }
  }
}

template <typename TOut>
__global__ void __launch_bounds__(256) gemm_kernel(int ta, int tb, int M, int N, int K, float alpha, const float* A, int lda,
                                                   long long strideA, const float* B, int ldb, long long strideB, TOut* C,
                                                   int ldc, long long strideC, int k_total) {
  __shared__ __align__(16) float As[2][BK][BM + 4];
  __shared__ __align__(16) float Bs[2][BK][BN + 4];
  A += strideA * blockIdx.z;
  B += strideB * blockIdx.z;
  C += strideC * blockIdx.z;
  if (k_total > 0) K = max(0, min(K, k_total - static_cast<int>(blockIdx.z) * K));  // batch = slices of one long K
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const bool a_rows = !ta, b_rows = tb != 0;   // stored [rows, K]?
  const bool vec_a = (lda & 3) == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0;
  const bool vec_b = (ldb & 3) == 0 && (reinterpret_cast<uintptr_t>(B) & 15) == 0;
  TOut acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = TOut(0);
  TileRegs ra, rb;
  if (K > 0) {
    fetch_tile(ra, A, a_rows, vec_a, lda, m0, M, 0, K, tid);
    fetch_tile(rb, B, b_rows, vec_b, ldb, n0, N, 0, K, tid);
    stash_tile(ra, As[0], a_rows, tid);
    stash_tile(rb, Bs[0], b_rows, tid);
  }
  __syncthreads();
  for (int k0 = 0; k0 < K; k0 += BK) {
    const int buf = (k0 / BK) & 1;
    const bool more = k0 + BK < K;
    if (more) {
      fetch_tile(ra, A, a_rows, vec_a, lda, m0, M, k0 + BK, K, tid);
      fetch_tile(rb, B, b_rows, vec_b, ldb, n0, N, k0 + BK, K, tid);
    }
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][kk][ty * 4]), a1 = *reinterpret_cast<const float4*>(&As[buf][kk][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][kk][tx * 4]), b1 = *reinterpret_cast<const float4*>(&Bs[buf][kk][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] += static_cast<TOut>(a[i]) * static_cast<TOut>(b[j]);
    }
    if (more) {
      stash_tile(ra, As[buf ^ 1], a_rows, tid);
      stash_tile(rb, Bs[buf ^ 1], b_rows, tid);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + ty * 4 + (i & 3) + (i >> 2) * 64;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int n = n0 + tx * 4 + (j & 3) + (j >> 2) * 64;
      if (n < N) C[static_cast<size_t>(m) * ldc + n] = static_cast<TOut>(alpha) * acc[i][j];
    }
  }
}

cudaError_t gemm_f32(int ta, int tb, int M, int N, int K, float alpha, const float* A, int lda, long long strideA,
                     const float* B, int ldb, long long strideB, float* C, int ldc, long long strideC, int batch,
                     cudaStream_t stream) {
  if (M <= 0 || N <= 0 || batch <= 0) return cudaSuccess;
  dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM, batch);
  gemm_kernel<float><<<grid, 256, 0, stream>>>(ta, tb, M, N, K, alpha, A, lda, strideA, B, ldb, strideB, C, ldc, strideC, 0);
  return cudaGetLastError();
}

// G [r,r] (fp64) = Y^T Y for Y [m,r]: the long sum over m is cut into kGramSlices slices, one batch entry each
// (16 tiles alone would leave most SMs idle), and the partial sums are added in a fixed order.
constexpr int kGramSlices = kGramPartials;
__global__ void sum_slices_kernel(const double* part, int count, int slices, double* out) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= count) return;
  double s = 0.0;
  for (int i = 0; i < slices; ++i) s += part[static_cast<size_t>(i) * count + e];
  out[e] = s;
}
cudaError_t gram_f64(const float* Y, int m, int r, double* partial, double* G, cudaStream_t stream) {
  const int ks = (m + kGramSlices - 1) / kGramSlices;
  dim3 grid((r + BN - 1) / BN, (r + BM - 1) / BM, kGramSlices);
  gemm_kernel<double><<<grid, 256, 0, stream>>>(1, 0, r, r, ks, 1.f, Y, r, static_cast<long long>(ks) * r, Y, r,
                                                static_cast<long long>(ks) * r, partial, r, static_cast<long long>(r) * r, m);
  sum_slices_kernel<<<(r * r + 255) / 256, 256, 0, stream>>>(partial, r * r, kGramSlices, G);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------ RoRoPE helpers
// Position in the merged key of segment entry i of group G (i = p*g + j: frequency G*fold + p, head j), real part.
__device__ __forceinline__ int seg_pos(int G, int i, int g, int d, int fold) {
  const int p = i / g, j = i - p * g;
  return j * d + 2 * (G * fold + p);
}

__global__ void gather_segments_kernel(const float* K, int n, int g, int d, int fold, float* seg) {
  const int m = g * fold, G = blockIdx.y;
  const size_t total = static_cast<size_t>(2) * n * m;
  for (size_t e = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; e < total; e += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const int i = static_cast<int>(e % m);
    const size_t row = e / m;                       // 0..2n-1
    const int t = static_cast<int>(row % n), im = static_cast<int>(row / n);
    seg[static_cast<size_t>(G) * total + e] = K[static_cast<size_t>(t) * g * d + seg_pos(G, i, g, d, fold) + im];
  }
}

cudaError_t gather_segments(const float* K, int n, int g, int d, int fold, float* seg, cudaStream_t stream) {
  const int groups = d / 2 / fold;
  dim3 grid(296, groups);
  gather_segments_kernel<<<grid, 256, 0, stream>>>(K, n, g, d, fold, seg);
  return cudaGetLastError();
}

// Y[(q / fold, 2 (G fold + q % fold) + im), c] = sum_i U_G[i, q] X[seg_pos(G, i) + im, c]   (Eq. 18)
__global__ void rorope_apply_kernel(const float* X, int C, const float* U, int g, int d, int fold, float* Y) {
  const int m = g * fold, G = blockIdx.y, im = blockIdx.z;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  extern __shared__ float u_s[];  // U_G [m][m]
  for (int e = threadIdx.x; e < m * m; e += blockDim.x) u_s[e] = U[static_cast<size_t>(G) * m * m + e];
  __syncthreads();
  if (c >= C) return;
  for (int q0 = 0; q0 < m; q0 += 8) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int i = 0; i < m; ++i) {
      const float x = X[static_cast<size_t>(seg_pos(G, i, g, d, fold) + im) * C + c];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (q0 + u < m) acc[u] = fmaf(u_s[i * m + q0 + u], x, acc[u]);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int q = q0 + u;
      if (q < m) Y[static_cast<size_t>((q / fold) * d + 2 * (G * fold + q % fold) + im) * C + c] = acc[u];
    }
  }
}

cudaError_t rorope_apply(const float* X, int C, const float* U, int g, int d, int fold, float* Y, cudaStream_t stream) {
  const int m = g * fold, groups = d / 2 / fold;
  const size_t smem = static_cast<size_t>(m) * m * sizeof(float);
  if (smem > 48 * 1024) {
    if (cudaError_t e = cudaFuncSetAttribute(rorope_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        e != cudaSuccess)
      return e;
  }
  dim3 grid((C + 127) / 128, groups, 2);
  rorope_apply_kernel<<<grid, 128, smem, stream>>>(X, C, U, g, d, fold, Y);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------ Eq. 19
// norms[0..n) = ||k_nope,t||, norms[n..2n) = ||v_t||: one warp per row; then one block sums both halves in a fixed
// order (the same bits on every run) and writes alpha = mean ||k|| / mean ||v||.
__global__ void row_norms_kernel(const float* a, int n, int m, float* out) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= n) return;
  float s = 0.f;
  for (int c = lane; c < m; c += 32) { const float x = a[static_cast<size_t>(row) * m + c]; s = fmaf(x, x, s); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) out[row] = sqrtf(s);
}
__global__ void __launch_bounds__(1024) alpha_kernel(const float* norms, int n, float* alpha_out) {
  __shared__ double part[2][1024];
  double sk = 0.0, sv = 0.0;
  for (int i = threadIdx.x; i < n; i += 1024) { sk += norms[i]; sv += norms[n + i]; }
  part[0][threadIdx.x] = sk; part[1][threadIdx.x] = sv;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) { part[0][threadIdx.x] += part[0][threadIdx.x + o]; part[1][threadIdx.x] += part[1][threadIdx.x + o]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) *alpha_out = static_cast<float>(part[0][0] / part[1][0]);
}
cudaError_t row_norm_ratio(const float* k_nope, int n, int mk, const float* v, int mv, float* scratch, float* alpha_out,
                           cudaStream_t stream) {
  row_norms_kernel<<<(n + 7) / 8, 256, 0, stream>>>(k_nope, n, mk, scratch);
  row_norms_kernel<<<(n + 7) / 8, 256, 0, stream>>>(v, n, mv, scratch + n);
  alpha_kernel<<<1, 1024, 0, stream>>>(scratch, n, alpha_out);
  return cudaGetLastError();
}

// Z[t] = [k_nope,t / alpha ; v_t]   (App. D.2 step 1)
__global__ void balance_concat_kernel(const float* k_nope, int n, int mk, const float* v, int mv, const float* alpha, float* Z) {
  const float inv = 1.f / *alpha;
  const int m = mk + mv;
  const size_t total = static_cast<size_t>(n) * m;
  for (size_t e = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; e < total; e += static_cast<size_t>(gridDim.x) * blockDim.x) {
    const size_t t = e / m;
    const int c = static_cast<int>(e % m);
    Z[e] = c < mk ? k_nope[t * mk + c] * inv : v[t * mv + (c - mk)];
  }
}
cudaError_t balance_concat(const float* k_nope, int n, int mk, const float* v, int mv, const float* alpha, float* Z,
                           cudaStream_t stream) {
  balance_concat_kernel<<<592, 256, 0, stream>>>(k_nope, n, mk, v, mv, alpha, Z);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------ eigenvectors
// Parallel cyclic Jacobi for a symmetric matrix of order m <= 128, one block per matrix, A and V in shared memory.
// A round rotates m/2 disjoint index pairs (round-robin tournament), all with angles taken from the matrix as it
// stands before the round: columns first (A <- A J, V <- V J), then rows (A <- J^T A).  Sweeps stop when the
// off-diagonal mass is below fp32 resolution of the whole; the eigenvalues are then sorted in descending order.
constexpr int kEigMax = 128, kEigSweeps = 30, kEigThreads = 512;

__global__ void __launch_bounds__(kEigThreads) jacobi_eigh_kernel(const float* a_in, int m, float* eigvals, float* eigvecs,
                                                          int32_t* dev_status) {
  extern __shared__ float es[];
  const int ld = m + 1, mm = (m + 1) & ~1, half = mm / 2;
  float* A = es;                    // [m][ld]
  float* V = A + m * ld;            // [m][ld]
  float* cs = V + m * ld;           // [half][2]
  int* pq = reinterpret_cast<int*>(cs + 2 * half);  // [half][2]
  int* order = pq + 2 * half;       // [m]
  __shared__ float red[kEigThreads];
  __shared__ int done;
  const int tid = threadIdx.x;
  const float* src = a_in + static_cast<size_t>(blockIdx.x) * m * m;
  for (int e = tid; e < m * m; e += kEigThreads) {
    const int i = e / m, j = e % m;
    A[i * ld + j] = 0.5f * (src[e] + src[j * m + i]);  // exactly symmetric whatever rounding the input carries
    V[i * ld + j] = i == j ? 1.f : 0.f;
  }
  if (tid == 0) done = 0;
  __syncthreads();
  float prev_off = 3.4e38f;
  for (int sweep = 0; sweep < kEigSweeps; ++sweep) {
    // convergence: off-diagonal sum of squares against the whole
    float off = 0.f, tot = 0.f;
    for (int e = tid; e < m * m; e += kEigThreads) {
      const int i = e / m, j = e % m;
      const float x = A[i * ld + j];
      tot += x * x;
      if (i != j) off += x * x;
    }
    red[tid] = off; __syncthreads();
    for (int o = kEigThreads / 2; o > 0; o >>= 1) { if (tid < o) red[tid] += red[tid + o]; __syncthreads(); }
    const float off_all = red[0]; __syncthreads();
    red[tid] = tot; __syncthreads();
    for (int o = kEigThreads / 2; o > 0; o >>= 1) { if (tid < o) red[tid] += red[tid + o]; __syncthreads(); }
    const float tot_all = red[0]; __syncthreads();
    // converged: the off-diagonal mass is gone, or it sits at the fp32 rounding floor of the rotations (it has
    // stopped shrinking and is below 1e-8 of the whole)
    if (off_all <= 1e-13f * tot_all || (sweep >= 4 && off_all > 0.25f * prev_off && off_all <= 1e-8f * tot_all)) {
      if (tid == 0) done = 1;
      __syncthreads();
      break;
    }
    prev_off = off_all;
    for (int rd = 0; rd < mm - 1; ++rd) {
      if (tid < half) {
        int p, q;
        if (tid == 0) { p = mm - 1; q = rd; }
        else { p = (rd + tid) % (mm - 1); q = (rd - tid + mm - 1) % (mm - 1); }
        if (p > q) { const int t = p; p = q; q = t; }
        float c = 1.f, s = 0.f;
        if (q < m) {
          const float apq = A[p * ld + q], app = A[p * ld + p], aqq = A[q * ld + q];
          if (fabsf(apq) > 1e-30f) {
            const float theta = (aqq - app) / (2.f * apq);
            const float t = (theta >= 0.f ? 1.f : -1.f) / (fabsf(theta) + sqrtf(theta * theta + 1.f));
            c = 1.f / sqrtf(t * t + 1.f);
            s = t * c;
          }
        } else { p = -1; }
        pq[2 * tid] = p; pq[2 * tid + 1] = q; cs[2 * tid] = c; cs[2 * tid + 1] = s;
      }
      __syncthreads();
      for (int e = tid; e < half * m; e += kEigThreads) {      // columns p, q of A and V
        const int k = e / m, i = e % m, p = pq[2 * k], q = pq[2 * k + 1];
        if (p < 0) continue;
        const float c = cs[2 * k], s = cs[2 * k + 1];
        const float ap = A[i * ld + p], aq = A[i * ld + q];
        A[i * ld + p] = c * ap - s * aq; A[i * ld + q] = s * ap + c * aq;
        const float vp = V[i * ld + p], vq = V[i * ld + q];
        V[i * ld + p] = c * vp - s * vq; V[i * ld + q] = s * vp + c * vq;
      }
      __syncthreads();
      for (int e = tid; e < half * m; e += kEigThreads) {      // rows p, q of A
        const int k = e / m, j = e % m, p = pq[2 * k], q = pq[2 * k + 1];
        if (p < 0) continue;
        const float c = cs[2 * k], s = cs[2 * k + 1];
        const float ap = A[p * ld + j], aq = A[q * ld + j];
        A[p * ld + j] = c * ap - s * aq; A[q * ld + j] = s * ap + c * aq;
      }
      __syncthreads();
    }
  }
  if (tid == 0) {
    if (!done && dev_status != nullptr) atomicOr(dev_status, TRANSMLA_DEV_NUMERIC);
    for (int i = 0; i < m; ++i) order[i] = i;
    for (int i = 0; i < m; ++i) {       // selection sort, descending (stable for equal values)
      int best = i;
      for (int j = i + 1; j < m; ++j)
        if (A[order[j] * ld + order[j]] > A[order[best] * ld + order[best]]) best = j;
      const int t = order[best];
      for (int j = best; j > i; --j) order[j] = order[j - 1];
      order[i] = t;
    }
  }
  __syncthreads();
  float* w = eigvals + static_cast<size_t>(blockIdx.x) * m;
  float* vec = eigvecs + static_cast<size_t>(blockIdx.x) * m * m;
  for (int q = tid; q < m; q += kEigThreads) w[q] = A[order[q] * ld + order[q]];
  for (int e = tid; e < m * m; e += kEigThreads) { const int i = e / m, q = e % m; vec[e] = V[i * ld + order[q]]; }
}

cudaError_t sym_eig(float* a, int batch, int m, float* eigvals, float* eigvecs, int32_t* dev_status, cudaStream_t stream) {
  if (m < 1 || m > kEigMax) return cudaErrorInvalidValue;
  const int half = ((m + 1) & ~1) / 2;
  const size_t smem = (static_cast<size_t>(2) * m * (m + 1) + 4 * half + m) * sizeof(float);
  if (cudaError_t e = cudaFuncSetAttribute(jacobi_eigh_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
      e != cudaSuccess)
    return e;
  jacobi_eigh_kernel<<<batch, kEigThreads, smem, stream>>>(a, m, eigvals, eigvecs, dev_status);
  return cudaGetLastError();
}
// ------------------------------------------------------------------------------------------------ orthonormalisation
// Cholesky QR: G = Y^T Y = L L^T, Q = Y L^-T.
// cholesky_kernel: blocked right-looking factorisation of the fp64 Gram matrix in place, one block.  Panels of 32
// columns are factored in shared memory (all rows below the diagonal block with them); the trailing matrix then takes
// one rank-32 update per panel, so that an element of G is read and written 16 times instead of 512.  L is also
// written as fp32 for the solve.
constexpr int kCholMax = 1024, kCholNb = 32;
__global__ void __launch_bounds__(1024) cholesky_kernel(double* G, int r, float* L32, int32_t* dev_status) {
  extern __shared__ double ps[];  // panel [r - kb][kCholNb + 1]
  __shared__ int bad;
  constexpr int ld = kCholNb + 1;
  const int tid = threadIdx.x, tx = tid & 31, ty = tid >> 5;
  if (tid == 0) bad = 0;
  __syncthreads();
  for (int kb = 0; kb < r; kb += kCholNb) {
    const int nb = min(kCholNb, r - kb), rows = r - kb;
    for (int e = tid; e < rows * nb; e += 1024) { const int i = e / nb, j = e % nb; ps[i * ld + j] = G[static_cast<size_t>(kb + i) * r + kb + j]; }
    __syncthreads();
    for (int k = 0; k < nb; ++k) {
      if (tid == 0) {
        double d = ps[k * ld + k];
        if (!(d > 0.0)) { bad = 1; d = 1.0; }
        ps[k * ld + k] = sqrt(d);
      }
      __syncthreads();
      const double dk = ps[k * ld + k];
      for (int i = k + 1 + tid; i < rows; i += 1024) ps[i * ld + k] /= dk;
      __syncthreads();
      for (int e = tid; e < (rows - k - 1) * (nb - k - 1); e += 1024) {
        const int i = k + 1 + e / (nb - k - 1), j = k + 1 + e % (nb - k - 1);
        ps[i * ld + j] -= ps[i * ld + k] * ps[j * ld + k];
      }
      __syncthreads();
    }
    for (int e = tid; e < rows * nb; e += 1024) {
      const int i = e / nb, j = e % nb;
      const double v = (kb + j <= kb + i) ? ps[i * ld + j] : 0.0;
      G[static_cast<size_t>(kb + i) * r + kb + j] = v;
      L32[static_cast<size_t>(kb + i) * r + kb + j] = static_cast<float>(v);
    }
    // trailing update: G[i][j] -= sum_k P[i][k] P[j][k] for i >= j >= kb + nb
    for (int i = nb + ty; i < rows; i += 32) {
      for (int j = nb + tx; j <= i; j += 32) {
        double acc = 0.0;
#pragma unroll 8
        for (int k = 0; k < nb; ++k) acc += ps[i * ld + k] * ps[j * ld + k];
        G[static_cast<size_t>(kb + i) * r + kb + j] -= acc;
      }
    }
    __syncthreads();
  }
  for (int e = tid; e < r * r; e += 1024) { if (e % r > e / r) L32[e] = 0.f; }
  if (tid == 0 && bad && dev_status != nullptr) atomicOr(dev_status, TRANSMLA_DEV_NUMERIC);
}

// Q[row] L^T = Y[row]: forward substitution along the row, one warp per row (the dot product of step j is split
// over the lanes), 8 rows per block kept in shared memory.  Q may alias Y.
__global__ void __launch_bounds__(256) trsm_rows_kernel(const float* Y, int m, int r, const float* L32, float* Q) {
  extern __shared__ float qs[];  // [8][r]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + warp;
  if (row >= m) return;
  float* q = qs + warp * r;
  for (int c = lane; c < r; c += 32) q[c] = Y[static_cast<size_t>(row) * r + c];
  __syncwarp();
  for (int j = 0; j < r; ++j) {
    const float* lj = L32 + static_cast<size_t>(j) * r;
    float s = 0.f;
    for (int k = lane; k < j; k += 32) s = fmaf(q[k], lj[k], s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) q[j] = (q[j] - s) / lj[j];
    __syncwarp();
  }
  for (int c = lane; c < r; c += 32) Q[static_cast<size_t>(row) * r + c] = q[c];
}

cudaError_t cholesky_qr(const float* Y, int m, int r, double* partial, double* G, float* L32, float* Q, int32_t* dev_status,
                        cudaStream_t stream) {
  if (r > kCholMax) return cudaErrorInvalidValue;
  if (cudaError_t e = gram_f64(Y, m, r, partial, G, stream); e != cudaSuccess) return e;
  const size_t chol_smem = static_cast<size_t>(r) * (kCholNb + 1) * sizeof(double);
  if (cudaError_t e = cudaFuncSetAttribute(cholesky_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(chol_smem));
      e != cudaSuccess)
    return e;
  cholesky_kernel<<<1, 1024, chol_smem, stream>>>(G, r, L32, dev_status);
  const size_t smem = static_cast<size_t>(8) * r * sizeof(float);
  if (smem > 48 * 1024) {
    if (cudaError_t e = cudaFuncSetAttribute(trsm_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        e != cudaSuccess)
      return e;
  }
  trsm_rows_kernel<<<(m + 7) / 8, 256, smem, stream>>>(Y, m, r, L32, Q);
  return cudaGetLastError();
}

}  // namespace conv
}  // namespace transmla
