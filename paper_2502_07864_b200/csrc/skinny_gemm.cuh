// Skinny GEMM tile shared by the append and by the layer's linear maps: y[t, f0..f0+7] = x[t, :] . w[f0..f0+7, :]
// for a range of tokens t (the M dimension of the tensor-core tiles).  One block owns 8 consecutive output
// features; its 8 warps split the contracted dimension and meet in shared memory; every (token, feature pair)
// is handed to an epilogue functor.  Operands are read straight from global memory with 16-byte loads in a
// permuted k order (see small_kernels.cu).
#pragma once
#include "common.cuh"

namespace transmla {

__device__ __forceinline__ uint32_t ld_u32(const __nv_bfloat16* p) { return *reinterpret_cast<const uint32_t*>(p); }
__device__ __forceinline__ uint4 ld_u128(const __nv_bfloat16* p) { return *reinterpret_cast<const uint4*>(p); }

// RoPE of Eq. 1 on the pair (re, im) = elements (2l, 2l+1) of a d-vector at position pos.  The angle is formed
// and reduced to [-pi, pi] in fp64 so that positions of 10^5 keep their phase; sine and cosine are fp32.
__device__ __forceinline__ void rope_pair(float& re, float& im, int pos, int l, int d, float theta) {
  const double ang = static_cast<double>(pos) * exp2(-2.0 * l / d * log2(static_cast<double>(theta)));
  const double red_ang = ang - 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
  float sn, cs;
  sincosf(static_cast<float>(red_ang), &sn, &cs);
  const float nre = re * cs - im * sn, nim = im * cs + re * sn;
  re = nre;
  im = nim;
}

constexpr int kAppendMaxMT = 8;  // 16-token tiles per pass
constexpr size_t kAppendSmem = 8 * kAppendMaxMT * 16 * 8 * sizeof(float);  // 32 KB

// Partial products of one warp over its slice of the hidden dimension for tokens [t0, t0 + 16*MT).
template <int MT, int UNROLL, int MAXMT, int NT>
__device__ __forceinline__ void append_partial(const __nv_bfloat16* x, const __nv_bfloat16* __restrict__ wrow,
                                               int D, int T, int t0, int k_lo, int slice, int g, int t4,
                                               float (&acc)[MAXMT][NT][4]) {
  const __nv_bfloat16* xr[MT][2];
  bool ok[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int row = t0 + mt * 16 + g + hf * 8;
      ok[mt][hf] = row < T;
      xr[mt][hf] = x + static_cast<size_t>(min(row, T - 1)) * D + k_lo + t4 * 8;
    }
#pragma unroll UNROLL
  for (int k = 0; k < slice; k += 32) {
    uint4 wv[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) wv[nt] = ld_u128(wrow + static_cast<size_t>(nt) * 8 * D + k);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
      if (ok[mt][0]) x0 = ld_u128(xr[mt][0] + k);
      if (ok[mt][1]) x1 = ld_u128(xr[mt][1] + k);
      const uint32_t a0[4] = {x0.x, x1.x, x0.y, x1.y}, a1[4] = {x0.z, x1.z, x0.w, x1.w};
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        mma_bf16_16816(acc[mt][nt], a0, wv[nt].x, wv[nt].y);
        mma_bf16_16816(acc[mt][nt], a1, wv[nt].z, wv[nt].w);
      }
    }
  }
}

// Shared memory the tile needs for the meeting of its 8 warps.
constexpr size_t skinny_gemm_smem(int maxmt, int nt) { return static_cast<size_t>(8) * maxmt * 16 * 8 * nt * sizeof(float); }

// x [*, K] row-major, w [*, K] row-major (K a multiple of 256), tokens [t_begin, t_end), output features
// f0 .. f0 + 8*NT - 1.  smem_raw: skinny_gemm_smem(MAXMT, NT) bytes.
// epi(token, pair 0..4*NT-1, value of feature f0 + 2*pair, value of feature f0 + 2*pair + 1) is called once per pair.
// MAXMT: 16-token tiles per pass.  NT: 8-feature tiles per block; more of them re-read the activations less often,
// which is what bounds these kernels once the weights are large (every block reads all its tokens' activations).
template <int MAXMT = kAppendMaxMT, int NT = 1, class Epi>
__device__ __forceinline__ void skinny_gemm_tile(const __nv_bfloat16* x, const __nv_bfloat16* __restrict__ w,
                                                 int K, int f0, int t_begin, int t_end, unsigned char* smem_raw, Epi epi) {
  float* red = reinterpret_cast<float*>(smem_raw);  // [8 warps][MAXMT*16 rows][8*NT]
  constexpr int kCols = 8 * NT;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int slice = K / 8, k_lo = warp * slice;
  const __nv_bfloat16* wrow = w + static_cast<size_t>(f0 + g) * K + k_lo + t4 * 8;
  if (t4 == 0)
    for (int nt = 0; nt < NT; ++nt)
      for (int k = 0; k < slice; k += 64) prefetch_l2(wrow + static_cast<size_t>(nt) * 8 * K + k);  // this warp's weight lines
  pdl_wait();  // activations and everything the epilogue touches may belong to kernels still in flight; weights may not
  const int T = t_end;
  for (int t0 = t_begin; t0 < T; t0 += MAXMT * 16) {
    float acc[MAXMT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MAXMT; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) acc[mt][nt][0] = acc[mt][nt][1] = acc[mt][nt][2] = acc[mt][nt][3] = 0.f;
    const int left = T - t0;
    constexpr int U1 = NT == 1 ? 8 : 4, U2 = NT == 1 ? 4 : 2;
    if (left <= 16) append_partial<1, U1, MAXMT, NT>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    else if (MAXMT == 2 || left <= 32) append_partial<(MAXMT >= 2 ? 2 : MAXMT), U2, MAXMT, NT>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    else if (left <= 64) append_partial<(MAXMT >= 4 ? 4 : MAXMT), U2, MAXMT, NT>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    else append_partial<MAXMT, (NT == 1 ? 2 : 1), MAXMT, NT>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    __syncthreads();  // previous pass has consumed `red`
#pragma unroll
    for (int mt = 0; mt < MAXMT; ++mt) {
      if (mt * 16 < left) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float* d = red + (warp * MAXMT * 16 + mt * 16 + g) * kCols + nt * 8 + t4 * 2;
          *reinterpret_cast<float2*>(d) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
          *reinterpret_cast<float2*>(d + 8 * kCols) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
      }
    }
    __syncthreads();
    const int rows = min(MAXMT * 16, left);
    for (int i = tid; i < rows * 4 * NT; i += 256) {
      const int row = i / (4 * NT), pr = i % (4 * NT);
      float re = 0.f, im = 0.f;
#pragma unroll
      for (int wv = 0; wv < 8; ++wv) {
        const float2 v = *reinterpret_cast<const float2*>(red + (wv * MAXMT * 16 + row) * kCols + pr * 2);
        re += v.x; im += v.y;
      }
      epi(t0 + row, pr, re, im);
    }
  }
}

}  // namespace transmla
