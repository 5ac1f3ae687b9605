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
template <int MT, int UNROLL>
__device__ __forceinline__ void append_partial(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ wrow,
                                               int D, int T, int t0, int k_lo, int slice, int g, int t4,
                                               float (&acc)[kAppendMaxMT][4]) {
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
    const uint4 wv = ld_u128(wrow + k);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
      if (ok[mt][0]) x0 = ld_u128(xr[mt][0] + k);
      if (ok[mt][1]) x1 = ld_u128(xr[mt][1] + k);
      const uint32_t a0[4] = {x0.x, x1.x, x0.y, x1.y}, a1[4] = {x0.z, x1.z, x0.w, x1.w};
      mma_bf16_16816(acc[mt], a0, wv.x, wv.y);
      mma_bf16_16816(acc[mt], a1, wv.z, wv.w);
    }
  }
}


// x [*, K] row-major, w [*, K] row-major (K a multiple of 256), tokens [t_begin, t_end).  smem_raw: kAppendSmem bytes.
// epi(token, pair 0..3, value of feature f0 + 2*pair, value of feature f0 + 2*pair + 1) is called once per pair.
template <class Epi>
__device__ __forceinline__ void skinny_gemm_tile(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                                                 int K, int f0, int t_begin, int t_end, unsigned char* smem_raw, Epi epi) {
  float* red = reinterpret_cast<float*>(smem_raw);  // [8 warps][128 rows][8]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int slice = K / 8, k_lo = warp * slice;
  const __nv_bfloat16* wrow = w + static_cast<size_t>(f0 + g) * K + k_lo + t4 * 8;
  if (t4 == 0)
    for (int k = 0; k < slice; k += 64) prefetch_l2(wrow + k);  // 128-byte lines of this warp's 8 weight rows
  pdl_wait();  // activations and everything the epilogue touches may belong to kernels still in flight; weights may not
  const int T = t_end;
  for (int t0 = t_begin; t0 < T; t0 += kAppendMaxMT * 16) {
    float acc[kAppendMaxMT][4];
#pragma unroll
    for (int mt = 0; mt < kAppendMaxMT; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;
    const int left = T - t0;
    if (left <= 16) append_partial<1, 8>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    else if (left <= 32) append_partial<2, 4>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    else if (left <= 64) append_partial<4, 4>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    else append_partial<8, 2>(x, wrow, K, T, t0, k_lo, slice, g, t4, acc);
    __syncthreads();  // previous pass has consumed `red`
#pragma unroll
    for (int mt = 0; mt < kAppendMaxMT; ++mt) {
      if (mt * 16 < left) {
        float* d = red + (warp * kAppendMaxMT * 16 + mt * 16 + g) * 8 + t4 * 2;
        *reinterpret_cast<float2*>(d) = make_float2(acc[mt][0], acc[mt][1]);
        *reinterpret_cast<float2*>(d + 64) = make_float2(acc[mt][2], acc[mt][3]);
      }
    }
    __syncthreads();
    const int rows = min(kAppendMaxMT * 16, left);
    for (int i = tid; i < rows * 4; i += 256) {
      const int row = i >> 2, pr = i & 3;
      float re = 0.f, im = 0.f;
#pragma unroll
      for (int wv = 0; wv < 8; ++wv) {
        const float2 v = *reinterpret_cast<const float2*>(red + (wv * kAppendMaxMT * 16 + row) * 8 + pr * 2);
        re += v.x; im += v.y;
      }
      epi(t0 + row, pr, re, im);
    }
  }
}

}  // namespace transmla
