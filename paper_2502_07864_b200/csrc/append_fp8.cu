// Latent append into the FP8 cache (Eq. 7 left, then this library's FP8 row format): the projection and RoPE run as in
// the bf16 append but leave fp32 rows in a scratch buffer, because a row's scale is the maximum over all of its 512
// latent values, which 64 different blocks of the projection produce; a second, tiny launch quantises the rows.
#include <cuda_fp16.h>

#include "common.cuh"
#include "skinny_gemm.cuh"

namespace transmla {

// y[t, :] = [W_DKV; W_KR] x_t with RoPE on y[r:], fp32, into scratch [T, r + dR].
__global__ void __launch_bounds__(256) append_rows_f32_kernel(const __nv_bfloat16* x, const __nv_bfloat16* __restrict__ w,
                                                              const int32_t* positions, float* rows, int B, int S, int D, int r,
                                                              int dR, float theta) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_trigger();
  const int K = r + dR, f0 = blockIdx.x * 8;
  skinny_gemm_tile<kAppendMaxMT, 1>(x, w, D, f0, 0, B * S, smem_raw, [&](int t, int pr, float re, float im) {
    const int f = f0 + pr * 2;
    if (f >= r) rope_pair(re, im, positions[t / S] + t % S, (f - r) >> 1, dR, theta);  // RoPE pair l of the decoupled key (Eq. 1)
    *reinterpret_cast<float2*>(rows + static_cast<size_t>(t) * K + f) = make_float2(re, im);
  });
}

// One warp per token: scale = max|c| / 448 (1 for an all-zero row), codes = e4m3(c / scale), k^R / scale as bf16,
// written to the token's 656-byte row.  r = 512, dR = 64.
__global__ void __launch_bounds__(128) quantize_rows_kernel(const float* rows, const int32_t* positions, const int32_t* page_table,
                                                            unsigned char* cache, int32_t* dev_status, int B, int S,
                                                            int num_pages, int max_pages) {
  pdl_trigger();
  pdl_wait();
  const int t = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= B * S) return;
  const int b = t / S, pos = positions[b] + t % S, pj = pos / kPage;
  int page = -1;
  if (pos >= 0 && pj < max_pages) page = page_table[static_cast<size_t>(b) * max_pages + pj];
  if (page < 0 || page >= num_pages) {
    if (lane == 0) set_status(dev_status, TRANSMLA_DEV_BAD_PAGE);
    return;
  }
  const float* row = rows + static_cast<size_t>(t) * 576;
  float c[16];
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float4 v = *reinterpret_cast<const float4*>(row + lane * 16 + i * 4);
    c[4 * i] = v.x; c[4 * i + 1] = v.y; c[4 * i + 2] = v.z; c[4 * i + 3] = v.w;
    amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float scale = amax > 0.f ? amax / 448.f : 1.f;
  uint32_t codes[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint16_t lo, hi;
    asm volatile("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(c[4 * i + 1] / scale), "f"(c[4 * i] / scale));
    asm volatile("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(c[4 * i + 3] / scale), "f"(c[4 * i + 2] / scale));
    codes[i] = static_cast<uint32_t>(lo) | (static_cast<uint32_t>(hi) << 16);
  }
  unsigned char* dst = cache + (static_cast<size_t>(page) * kPage + pos % kPage) * TRANSMLA_FP8_ROW_BYTES;
  *reinterpret_cast<uint4*>(dst + lane * 16) = make_uint4(codes[0], codes[1], codes[2], codes[3]);
  const float2 kr = *reinterpret_cast<const float2*>(row + 512 + lane * 2);
  *reinterpret_cast<uint32_t*>(dst + 512 + lane * 4) = pack_bf16(kr.x / scale, kr.y / scale);
  if (lane < 4) *reinterpret_cast<uint32_t*>(dst + 640 + lane * 4) = lane == 0 ? __float_as_uint(scale) : 0u;
}

cudaError_t launch_append_fp8(const transmla_params_t& p, const __nv_bfloat16* x, const __nv_bfloat16* w, const int32_t* positions,
                              const int32_t* page_table, void* cache_fp8, float* scratch, int32_t* dev_status,
                              cudaStream_t stream) {
  const int K = p.kv_lora_rank + p.qk_rope_dim, T = p.batch * p.q_len;
  cudaError_t e = launch_pdl(append_rows_f32_kernel, dim3(K / 8), dim3(256), kAppendSmem, stream, x, w, positions, scratch, p.batch,
                             p.q_len, p.hidden_dim, p.kv_lora_rank, p.qk_rope_dim, p.rope_theta);
  if (e != cudaSuccess) return e;
  return launch_pdl(quantize_rows_kernel, dim3((T + 3) / 4), dim3(128), static_cast<size_t>(0), stream,
                    static_cast<const float*>(scratch), positions, page_table, static_cast<unsigned char*>(cache_fp8), dev_status,
                    p.batch, p.q_len, p.num_pages, p.max_pages_per_seq);
}

}  // namespace transmla
