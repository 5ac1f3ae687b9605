// Plan, absorb, append and combine kernels of the absorbed-MLA decode step.
//
// These four touch a few MB (weights, queries, split partials) against the hundreds of MB the
// split-KV kernel streams, so they are written for low launch latency and coalesced access rather
// than tensor cores.
#include "common.cuh"

namespace transmla {

// ------------------------------------------------------------------------------------------------
// Split plan.  cum[b] = sum_{b'<b} ceil(L_b'/P); partition i owns flat pages
// [floor(i*T/G), floor((i+1)*T/G)); plan row = (begin, end, sequence of first page, of last page).
// One block; the scan runs in chunks of blockDim.x sequences.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int seq_of_page(const int32_t* cum, int B, int x) {
  // largest b in [0, B) with cum[b] <= x < cum[b+1]  ==  (first index with cum > x) - 1
  int lo = 0, hi = B + 1;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (cum[mid] > x) hi = mid; else lo = mid + 1;
  }
  return lo - 1;
}

__global__ void __launch_bounds__(1024) plan_kernel(const int32_t* __restrict__ seqlens, int B, int G,
                                                     int32_t* __restrict__ cum, int32_t* __restrict__ plan) {
  __shared__ int warp_sums[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; cum[0] = 0; }
  __syncthreads();
  for (int base = 0; base < B; base += blockDim.x) {
    const int b = base + tid;
    int n = 0;
    if (b < B) { int L = seqlens[b]; n = L > 0 ? (L + kPage - 1) / kPage : 0; }
    int v = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += t; }
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sums[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += t; }
      warp_sums[lane] = w;
    }
    __syncthreads();
    const int incl = v + (warp > 0 ? warp_sums[warp - 1] : 0) + carry;
    if (b < B) cum[b + 1] = incl;
    __syncthreads();
    if (tid == blockDim.x - 1) carry = incl;
    __syncthreads();
  }
  const long long T = cum[B];
  for (int i = tid; i < G; i += blockDim.x) {
    const int p0 = static_cast<int>((static_cast<long long>(i) * T) / G);
    const int p1 = static_cast<int>((static_cast<long long>(i + 1) * T) / G);
    int b0 = -1, b1 = -1;
    if (p1 > p0) { b0 = seq_of_page(cum, B, p0); b1 = seq_of_page(cum, B, p1 - 1); }
    reinterpret_cast<int4*>(plan)[i] = make_int4(p0, p1, b0, b1);
  }
}

cudaError_t launch_plan(const int32_t* seqlens, int B, int G, int32_t* cum, int32_t* plan, cudaStream_t stream) {
  plan_kernel<<<1, 1024, 0, stream>>>(seqlens, B, G, cum, plan);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Absorb (Eq. 9 right, first line): q_hat[bs,h,:r] = W_UK_h^T q_nope[bs,h,:], q_hat[bs,h,r:] = q_pe[bs,h,:].
// grid (H, ceil(BS/8), ceil(r/128)), 128 threads; thread n owns one latent column for 8 query rows.
// ------------------------------------------------------------------------------------------------
constexpr int kAbsorbRows = 8;

__global__ void __launch_bounds__(128) absorb_kernel(const __nv_bfloat16* __restrict__ q_nope,
                                                     const __nv_bfloat16* __restrict__ q_pe,
                                                     const __nv_bfloat16* __restrict__ w_uk,
                                                     __nv_bfloat16* __restrict__ q_hat, int BS, int H, int dn, int dR,
                                                     int r) {
  extern __shared__ float q_s[];  // [kAbsorbRows][dn]
  const int h = blockIdx.x, row0 = blockIdx.y * kAbsorbRows, n = blockIdx.z * 128 + threadIdx.x;
  for (int i = threadIdx.x; i < kAbsorbRows * dn; i += 128) {
    const int rr = row0 + i / dn;
    q_s[i] = rr < BS ? __bfloat162float(q_nope[(static_cast<size_t>(rr) * H + h) * dn + i % dn]) : 0.f;
  }
  __syncthreads();
  const int K = r + dR;
  if (n < r) {
    float acc[kAbsorbRows];
#pragma unroll
    for (int i = 0; i < kAbsorbRows; ++i) acc[i] = 0.f;
    const __nv_bfloat16* w = w_uk + static_cast<size_t>(h) * dn * r + n;
    for (int k = 0; k < dn; ++k) {
      const float wv = __bfloat162float(w[static_cast<size_t>(k) * r]);
#pragma unroll
      for (int i = 0; i < kAbsorbRows; ++i) acc[i] = fmaf(q_s[i * dn + k], wv, acc[i]);
    }
#pragma unroll
    for (int i = 0; i < kAbsorbRows; ++i)
      if (row0 + i < BS) q_hat[(static_cast<size_t>(row0 + i) * H + h) * K + n] = __float2bfloat16_rn(acc[i]);
  }
  if (blockIdx.z == 0) {
    for (int i = threadIdx.x; i < kAbsorbRows * dR; i += 128) {
      const int rr = row0 + i / dR, c = i % dR;
      if (rr < BS) q_hat[(static_cast<size_t>(rr) * H + h) * K + r + c] = q_pe[(static_cast<size_t>(rr) * H + h) * dR + c];
    }
  }
}

cudaError_t launch_absorb(const transmla_params_t& p, const __nv_bfloat16* q_nope, const __nv_bfloat16* q_pe,
                          const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat, cudaStream_t stream) {
  const int BS = p.batch * p.q_len;
  dim3 grid(p.num_heads, (BS + kAbsorbRows - 1) / kAbsorbRows, (p.kv_lora_rank + 127) / 128);
  absorb_kernel<<<grid, 128, kAbsorbRows * p.qk_nope_dim * sizeof(float), stream>>>(
      q_nope, q_pe, w_uk, q_hat, BS, p.num_heads, p.qk_nope_dim, p.qk_rope_dim, p.kv_lora_rank);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Latent append (Eq. 7 left): y = [W_DKV; W_KR] x, RoPE (Eq. 1) on y[r:], bf16, scatter to the page slot.
// One block owns 8 consecutive output features (so a RoPE pair never straddles blocks) and keeps
// their weight rows in shared memory; each warp walks tokens.
// ------------------------------------------------------------------------------------------------
constexpr int kAppendFeat = 8;

__global__ void __launch_bounds__(256) append_kernel(const __nv_bfloat16* __restrict__ x,
                                                     const __nv_bfloat16* __restrict__ w,
                                                     const int32_t* __restrict__ positions,
                                                     const int32_t* __restrict__ page_table,
                                                     __nv_bfloat16* __restrict__ cache, int32_t* dev_status, int B,
                                                     int S, int D, int r, int dR, int num_pages, int max_pages,
                                                     float theta) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* w_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [8][D]
  const int K = r + dR, f0 = blockIdx.x * kAppendFeat;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunks = D / 8;  // 16-byte chunks per row
  for (int i = threadIdx.x; i < kAppendFeat * chunks; i += 256) {
    const int f = i / chunks, c = i % chunks;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (f0 + f < K) v = *reinterpret_cast<const uint4*>(w + static_cast<size_t>(f0 + f) * D + c * 8);
    *reinterpret_cast<uint4*>(w_s + static_cast<size_t>(f) * D + c * 8) = v;
  }
  __syncthreads();
  for (int t = warp; t < B * S; t += 8) {
    float acc[kAppendFeat];
#pragma unroll
    for (int f = 0; f < kAppendFeat; ++f) acc[f] = 0.f;
    const __nv_bfloat16* xr = x + static_cast<size_t>(t) * D;
    for (int c = lane; c < chunks; c += 32) {
      const uint4 xv = *reinterpret_cast<const uint4*>(xr + c * 8);
      const uint32_t xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
      for (int f = 0; f < kAppendFeat; ++f) {
        const uint4 wv = *reinterpret_cast<const uint4*>(w_s + static_cast<size_t>(f) * D + c * 8);
        const uint32_t ws[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[f] = fmaf(bf16_lo(xs[j]), bf16_lo(ws[j]), acc[f]);
          acc[f] = fmaf(bf16_hi(xs[j]), bf16_hi(ws[j]), acc[f]);
        }
      }
    }
#pragma unroll
    for (int f = 0; f < kAppendFeat; ++f)
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[f] += __shfl_xor_sync(0xffffffffu, acc[f], o);
    if (lane == 0) {
      const int b = t / S, s = t % S;
      const int pos = positions[b] + s;
      const int pj = pos / kPage;
      int page = -1;
      if (pos >= 0 && pj < max_pages) page = page_table[static_cast<size_t>(b) * max_pages + pj];
      if (page < 0 || page >= num_pages) {
        set_status(dev_status, TRANSMLA_DEV_BAD_PAGE);
      } else {
        if (f0 >= r) {  // RoPE pairs (2l, 2l+1) of the rope part; angle in fp64 so that long positions stay exact
#pragma unroll
          for (int f = 0; f < kAppendFeat; f += 2) {
            const int l = (f0 + f - r) / 2;
            const double ang = static_cast<double>(pos) * pow(static_cast<double>(theta), -2.0 * l / dR);
            double sn, cs;
            sincos(ang, &sn, &cs);
            const float re = acc[f], im = acc[f + 1];
            acc[f] = static_cast<float>(re * cs - im * sn);
            acc[f + 1] = static_cast<float>(im * cs + re * sn);
          }
        }
        uint4 o;
        o.x = pack_bf16(acc[0], acc[1]); o.y = pack_bf16(acc[2], acc[3]);
        o.z = pack_bf16(acc[4], acc[5]); o.w = pack_bf16(acc[6], acc[7]);
        *reinterpret_cast<uint4*>(cache + (static_cast<size_t>(page) * kPage + pos % kPage) * K + f0) = o;
      }
    }
  }
}

cudaError_t launch_append(const transmla_params_t& p, const __nv_bfloat16* x, const __nv_bfloat16* w,
                          const int32_t* positions, const int32_t* page_table, __nv_bfloat16* cache,
                          int32_t* dev_status, cudaStream_t stream) {
  const int K = p.kv_lora_rank + p.qk_rope_dim;
  const size_t smem = static_cast<size_t>(kAppendFeat) * p.hidden_dim * sizeof(__nv_bfloat16);
  cudaError_t e = cudaFuncSetAttribute(append_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  append_kernel<<<K / kAppendFeat, 256, smem, stream>>>(x, w, positions, page_table, cache, dev_status, p.batch,
                                                        p.q_len, p.hidden_dim, p.kv_lora_rank, p.qk_rope_dim,
                                                        p.num_pages, p.max_pages_per_seq, p.rope_theta);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Combine + up-projection (Eq. 9 right, last line before W_O).  Block = one head, 4 query rows.
// Segments of sequence b live in slots i + b for the partitions i that overlap its pages.
// ------------------------------------------------------------------------------------------------
constexpr int kCombineRows = 4;

__global__ void __launch_bounds__(128) combine_kernel(const int32_t* __restrict__ cum,
                                                      const float* __restrict__ partial_o,
                                                      const float* __restrict__ partial_lse,
                                                      const __nv_bfloat16* __restrict__ w_uv,
                                                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse_out,
                                                      int B, int S, int H, int r, int dv, int G) {
  extern __shared__ float o_s[];  // [kCombineRows][r]
  const int h = blockIdx.x, bs0 = blockIdx.y * kCombineRows;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int SH = S * H;
  const long long T = cum[B];
  for (int i = 0; i < kCombineRows; ++i) {
    const int bs = bs0 + i;
    float* o_row = o_s + i * r;
    for (int k = tid; k < r; k += 128) o_row[k] = 0.f;
    if (bs >= B * S) continue;
    const int b = bs / S, s = bs % S, row = s * H + h;
    const int c0 = cum[b], c1 = cum[b + 1];
    float lse = -INFINITY;
    if (c1 > c0) {
      const int i_first = static_cast<int>(((static_cast<long long>(c0) + 1) * G - 1) / T);
      const int i_last = static_cast<int>((static_cast<long long>(c1) * G - 1) / T);
      float m = -INFINITY;
      for (int pi = i_first; pi <= i_last; ++pi) {
        const long long p0 = (static_cast<long long>(pi) * T) / G, p1 = (static_cast<long long>(pi + 1) * T) / G;
        if (p1 > p0) m = fmaxf(m, partial_lse[static_cast<size_t>(pi + b) * SH + row]);
      }
      if (m > -INFINITY) {
        float den = 0.f;
        for (int pi = i_first; pi <= i_last; ++pi) {
          const long long p0 = (static_cast<long long>(pi) * T) / G, p1 = (static_cast<long long>(pi + 1) * T) / G;
          if (p1 <= p0) continue;
          const float l = partial_lse[static_cast<size_t>(pi + b) * SH + row];
          if (l == -INFINITY) continue;
          const float wgt = __expf(l - m);
          den += wgt;
          const float* po = partial_o + (static_cast<size_t>(pi + b) * SH + row) * r;
          for (int k = tid; k < r; k += 128) o_row[k] = fmaf(wgt, po[k], o_row[k]);
        }
        const float inv = 1.f / den;
        for (int k = tid; k < r; k += 128) o_row[k] *= inv;
        lse = m + __logf(den);
      }
    }
    if (lse_out != nullptr && tid == 0) lse_out[(static_cast<size_t>(b) * S + s) * H + h] = lse;
  }
  __syncthreads();
  const __nv_bfloat16* w_h = w_uv + static_cast<size_t>(h) * dv * r;
  for (int v = warp; v < dv; v += 4) {
    float acc[kCombineRows];
#pragma unroll
    for (int i = 0; i < kCombineRows; ++i) acc[i] = 0.f;
    for (int k = lane * 8; k < r; k += 256) {
      const uint4 wv = *reinterpret_cast<const uint4*>(w_h + static_cast<size_t>(v) * r + k);
      const uint32_t ws[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int i = 0; i < kCombineRows; ++i) {
        const float* o_row = o_s + i * r + k;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i] = fmaf(bf16_lo(ws[j]), o_row[2 * j], acc[i]);
          acc[i] = fmaf(bf16_hi(ws[j]), o_row[2 * j + 1], acc[i]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < kCombineRows; ++i)
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < kCombineRows; ++i) {
        const int bs = bs0 + i;
        if (bs < B * S) out[(static_cast<size_t>(bs) * H + h) * dv + v] = __float2bfloat16_rn(acc[i]);
      }
    }
  }
}

cudaError_t launch_combine(const transmla_params_t& p, int G, const int32_t* cum, const float* partial_o,
                           const float* partial_lse, const __nv_bfloat16* w_uv, __nv_bfloat16* out, float* lse_out,
                           cudaStream_t stream) {
  const int BS = p.batch * p.q_len;
  dim3 grid(p.num_heads, (BS + kCombineRows - 1) / kCombineRows);
  combine_kernel<<<grid, 128, kCombineRows * p.kv_lora_rank * sizeof(float), stream>>>(
      cum, partial_o, partial_lse, w_uv, out, lse_out, p.batch, p.q_len, p.num_heads, p.kv_lora_rank, p.v_dim, G);
  return cudaGetLastError();
}

}  // namespace transmla
