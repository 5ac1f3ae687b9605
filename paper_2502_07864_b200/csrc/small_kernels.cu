// Plan, absorb, append and combine kernels of the absorbed-MLA decode step.
//
// These touch a few MB (weights, queries, split partials) against the hundreds of MB the split-KV
// kernel streams.  They are small GEMMs with M = number of query rows or new tokens, so they run on
// mma.sync tensor-core tiles with operands read straight from global memory or L2, and they are
// fused into as few launches as the data dependencies allow: one "prologue" launch holds the append
// blocks, the absorb blocks and the plan block.
#include "common.cuh"

namespace transmla {

__device__ __forceinline__ uint32_t ld_u32(const __nv_bfloat16* p) { return *reinterpret_cast<const uint32_t*>(p); }

// ------------------------------------------------------------------------------------------------
// Split plan.  cum[b] = sum_{b'<b} ceil(L_b'/P); partition i owns flat pages
// [floor(i*T/G), floor((i+1)*T/G)); plan row = (begin, end, sequence of first page, of last page).
// One block of 256 threads; the scan runs in chunks of 256 sequences.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int seq_of_page(const int32_t* cum, int B, int x) {
  // the b in [0, B) with cum[b] <= x < cum[b+1]  ==  (first index with cum > x) - 1
  int lo = 0, hi = B + 1;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (cum[mid] > x) hi = mid; else lo = mid + 1;
  }
  return lo - 1;
}

__device__ void plan_block(const int32_t* __restrict__ seqlens, int B, int G, int32_t* cum, int32_t* plan) {
  __shared__ int warp_sums[8];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; cum[0] = 0; }
  __syncthreads();
  for (int base = 0; base < B; base += 256) {
    const int b = base + tid;
    int n = 0;
    if (b < B) { int L = seqlens[b]; n = L > 0 ? (L + kPage - 1) / kPage : 0; }
    int v = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += t; }
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    const int incl = v + before;
    if (b < B) cum[b + 1] = incl;
    __syncthreads();
    if (tid == 255) carry = incl;
    __syncthreads();
  }
  const long long T = cum[B];
  for (int i = tid; i < G; i += 256) {
    const int p0 = static_cast<int>((static_cast<long long>(i) * T) / G);
    const int p1 = static_cast<int>((static_cast<long long>(i + 1) * T) / G);
    int b0 = -1, b1 = -1;
    if (p1 > p0) { b0 = seq_of_page(cum, B, p0); b1 = seq_of_page(cum, B, p1 - 1); }
    reinterpret_cast<int4*>(plan)[i] = make_int4(p0, p1, b0, b1);
  }
}

// ------------------------------------------------------------------------------------------------
// Absorb (Eq. 9 right, first line): q_hat[bs,h,:r] = W_UK_h^T q_nope[bs,h,:], q_hat[bs,h,r:] = q_pe[bs,h,:].
// Block (h, rt) owns 128 latent columns of one head: it stages W_UK_h[:, tile] in shared memory once
// and walks all query rows in 16-row tiles, so W_UK is read once in total.
// ------------------------------------------------------------------------------------------------
constexpr int kAbsorbPitch = 128 + 8;

__device__ void absorb_block(const __nv_bfloat16* __restrict__ q_nope, const __nv_bfloat16* __restrict__ q_pe,
                             const __nv_bfloat16* __restrict__ w_uk, __nv_bfloat16* __restrict__ q_hat, int BS, int H,
                             int dn, int dR, int r, int h, int rt, unsigned char* smem_raw) {
  __nv_bfloat16* w_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [dn][kAbsorbPitch]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int n0 = rt * 128, K = r + dR;
  for (int i = tid; i < dn * 16; i += 256) {
    const int k = i >> 4, c = i & 15;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (n0 + c * 8 < r) v = *reinterpret_cast<const uint4*>(w_uk + (static_cast<size_t>(h) * dn + k) * r + n0 + c * 8);
    *reinterpret_cast<uint4*>(w_s + k * kAbsorbPitch + c * 8) = v;
  }
  __syncthreads();
  const int mi = lane >> 3;
  for (int m0 = 0; m0 < BS; m0 += 16) {
    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    const int r0 = m0 + g, r1 = m0 + g + 8;
    const __nv_bfloat16* q0 = q_nope + (static_cast<size_t>(min(r0, BS - 1)) * H + h) * dn + t4 * 2;
    const __nv_bfloat16* q1 = q_nope + (static_cast<size_t>(min(r1, BS - 1)) * H + h) * dn + t4 * 2;
#pragma unroll 4
    for (int ks = 0; ks < dn / 16; ++ks) {
      uint32_t a[4];
      a[0] = r0 < BS ? ld_u32(q0 + ks * 16) : 0u;
      a[1] = r1 < BS ? ld_u32(q1 + ks * 16) : 0u;
      a[2] = r0 < BS ? ld_u32(q0 + ks * 16 + 8) : 0u;
      a[3] = r1 < BS ? ld_u32(q1 + ks * 16 + 8) : 0u;
      uint32_t bf[4];
      ldmatrix_x4_trans(bf, w_s + (ks * 16 + (mi & 1) * 8 + (lane & 7)) * kAbsorbPitch + warp * 16 + (mi >> 1) * 8);
      mma_bf16_16816(acc[0], a, bf[0], bf[1]);
      mma_bf16_16816(acc[1], a, bf[2], bf[3]);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int col = n0 + warp * 16 + j * 8 + t4 * 2;
      if (col < r) {
        if (r0 < BS) *reinterpret_cast<uint32_t*>(q_hat + (static_cast<size_t>(r0) * H + h) * K + col) = pack_bf16(acc[j][0], acc[j][1]);
        if (r1 < BS) *reinterpret_cast<uint32_t*>(q_hat + (static_cast<size_t>(r1) * H + h) * K + col) = pack_bf16(acc[j][2], acc[j][3]);
      }
    }
  }
  if (rt == 0 && dR > 0) {
    const int pairs = dR / 2;
    for (int i = tid; i < BS * pairs; i += 256) {
      const int row = i / pairs, c = (i % pairs) * 2;
      *reinterpret_cast<uint32_t*>(q_hat + (static_cast<size_t>(row) * H + h) * K + r + c) =
          ld_u32(q_pe + (static_cast<size_t>(row) * H + h) * dR + c);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Latent append (Eq. 7 left): y = [W_DKV; W_KR] x, RoPE (Eq. 1) on y[r:], bf16, scatter to the page slot.
// One block owns 8 consecutive output features (a RoPE pair never straddles blocks); its 8 warps
// split the hidden dimension and meet in shared memory.  Tokens are the M dimension of the tiles.
// Token (b, s) sits at position pos_base[b] + pos_shift + s.
// ------------------------------------------------------------------------------------------------
constexpr int kAppendMT = 8;  // 16-token tiles per pass

__device__ void append_block(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                             const int32_t* __restrict__ pos_base, int pos_shift,
                             const int32_t* __restrict__ page_table, __nv_bfloat16* __restrict__ cache,
                             int32_t* dev_status, int B, int S, int D, int r, int dR, int num_pages, int max_pages,
                             float theta, int nb, unsigned char* smem_raw) {
  float* red = reinterpret_cast<float*>(smem_raw);  // [8 warps][kAppendMT*16 rows][8]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int K = r + dR, f0 = nb * 8, T = B * S;
  const int slice = D / 8, k_lo = warp * slice;
  const __nv_bfloat16* wrow = w + static_cast<size_t>(f0 + g) * D + k_lo + t4 * 2;
  for (int t0 = 0; t0 < T; t0 += kAppendMT * 16) {
    float acc[kAppendMT][4];
#pragma unroll
    for (int mt = 0; mt < kAppendMT; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;
#pragma unroll 2
    for (int k = 0; k < slice; k += 16) {
      const uint32_t b0 = ld_u32(wrow + k), b1 = ld_u32(wrow + k + 8);
#pragma unroll
      for (int mt = 0; mt < kAppendMT; ++mt) {
        if (t0 + mt * 16 < T) {
          const int r0 = t0 + mt * 16 + g, r1 = r0 + 8;
          const __nv_bfloat16* x0 = x + static_cast<size_t>(min(r0, T - 1)) * D + k_lo + k + t4 * 2;
          const __nv_bfloat16* x1 = x + static_cast<size_t>(min(r1, T - 1)) * D + k_lo + k + t4 * 2;
          uint32_t a[4];
          a[0] = r0 < T ? ld_u32(x0) : 0u;
          a[1] = r1 < T ? ld_u32(x1) : 0u;
          a[2] = r0 < T ? ld_u32(x0 + 8) : 0u;
          a[3] = r1 < T ? ld_u32(x1 + 8) : 0u;
          mma_bf16_16816(acc[mt], a, b0, b1);
        }
      }
    }
    __syncthreads();  // previous pass has consumed `red`
#pragma unroll
    for (int mt = 0; mt < kAppendMT; ++mt) {
      if (t0 + mt * 16 < T) {
        float* d = red + (warp * kAppendMT * 16 + mt * 16 + g) * 8 + t4 * 2;
        *reinterpret_cast<float2*>(d) = make_float2(acc[mt][0], acc[mt][1]);
        *reinterpret_cast<float2*>(d + 64) = make_float2(acc[mt][2], acc[mt][3]);
      }
    }
    __syncthreads();
    const int rows = min(kAppendMT * 16, T - t0);
    for (int i = tid; i < rows * 4; i += 256) {
      const int row = i >> 2, pr = i & 3;
      float re = 0.f, im = 0.f;
#pragma unroll
      for (int wv = 0; wv < 8; ++wv) {
        const float2 v = *reinterpret_cast<const float2*>(red + (wv * kAppendMT * 16 + row) * 8 + pr * 2);
        re += v.x; im += v.y;
      }
      const int t = t0 + row, b = t / S, s = t % S;
      const int pos = pos_base[b] + pos_shift + s;
      const int pj = pos / kPage;
      int page = -1;
      if (pos >= 0 && pj < max_pages) page = page_table[static_cast<size_t>(b) * max_pages + pj];
      if (page < 0 || page >= num_pages) {
        set_status(dev_status, TRANSMLA_DEV_BAD_PAGE);
        continue;
      }
      const int f = f0 + pr * 2;
      if (f >= r) {
        // RoPE pair l (Eq. 1).  The angle is formed and reduced to [-pi, pi] in fp64 so that positions of
        // 10^5 keep their phase; the sine and cosine of the reduced angle are fp32.
        const int l = (f - r) >> 1;
        const double ang = static_cast<double>(pos) * exp2(-2.0 * l / dR * log2(static_cast<double>(theta)));
        const double red_ang = ang - 6.283185307179586476925 * rint(ang * 0.15915494309189533577);
        float sn, cs;
        sincosf(static_cast<float>(red_ang), &sn, &cs);
        const float nre = re * cs - im * sn, nim = im * cs + re * sn;
        re = nre; im = nim;
      }
      *reinterpret_cast<uint32_t*>(cache + (static_cast<size_t>(page) * kPage + pos % kPage) * K + f) = pack_bf16(re, im);
    }
  }
}

constexpr size_t kAppendSmem = 8 * kAppendMT * 16 * 8 * sizeof(float);  // 32 KB

__global__ void __launch_bounds__(256) append_kernel(const __nv_bfloat16* __restrict__ x,
                                                     const __nv_bfloat16* __restrict__ w,
                                                     const int32_t* __restrict__ positions,
                                                     const int32_t* __restrict__ page_table,
                                                     __nv_bfloat16* __restrict__ cache, int32_t* dev_status, int B,
                                                     int S, int D, int r, int dR, int num_pages, int max_pages,
                                                     float theta) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  append_block(x, w, positions, 0, page_table, cache, dev_status, B, S, D, r, dR, num_pages, max_pages, theta,
               blockIdx.x, smem_raw);
}

// Absorb blocks followed by one plan block: everything transmla_mla_decode needs before the split-KV kernel.
__global__ void __launch_bounds__(256) absorb_plan_kernel(const __nv_bfloat16* __restrict__ q_nope,
                                                          const __nv_bfloat16* __restrict__ q_pe,
                                                          const __nv_bfloat16* __restrict__ w_uk,
                                                          __nv_bfloat16* __restrict__ q_hat,
                                                          const int32_t* __restrict__ seqlens, int32_t* cum,
                                                          int32_t* plan, int B, int S, int H, int dn, int dR, int r,
                                                          int G) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int r_tiles = (r + 127) / 128;
  const int n_absorb = H * r_tiles;
  if (static_cast<int>(blockIdx.x) < n_absorb) {
    absorb_block(q_nope, q_pe, w_uk, q_hat, B * S, H, dn, dR, r, blockIdx.x / r_tiles, blockIdx.x % r_tiles, smem_raw);
  } else {
    plan_block(seqlens, B, G, cum, plan);
  }
}

// The whole prologue of a decode step in one launch: append blocks, absorb blocks, plan block.
// The appended token of sequence b sits at seqlens[b] - S + s.
__global__ void __launch_bounds__(256) prologue_kernel(
    const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w_dkv_kr,
    const int32_t* __restrict__ page_table, __nv_bfloat16* __restrict__ cache, const __nv_bfloat16* __restrict__ q_nope,
    const __nv_bfloat16* __restrict__ q_pe, const __nv_bfloat16* __restrict__ w_uk, __nv_bfloat16* __restrict__ q_hat,
    const int32_t* __restrict__ seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status, int B, int S, int H, int D,
    int dn, int dR, int r, int num_pages, int max_pages, float theta, int G) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_append = (r + dR) / 8;
  const int r_tiles = (r + 127) / 128;
  const int n_absorb = H * r_tiles;
  const int bid = blockIdx.x;
  if (bid < n_append) {
    append_block(x, w_dkv_kr, seqlens, -S, page_table, cache, dev_status, B, S, D, r, dR, num_pages, max_pages, theta,
                 bid, smem_raw);
  } else if (bid < n_append + n_absorb) {
    const int a = bid - n_append;
    absorb_block(q_nope, q_pe, w_uk, q_hat, B * S, H, dn, dR, r, a / r_tiles, a % r_tiles, smem_raw);
  } else {
    plan_block(seqlens, B, G, cum, plan);
  }
}

static size_t absorb_smem(int dn) { return static_cast<size_t>(dn) * kAbsorbPitch * sizeof(__nv_bfloat16); }

cudaError_t launch_append(const transmla_params_t& p, const __nv_bfloat16* x, const __nv_bfloat16* w,
                          const int32_t* positions, const int32_t* page_table, __nv_bfloat16* cache,
                          int32_t* dev_status, cudaStream_t stream) {
  const int K = p.kv_lora_rank + p.qk_rope_dim;
  append_kernel<<<K / 8, 256, kAppendSmem, stream>>>(x, w, positions, page_table, cache, dev_status, p.batch, p.q_len,
                                                     p.hidden_dim, p.kv_lora_rank, p.qk_rope_dim, p.num_pages,
                                                     p.max_pages_per_seq, p.rope_theta);
  return cudaGetLastError();
}

cudaError_t launch_absorb_plan(const transmla_params_t& p, int G, const __nv_bfloat16* q_nope,
                               const __nv_bfloat16* q_pe, const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat,
                               const int32_t* seqlens, int32_t* cum, int32_t* plan, cudaStream_t stream) {
  const size_t smem = absorb_smem(p.qk_nope_dim);
  static bool attr_set = false;  // 68 KB at dn = 256 exceeds the default dynamic shared memory limit
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(absorb_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 72 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int blocks = p.num_heads * ((p.kv_lora_rank + 127) / 128) + 1;
  absorb_plan_kernel<<<blocks, 256, smem, stream>>>(q_nope, q_pe, w_uk, q_hat, seqlens, cum, plan, p.batch, p.q_len,
                                                    p.num_heads, p.qk_nope_dim, p.qk_rope_dim, p.kv_lora_rank, G);
  return cudaGetLastError();
}

cudaError_t launch_prologue(const transmla_params_t& p, int G, const __nv_bfloat16* x, const __nv_bfloat16* w_dkv_kr,
                            const int32_t* page_table, __nv_bfloat16* cache, const __nv_bfloat16* q_nope,
                            const __nv_bfloat16* q_pe, const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat,
                            const int32_t* seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status,
                            cudaStream_t stream) {
  size_t smem = absorb_smem(p.qk_nope_dim);
  if (smem < kAppendSmem) smem = kAppendSmem;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(prologue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 72 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int blocks = (p.kv_lora_rank + p.qk_rope_dim) / 8 + p.num_heads * ((p.kv_lora_rank + 127) / 128) + 1;
  prologue_kernel<<<blocks, 256, smem, stream>>>(x, w_dkv_kr, page_table, cache, q_nope, q_pe, w_uk, q_hat, seqlens, cum,
                                                 plan, dev_status, p.batch, p.q_len, p.num_heads, p.hidden_dim,
                                                 p.qk_nope_dim, p.qk_rope_dim, p.kv_lora_rank, p.num_pages,
                                                 p.max_pages_per_seq, p.rope_theta, G);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Combine + up-projection (Eq. 9 right, last line before W_O).  Block = one head x 16 query rows.
// Phase 1: each warp merges the split partials of two rows by their lse (segments of sequence b live
// in slots i + b for the partitions i that overlap its pages) into shared memory as a bf16 hi/lo
// pair, so that the tensor-core product of phase 2 carries fp32-like precision of o_hat.
// Phase 2: out[rows, h, :] = o_hat W_UV_h^T with W_UV_h read straight from global memory.
// ------------------------------------------------------------------------------------------------
constexpr int kCombineRows = 16;

__global__ void __launch_bounds__(256) combine_kernel(const int32_t* __restrict__ cum,
                                                      const float* __restrict__ partial_o,
                                                      const float* __restrict__ partial_lse,
                                                      const __nv_bfloat16* __restrict__ w_uv,
                                                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse_out,
                                                      int B, int S, int H, int r, int dv, int G, int rows_per_block) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch = r + 8;
  __nv_bfloat16* o_hi = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [16][pitch]
  __nv_bfloat16* o_lo = o_hi + kCombineRows * pitch;                 // [16][pitch]
  const int h = blockIdx.x, bs0 = blockIdx.y * rows_per_block;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int SH = S * H, BS = B * S;
  const long long T = cum[B];

  for (int rr = warp; rr < kCombineRows; rr += 8) {
    const int bs = bs0 + rr;
    float acc[4][4];
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.f;
    float lse = -INFINITY, inv = 0.f;
    if (rr < rows_per_block && bs < BS) {
      const int b = bs / S, s = bs % S, row = s * H + h;
      const int c0 = cum[b], c1 = cum[b + 1];
      if (c1 > c0) {
        const int i_first = static_cast<int>(((static_cast<long long>(c0) + 1) * G - 1) / T);
        const int i_last = static_cast<int>((static_cast<long long>(c1) * G - 1) / T);
        const int nseg = i_last - i_first + 1;
        auto seg_lse = [&](int j) -> float {  // lse of the j-th candidate partition, -inf if it is empty or absent
          if (j >= nseg) return -INFINITY;
          const int pi = i_first + j;
          const long long p0 = (static_cast<long long>(pi) * T) / G, p1 = (static_cast<long long>(pi + 1) * T) / G;
          return p1 > p0 ? partial_lse[static_cast<size_t>(pi + b) * SH + row] : -INFINITY;
        };
        float m = -INFINITY;
        for (int base = 0; base < nseg; base += 32) m = fmaxf(m, seg_lse(base + lane));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (m > -INFINITY) {
          float den = 0.f;
          for (int base = 0; base < nseg; base += 32) {
            const float l = seg_lse(base + lane);
            const float wgt = l > -INFINITY ? __expf(l - m) : 0.f;
            den += wgt;
            const int cnt = min(32, nseg - base);
            for (int j = 0; j < cnt; ++j) {
              const float wj = __shfl_sync(0xffffffffu, wgt, j);
              if (wj == 0.f) continue;
              const float* po = partial_o + (static_cast<size_t>(i_first + base + j + b) * SH + row) * r;
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const int k = c * 128 + lane * 4;
                if (k < r) {
                  const float4 v = *reinterpret_cast<const float4*>(po + k);
                  acc[c][0] = fmaf(wj, v.x, acc[c][0]); acc[c][1] = fmaf(wj, v.y, acc[c][1]);
                  acc[c][2] = fmaf(wj, v.z, acc[c][2]); acc[c][3] = fmaf(wj, v.w, acc[c][3]);
                }
              }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
          inv = 1.f / den;
          lse = m + __logf(den);
        }
      }
      if (lse_out != nullptr && lane == 0) lse_out[(static_cast<size_t>(b) * S + s) * H + h] = lse;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int k = c * 128 + lane * 4;
      if (k < r) {
        float v[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          v[e] = acc[c][e] * inv;
          lo[e] = v[e] - __bfloat162float(__float2bfloat16_rn(v[e]));
        }
        *reinterpret_cast<uint2*>(o_hi + rr * pitch + k) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
        *reinterpret_cast<uint2*>(o_lo + rr * pitch + k) = make_uint2(pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]));
      }
    }
  }
  __syncthreads();

  const int g = lane >> 2, t4 = lane & 3, mi = lane >> 3;
  for (int nt = warp; nt < dv / 8; nt += 8) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const __nv_bfloat16* wrow = w_uv + (static_cast<size_t>(h) * dv + nt * 8 + g) * r + t4 * 2;
#pragma unroll 4
    for (int ks = 0; ks < r / 16; ++ks) {
      const uint32_t b0 = ld_u32(wrow + ks * 16), b1 = ld_u32(wrow + ks * 16 + 8);
      uint32_t ah[4], al[4];
      const int off = ((mi & 1) * 8 + (lane & 7)) * pitch + ks * 16 + (mi >> 1) * 8;
      ldmatrix_x4(ah, o_hi + off);
      ldmatrix_x4(al, o_lo + off);
      mma_bf16_16816(acc, ah, b0, b1);
      mma_bf16_16816(acc, al, b0, b1);
    }
    const int col = nt * 8 + t4 * 2;
    const int bs_a = bs0 + g, bs_b = bs0 + g + 8;
    if (g < rows_per_block && bs_a < BS)
      *reinterpret_cast<uint32_t*>(out + (static_cast<size_t>(bs_a) * H + h) * dv + col) = pack_bf16(acc[0], acc[1]);
    if (g + 8 < rows_per_block && bs_b < BS)
      *reinterpret_cast<uint32_t*>(out + (static_cast<size_t>(bs_b) * H + h) * dv + col) = pack_bf16(acc[2], acc[3]);
  }
}

cudaError_t launch_combine(const transmla_params_t& p, int G, const int32_t* cum, const float* partial_o,
                           const float* partial_lse, const __nv_bfloat16* w_uv, __nv_bfloat16* out, float* lse_out,
                           cudaStream_t stream) {
  const int BS = p.batch * p.q_len;
  const int rows = BS <= 64 ? 8 : 16;  // smaller blocks when there are few query rows, for more parallelism
  dim3 grid(p.num_heads, (BS + rows - 1) / rows);
  const size_t smem = 2 * kCombineRows * (p.kv_lora_rank + 8) * sizeof(__nv_bfloat16);
  combine_kernel<<<grid, 256, smem, stream>>>(cum, partial_o, partial_lse, w_uv, out, lse_out, p.batch, p.q_len,
                                              p.num_heads, p.kv_lora_rank, p.v_dim, G, rows);
  return cudaGetLastError();
}

}  // namespace transmla
