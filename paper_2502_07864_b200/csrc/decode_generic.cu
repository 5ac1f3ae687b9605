// Split-KV absorbed-MLA decode (Eq. 9 right, second line), register-accumulator version.
//
// One CTA = one (partition, block of 32 query rows).  It walks the partition's segments; for each
// 64-token page it stages the page in shared memory once (cp.async, double buffered) and uses the
// same tile for both contractions: S = Q_hat K_hat^T over all r+dR columns and O += P C over the
// first r columns.  Works for every supported (r, dR); the TMA/tcgen05 kernel in decode_sm100.cu
// takes over for the production shape.
#include "common.cuh"

namespace transmla {

template <int R, int DR>
struct GenericCfg {
  static constexpr int K = R + DR;          // columns of a cache row
  static constexpr int KP = K + 8;          // padded shared-memory pitch (elements)
  static constexpr int KS = K / 16;         // k-steps of the QK^T contraction
  static constexpr int KSW = (KS + 3) / 4;  // k-steps per k-warp (4 k-warps)
  static constexpr int NT = R / 64;         // 8-column output tiles per warp (8 warps share r columns)
  static constexpr int SP = kPage + 4;      // pitch of the fp32 score partials
  static constexpr int PP = kPage + 8;      // pitch of the bf16 probabilities
  static constexpr size_t smem_bytes = sizeof(__nv_bfloat16) * (2 * kPage * KP + kRowBlock * KP + kRowBlock * PP) +
                                       sizeof(float) * (4 * kRowBlock * SP + 3 * kRowBlock);
  static_assert(K % 16 == 0 && R % 64 == 0, "unsupported latent shape");
};

template <int R, int DR>
__global__ void __launch_bounds__(256, 1)
decode_generic_kernel(const __nv_bfloat16* q_hat, const __nv_bfloat16* cache,
                      const int32_t* page_table, const int32_t* seqlens,
                      const int32_t* cum, const int32_t* plan,
                      float* partial_o, float* partial_lse, int32_t* dev_status, int S, int H,
                      int num_pages, int max_pages, float scale_log2) {
  using C = GenericCfg<R, DR>;
  constexpr int K = C::K, KP = C::KP, KSW = C::KSW, NT = C::NT, SP = C::SP, PP = C::PP;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* page_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);        // [2][64][KP]
  __nv_bfloat16* q_s = page_s + 2 * kPage * KP;                              // [32][KP]
  __nv_bfloat16* p_s = q_s + kRowBlock * KP;                                 // [32][PP]
  float* s_s = reinterpret_cast<float*>(p_s + kRowBlock * PP);               // [4][32][SP]
  float* alpha_s = s_s + 4 * kRowBlock * SP;                                 // [32]
  float* m_s = alpha_s + kRowBlock;                                          // [32]
  float* l_s = m_s + kRowBlock;                                              // [32]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int wk = warp & 3, wn = warp >> 2;
  const int part = blockIdx.x, rb = blockIdx.y;
  const int SH = S * H;
  pdl_trigger();
  pdl_wait();
  const int4 pl = reinterpret_cast<const int4*>(plan)[part];
  if (pl.y <= pl.x) return;

  const int srow = tid >> 3, ssub = tid & 7;  // softmax: 8 threads per query row, 8 tokens each

  for (int b = pl.z; b <= pl.w; ++b) {
    const int c0 = cum[b] + kSegCost;  // slot of page 0 of sequence b
    const int pg_lo = max(pl.x, c0) - c0, pg_hi = min(pl.y, cum[b + 1]) - c0;
    if (pg_hi <= pg_lo) continue;
    const int L = clamped_len(seqlens[b], max_pages, nullptr);  // the plan block has already reported a bad length
    const int slot = part + b;
    __syncthreads();  // previous segment fully done with shared memory

    // ---- stage this sequence's 32 absorbed query rows, zero rows beyond S*H
    for (int i = tid; i < kRowBlock * (K / 8); i += 256) {
      const int rr = i / (K / 8), c = i % (K / 8);
      const int row = rb * kRowBlock + rr;
      const __nv_bfloat16* src = q_hat + (static_cast<size_t>(b) * SH + min(row, SH - 1)) * K + c * 8;
      cp_async16(q_s + rr * KP + c * 8, src, row < SH ? 16 : 0);
    }
    auto load_page = [&](int pj, int stage) {
      int idx = page_table[static_cast<size_t>(b) * max_pages + pj];
      const bool ok = idx >= 0 && idx < num_pages;
      if (!ok) { if (tid == 0) set_status(dev_status, TRANSMLA_DEV_BAD_PAGE); idx = 0; }
      const int valid = ok ? min(kPage, L - pj * kPage) : 0;  // rows beyond it are zero-filled
      const __nv_bfloat16* src = cache + static_cast<size_t>(idx) * kPage * K;
      __nv_bfloat16* dst = page_s + stage * kPage * KP;
      for (int i = tid; i < kPage * (K / 8); i += 256) {
        const int tok = i / (K / 8), c = i % (K / 8);
        cp_async16(dst + tok * KP + c * 8, src + static_cast<size_t>(tok) * K + c * 8, tok < valid ? 16 : 0);
      }
    };
    load_page(pg_lo, 0);
    cp_async_commit();

    const int my_row = rb * kRowBlock + srow;
    const int n_vis = my_row < SH ? L - (S - 1 - my_row / H) : 0;  // visible tokens of this thread's softmax row
    float m_run = -INFINITY, l_run = 0.f;
    float o[2][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[mt][nt][e] = 0.f;
    uint32_t qa[2][KSW][4];
    bool q_loaded = false;

    for (int pj = pg_lo; pj < pg_hi; ++pj) {
      const int stage = (pj - pg_lo) & 1;
      const int idx_cur = page_table[static_cast<size_t>(b) * max_pages + pj];
      // tokens of a page whose index is out of range are masked like tokens beyond the sequence
      const int tok_end = (idx_cur >= 0 && idx_cur < num_pages) ? n_vis - pj * kPage : 0;
      cp_async_wait<0>();
      __syncthreads();  // page pj (and, first time, the queries) landed; everyone is done with the other stage
      if (pj + 1 < pg_hi) { load_page(pj + 1, stage ^ 1); cp_async_commit(); }
      if (!q_loaded) {
        q_loaded = true;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
          for (int ks = 0; ks < KSW; ++ks) {
            const int kk = (wk * KSW + ks) * 16;
            if (kk < K) {
              const int mi = lane >> 3;
              ldmatrix_x4(qa[mt][ks], q_s + (mt * 16 + (mi & 1) * 8 + (lane & 7)) * KP + kk + (mi >> 1) * 8);
            } else {
              qa[mt][ks][0] = qa[mt][ks][1] = qa[mt][ks][2] = qa[mt][ks][3] = 0u;
            }
          }
      }
      const __nv_bfloat16* pg = page_s + stage * kPage * KP;

      // ---- S partial = Q_hat[:, k-slice] * K_hat[tokens of this warp, k-slice]^T
      float acc[2][4][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KSW; ++ks) {
        const int kk = (wk * KSW + ks) * 16;
        if (kk < K) {
#pragma unroll
          for (int np = 0; np < 2; ++np) {
            uint32_t bf[4];
            const int mi = lane >> 3;
            ldmatrix_x4(bf, pg + (wn * 32 + np * 16 + (mi >> 1) * 8 + (lane & 7)) * KP + kk + (mi & 1) * 8);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              mma_bf16_16816(acc[mt][np * 2], qa[mt][ks], bf[0], bf[1]);
              mma_bf16_16816(acc[mt][np * 2 + 1], qa[mt][ks], bf[2], bf[3]);
            }
          }
        }
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          float* d = s_s + (wk * kRowBlock + mt * 16 + g) * SP + wn * 32 + nt * 8 + t4 * 2;
          *reinterpret_cast<float2*>(d) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
          *reinterpret_cast<float2*>(d + 8 * SP) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
      __syncthreads();

      // ---- online softmax (base 2), 8 threads per row
      {
        float z[8];
        float tmax = -INFINITY;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int tok = ssub * 8 + j;
          float v = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w) v += s_s[(w * kRowBlock + srow) * SP + tok];
          v = (tok < tok_end) ? v * scale_log2 : -INFINITY;
          z[j] = v;
          tmax = fmaxf(tmax, v);
        }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 4));
        const float m_new = fmaxf(m_run, tmax);
        float alpha = 1.f, psum = 0.f;
        uint32_t pk[4];
        if (m_new == -INFINITY) {
          pk[0] = pk[1] = pk[2] = pk[3] = 0u;
        } else {
          alpha = exp2f(m_run - m_new);
#pragma unroll
          for (int j = 0; j < 8; j += 2) {
            const float p0 = exp2f(z[j] - m_new), p1 = exp2f(z[j + 1] - m_new);
            psum += p0 + p1;
            pk[j >> 1] = pack_bf16(p0, p1);
          }
        }
        psum += __shfl_xor_sync(0xffffffffu, psum, 1);
        psum += __shfl_xor_sync(0xffffffffu, psum, 2);
        psum += __shfl_xor_sync(0xffffffffu, psum, 4);
        l_run = l_run * alpha + psum;
        m_run = m_new;
        *reinterpret_cast<uint4*>(p_s + srow * PP + ssub * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        if (ssub == 0) alpha_s[srow] = alpha;
      }
      __syncthreads();

      // ---- O = O * alpha + P * C[:, columns of this warp]
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const float a0 = alpha_s[mt * 16 + g], a1 = alpha_s[mt * 16 + g + 8];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          o[mt][nt][0] *= a0; o[mt][nt][1] *= a0; o[mt][nt][2] *= a1; o[mt][nt][3] *= a1;
        }
      }
#pragma unroll
      for (int ks = 0; ks < kPage / 16; ++ks) {
        uint32_t pa[2][4];
        const int mi = lane >> 3;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
          ldmatrix_x4(pa[mt], p_s + (mt * 16 + (mi & 1) * 8 + (lane & 7)) * PP + ks * 16 + (mi >> 1) * 8);
        const int col0 = warp * (R / 8);
        if constexpr (NT >= 2) {
#pragma unroll
          for (int np = 0; np < NT / 2; ++np) {
            uint32_t bf[4];
            ldmatrix_x4_trans(bf, pg + (ks * 16 + (mi & 1) * 8 + (lane & 7)) * KP + col0 + np * 16 + (mi >> 1) * 8);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
              mma_bf16_16816(o[mt][np * 2], pa[mt], bf[0], bf[1]);
              mma_bf16_16816(o[mt][np * 2 + 1], pa[mt], bf[2], bf[3]);
            }
          }
        } else {
          uint32_t bf[2];
          ldmatrix_x2_trans(bf, pg + (ks * 16 + (mi & 1) * 8 + (lane & 7)) * KP + col0);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) mma_bf16_16816(o[mt][0], pa[mt], bf[0], bf[1]);
        }
      }
    }

    // ---- normalise and store the segment's partial result
    if (ssub == 0) { m_s[srow] = m_run; l_s[srow] = l_run; }
    __syncthreads();
    if (tid < kRowBlock) {
      const int row = rb * kRowBlock + tid;
      if (row < SH) {
        const float l = l_s[tid];
        partial_lse[static_cast<size_t>(slot) * SH + row] = l > 0.f ? (m_s[tid] + log2f(l)) * kLn2 : -INFINITY;
      }
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int rr = mt * 16 + g + hf * 8;
        const int row = rb * kRowBlock + rr;
        if (row >= SH) continue;
        const float l = l_s[rr];
        const float inv = l > 0.f ? 1.f / l : 0.f;
        float* dst = partial_o + (static_cast<size_t>(slot) * SH + row) * R + warp * (R / 8) + t4 * 2;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
          *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(o[mt][nt][hf * 2] * inv, o[mt][nt][hf * 2 + 1] * inv);
      }
  }
}

template <int R, int DR>
static cudaError_t launch_one(const transmla_params_t& p, int G, const __nv_bfloat16* q_hat,
                              const __nv_bfloat16* cache, const int32_t* page_table, const int32_t* seqlens,
                              const int32_t* cum, const int32_t* plan, float* partial_o, float* partial_lse,
                              int32_t* dev_status, cudaStream_t stream) {
  using C = GenericCfg<R, DR>;
  auto kern = decode_generic_kernel<R, DR>;
  static PerDeviceFlag smem_set;  // zero-initialised; one slot per device
  if (cudaError_t e = ensure_dynamic_smem(kern, static_cast<int>(C::smem_bytes), smem_set); e != cudaSuccess) return e;
  const int SH = p.q_len * p.num_heads;
  dim3 grid(G, (SH + kRowBlock - 1) / kRowBlock);
  return launch_pdl(kern, grid, dim3(256), C::smem_bytes, stream, q_hat, cache, page_table, seqlens, cum, plan, partial_o,
                    partial_lse, dev_status, p.q_len, p.num_heads, p.num_pages, p.max_pages_per_seq,
                    p.softmax_scale * kLog2e);
}

cudaError_t launch_decode_generic(const transmla_params_t& p, int G, const __nv_bfloat16* q_hat,
                                  const __nv_bfloat16* cache, const int32_t* page_table, const int32_t* seqlens,
                                  const int32_t* cum, const int32_t* plan, float* partial_o, float* partial_lse,
                                  int32_t* dev_status, cudaStream_t stream) {
  const int r = p.kv_lora_rank, dR = p.qk_rope_dim;
  if (r == 512 && dR == 64)
    return launch_one<512, 64>(p, G, q_hat, cache, page_table, seqlens, cum, plan, partial_o, partial_lse, dev_status, stream);
  if (r == 128 && dR == 0)
    return launch_one<128, 0>(p, G, q_hat, cache, page_table, seqlens, cum, plan, partial_o, partial_lse, dev_status, stream);
  if (r == 64 && dR == 16)
    return launch_one<64, 16>(p, G, q_hat, cache, page_table, seqlens, cum, plan, partial_o, partial_lse, dev_status, stream);
  return cudaErrorInvalidValue;
}

}  // namespace transmla
