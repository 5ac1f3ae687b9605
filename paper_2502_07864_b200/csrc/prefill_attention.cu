// Causal attention of a chunk of query positions over the decompressed keys and values (Eq. 9 left): prefill in
// the MHA form, per head  z = q_nope . k^C + q_pe . k^R,  softmax,  sum p v.
//
// One CTA = 128 query positions x one head x one sequence.  Per 64-token page:
//   S [128 x 64]  = Q (tensor memory, 96 columns: q_nope | q_pe) x [k^C | k^R]^T (shared memory, K-major), K = 192
//   O [128 x 128] += P (tensor memory, bf16, written by the softmax threads) x V (shared memory, MN-major)
// Query rows sit on the tensor-memory lanes, so a row's maximum, sum and rescale factor stay in its thread.
// S and P are double-buffered: the scores of page n+1 run under the softmax of page n, and the probabilities of
// page n+1 are written while PV of page n reads its own.
// k^C and v come from the decompressed store (row page*64 + slot, columns h*256 ..), k^R from the latent cache
// itself (columns 512..575 of the same row), all through the page table.
// Warps 0-3 softmax + write-out, warp 4 TMA, warp 5 issues QK^T, warp 6 issues PV.  Bounded waits throughout.
#include "prefill.cuh"
#include "sm100_ptx.cuh"

namespace transmla {
namespace prefill {

using namespace sm100;

constexpr int R_ = 512, DR_ = 64, DN_ = 128, DV_ = 128;
constexpr int kQRows = 128;
constexpr int kSub64 = kPage * 128;                // 8192: 64 tokens x 128 bytes
constexpr int kQSub = kQRows * 128;                // 16384: 128 query rows x 128 bytes
constexpr int kQBytes = 3 * kQSub;                 // q_nope (2 sub-tiles) | q_pe (1)
constexpr int kKvStage = 5 * kSub64;               // k^C (2) | k^R (1) | v (2) = 40960
constexpr int kKvStages = 4;
constexpr int kOffQ = 0, kOffKv = kQBytes, kOffBarA = kOffKv + kKvStages * kKvStage, kOffMiscA = kOffBarA + 256;
constexpr int kAttnSmem = kOffMiscA + 64 + 1024;
static_assert(kOffBarA % 256 == 0 && kAttnSmem <= 232448, "shared memory map");
constexpr uint32_t kColQ = 0, kColS = 96, kColP = 224, kColO = 288;  // S 2 x 64, P 2 x 32, O 128
enum { A_Q_FULL = 0, A_Q_READY, A_KV_FULL, A_KV_EMPTY = A_KV_FULL + kKvStages, A_S_FULL = A_KV_EMPTY + kKvStages,
       A_S_FREE = A_S_FULL + 2, A_P_READY = A_S_FREE + 2, A_PV_DONE = A_P_READY + 2 };

__host__ __device__ constexpr uint32_t idesc_attn(int m, int n, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(224, 1)
prefill_attention_kernel(const __grid_constant__ CUtensorMap qn_map, const __grid_constant__ CUtensorMap qr_map,
                         const __grid_constant__ CUtensorMap kv_map, const __grid_constant__ CUtensorMap cache_map,
                         const int32_t* page_table, const int32_t* seqlens, __nv_bfloat16* out, float* lse_out,
                         int32_t* dev_status, int S, int H, int num_pages, int max_pages, float scale_log2) {
  extern __shared__ unsigned char smem_unaligned[];
  const uint32_t raw = smem_u32(smem_unaligned);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_unaligned + (base - raw);
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(sm + kOffMiscA);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);
  auto bar = [&](int i) -> uint32_t { return base + kOffBarA + 8 * i; };
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  pdl_trigger();
  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&qn_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&qr_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&kv_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&cache_map)) : "memory");
    mbar_init(bar(A_Q_FULL), 1);
    mbar_init(bar(A_Q_READY), 128);
    for (int i = 0; i < kKvStages; ++i) { mbar_init(bar(A_KV_FULL + i), 1); mbar_init(bar(A_KV_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(A_S_FULL + i), 1);
      mbar_init(bar(A_S_FREE + i), 128);
      mbar_init(bar(A_P_READY + i), 128);
      mbar_init(bar(A_PV_DONE + i), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  pdl_wait();
  const int L = clamped_len(seqlens[b], max_pages, (tid == 0 && qt == 0 && h == 0) ? dev_status : nullptr);
  // Query position s of the chunk sees tokens [0, L - (S - 1 - s)); the tile's last position sees the most.
  const int s_first = qt * kQRows, s_last = min(S, s_first + kQRows) - 1;
  const int vis_max = max(0, L - (S - 1 - s_last));
  const int n_tiles = (vis_max + kPage - 1) / kPage;  // block-uniform

  if (n_tiles > 0) {
    if (warp == 4) {
      // ======================================================================== TMA producer
      if (elect_one()) {
        mbar_arrive_expect_tx(bar(A_Q_FULL), kQBytes);
        const int row0 = b * S + s_first;
        tma_load_2d(base + kOffQ, &qn_map, h * DN_, row0, bar(A_Q_FULL));
        tma_load_2d(base + kOffQ + kQSub, &qn_map, h * DN_ + 64, row0, bar(A_Q_FULL));
        tma_load_2d(base + kOffQ + 2 * kQSub, &qr_map, h * DR_, row0, bar(A_Q_FULL));
      }
      __syncwarp();
      const int32_t* row = page_table + static_cast<size_t>(b) * max_pages;
      for (int n = 0; n < n_tiles; ++n) {
        int idx = row[n];
        const bool ok = idx >= 0 && idx < num_pages;
        if (!ok) { if (lane == 0) set_status(dev_status, TRANSMLA_DEV_BAD_PAGE); idx = 0; }
        const int stage = n % kKvStages, use = n / kKvStages;
        mbar_wait(bar(A_KV_EMPTY + stage), (use & 1) ^ 1, abort_flag, dev_status);
        if (!*abort_flag && elect_one()) {
          mbar_arrive_expect_tx(bar(A_KV_FULL + stage), kKvStage);
          const uint32_t dst = base + kOffKv + stage * kKvStage;
          const int x = h * (DN_ + DV_), y = idx * kPage;
          tma_load_2d(dst, &kv_map, x, y, bar(A_KV_FULL + stage));
          tma_load_2d(dst + kSub64, &kv_map, x + 64, y, bar(A_KV_FULL + stage));
          tma_load_2d(dst + 2 * kSub64, &cache_map, R_, y, bar(A_KV_FULL + stage));
          tma_load_2d(dst + 3 * kSub64, &kv_map, x + DN_, y, bar(A_KV_FULL + stage));
          tma_load_2d(dst + 4 * kSub64, &kv_map, x + DN_ + 64, y, bar(A_KV_FULL + stage));
        }
        __syncwarp();
      }
    } else if (warp == 5) {
      // ======================================================================== MMA issuer, scores
      constexpr uint32_t idesc_qk = idesc_attn(kQRows, kPage, false);
      mbar_wait(bar(A_Q_READY), 0, abort_flag, dev_status);
      for (int n = 0; n < n_tiles; ++n) {
        const int stage = n % kKvStages, use = n / kKvStages, buf = n & 1;
        mbar_wait(bar(A_KV_FULL + stage), use & 1, abort_flag, dev_status);
        if (n >= 2) mbar_wait(bar(A_S_FREE + buf), ((n >> 1) - 1) & 1, abort_flag, dev_status);
        tc_fence_after();
        const uint64_t k0 = smem_desc(base + kOffKv + stage * kKvStage, 16, 1024);
#pragma unroll
        for (int c = 0; c < 3; ++c) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            if (elect_one())
              mma_ts(tmem + kColS + buf * 64, tmem + kColQ + c * 32 + kk * 8, desc_advance(k0, c * kSub64 + kk * 32), idesc_qk,
                     (c | kk) ? 1u : 0u);
          }
        }
        if (elect_one()) tc_commit(bar(A_S_FULL + buf));
        __syncwarp();
      }
    } else if (warp == 6) {
      // ======================================================================== MMA issuer, products
      constexpr uint32_t idesc_pv = idesc_attn(kQRows, DV_, true);
      for (int n = 0; n < n_tiles; ++n) {
        const int stage = n % kKvStages, use = n / kKvStages, buf = n & 1;
        mbar_wait(bar(A_KV_FULL + stage), use & 1, abort_flag, dev_status);
        mbar_wait(bar(A_P_READY + buf), (n >> 1) & 1, abort_flag, dev_status);
        tc_fence_after();
        const uint64_t v0 = smem_desc(base + kOffKv + stage * kKvStage + 3 * kSub64, kSub64, 1024);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          if (elect_one())
            mma_ts(tmem + kColO, tmem + kColP + buf * 32 + kk * 8, desc_advance(v0, kk * 2048), idesc_pv, (n | kk) ? 1u : 0u);
        }
        if (elect_one()) {
          tc_commit(bar(A_KV_EMPTY + stage));
          tc_commit(bar(A_PV_DONE + buf));
        }
        __syncwarp();
      }
    } else if (warp < 4) {
      // ======================================================================== softmax + write-out (warps 0-3)
      const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
      const int row = warp * 32 + lane, s = s_first + row;
      const bool in_chunk = s < S;
      // rows of the tile beyond the chunk are computed unmasked and never stored
      const int n_vis = in_chunk ? max(0, L - (S - 1 - s)) : 0x3fffffff;
      mbar_wait(bar(A_Q_FULL), 0, abort_flag, dev_status);
      {  // this thread's query row: shared memory (swizzled sub-tiles of 128 rows x 128 bytes) -> tensor memory
        const unsigned char* qrow = sm + kOffQ + row * 128;
#pragma unroll 1
        for (int c = 0; c < 3; ++c) {
          uint32_t v[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(qrow + c * kQSub + ((j ^ (row & 7)) << 4));
            v[4 * j] = x.x; v[4 * j + 1] = x.y; v[4 * j + 2] = x.z; v[4 * j + 3] = x.w;
          }
          tmem_st32(tmem + lane_base + kColQ + c * 32, v);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar(A_Q_READY));
      }
      const bool pos_scale = scale_log2 >= 0.f;
      float m_used = -INFINITY, l_run = 0.f;
      for (int n = 0; n < n_tiles; ++n) {
        const int buf = n & 1;
        mbar_wait(bar(A_S_FULL + buf), (n >> 1) & 1, abort_flag, dev_status);
        tc_fence_after();
        uint32_t sq[64];
        tmem_ld32(tmem + lane_base + kColS + buf * 64, sq);
        tmem_ld32(tmem + lane_base + kColS + buf * 64 + 32, sq + 32);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(A_S_FREE + buf));
        const int tok_end = n_vis - n * kPage;  // tokens [0, tok_end) of the page are visible to this row
        const bool full = __all_sync(0xffffffffu, tok_end >= kPage) && pos_scale;
        float rowmax = -INFINITY;
        if (full) {
          float a = __uint_as_float(sq[0]), c2 = __uint_as_float(sq[1]);
#pragma unroll
          for (int j = 2; j < 64; j += 2) { a = fmaxf(a, __uint_as_float(sq[j])); c2 = fmaxf(c2, __uint_as_float(sq[j + 1])); }
          rowmax = fmaxf(a, c2) * scale_log2;
        } else {
#pragma unroll
          for (int j = 0; j < 64; ++j) rowmax = fmaxf(rowmax, j < tok_end ? __uint_as_float(sq[j]) * scale_log2 : -INFINITY);
        }
        // Lazy rescale: the reference maximum only moves when some row of the warp exceeds it by 2^8.
        bool resc = false;
        float alpha = 1.f;
        if (n == 0) {
          m_used = rowmax;
        } else {
          resc = __any_sync(0xffffffffu, rowmax > m_used + 8.f);
          if (resc) {
            const float m_new = fmaxf(m_used, rowmax);
            alpha = (m_new == -INFINITY) ? 1.f : exp2f(m_used - m_new);
            m_used = m_new;
            l_run *= alpha;
          }
        }
        const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
        uint32_t pk[32];
        float ps0 = 0.f, ps1 = 0.f;
        if (full) {
#pragma unroll
          for (int j = 0; j < 64; j += 2) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(sq[j]), scale_log2, neg_m));
            const float p1 = ex2_approx(fmaf(__uint_as_float(sq[j + 1]), scale_log2, neg_m));
            ps0 += p0; ps1 += p1;
            pk[j >> 1] = pack_bf16(p0, p1);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 64; j += 2) {
            const float p0 = j < tok_end ? ex2_approx(fmaf(__uint_as_float(sq[j]), scale_log2, neg_m)) : 0.f;
            const float p1 = j + 1 < tok_end ? ex2_approx(fmaf(__uint_as_float(sq[j + 1]), scale_log2, neg_m)) : 0.f;
            ps0 += p0; ps1 += p1;
            pk[j >> 1] = pack_bf16(p0, p1);
          }
        }
        l_run += ps0 + ps1;
        // P buffer `buf` was read by PV of page n-2
        if (n >= 2) mbar_wait(bar(A_PV_DONE + buf), ((n >> 1) - 1) & 1, abort_flag, dev_status);
        if (resc) {  // warp-uniform; O must be at rest: PV of page n-1 complete
          mbar_wait(bar(A_PV_DONE + ((n - 1) & 1)), ((n - 1) >> 1) & 1, abort_flag, dev_status);
          tc_fence_after();
#pragma unroll 1
          for (int g = 0; g < DV_ / 32; ++g) {
            uint32_t ov[32];
            tmem_ld32(tmem + lane_base + kColO + g * 32, ov);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
            tmem_st32(tmem + lane_base + kColO + g * 32, ov);
          }
        }
        tmem_st32(tmem + lane_base + kColP + buf * 32, pk);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar(A_P_READY + buf));
      }
      // ---- write-out: wait for the last PV, normalise, store the row
      const int last = n_tiles - 1;
      mbar_wait(bar(A_PV_DONE + (last & 1)), (last >> 1) & 1, abort_flag, dev_status);
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      __nv_bfloat16* dst = out + ((static_cast<size_t>(b) * S + s) * H + h) * DV_;
#pragma unroll 1
      for (int g = 0; g < DV_ / 32; ++g) {
        uint32_t ov[32];
        tmem_ld32(tmem + lane_base + kColO + g * 32, ov);
        tc_wait_ld();
        if (in_chunk) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint4 o;
            o.x = pack_bf16(__uint_as_float(ov[8 * q]) * inv, __uint_as_float(ov[8 * q + 1]) * inv);
            o.y = pack_bf16(__uint_as_float(ov[8 * q + 2]) * inv, __uint_as_float(ov[8 * q + 3]) * inv);
            o.z = pack_bf16(__uint_as_float(ov[8 * q + 4]) * inv, __uint_as_float(ov[8 * q + 5]) * inv);
            o.w = pack_bf16(__uint_as_float(ov[8 * q + 6]) * inv, __uint_as_float(ov[8 * q + 7]) * inv);
            reinterpret_cast<uint4*>(dst + g * 32)[q] = o;
          }
        }
      }
      if (in_chunk && lse_out != nullptr)
        lse_out[(static_cast<size_t>(b) * S + s) * H + h] = l_run > 0.f ? (m_used + log2f(l_run)) * kLn2 : -INFINITY;
      tc_fence_before();
    }
  } else if (warp < 4) {
    // nothing visible to any row of the tile (L < S): zeros and lse = -inf
    const int s = s_first + warp * 32 + lane;
    if (s < S) {
      uint4* dst = reinterpret_cast<uint4*>(out + ((static_cast<size_t>(b) * S + s) * H + h) * DV_);
      for (int q = 0; q < DV_ / 8; ++q) dst[q] = make_uint4(0, 0, 0, 0);
      if (lse_out != nullptr) lse_out[(static_cast<size_t>(b) * S + s) * H + h] = -INFINITY;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

}  // namespace prefill

cudaError_t launch_prefill_attention(const transmla_params_t& p, const __nv_bfloat16* q_nope, const __nv_bfloat16* q_pe,
                                     const __nv_bfloat16* cache, const __nv_bfloat16* kv_dec, const int32_t* page_table,
                                     const int32_t* seqlens, __nv_bfloat16* out, float* lse, int32_t* dev_status,
                                     cudaStream_t stream) {
  using namespace prefill;
  // q_nope as [B*S rows, H*dn], q_pe as [B*S, H*dR]: a box is 128 rows (positions) x 64 columns of one head.
  CUtensorMap qn, qr, kv, cm;
  const uint64_t rows = static_cast<uint64_t>(p.batch) * p.q_len;
  if (!sm100::tensor_map_2d(&qn, q_nope, rows, p.num_heads * DN_, kQRows) ||
      !sm100::tensor_map_2d(&qr, q_pe, rows, p.num_heads * DR_, kQRows) ||
      !sm100::tensor_map_2d(&kv, kv_dec, static_cast<uint64_t>(p.num_pages) * kPage, p.num_heads * (DN_ + DV_), kPage) ||
      !sm100::tensor_map_2d(&cm, cache, static_cast<uint64_t>(p.num_pages) * kPage, R_ + DR_, kPage))
    return cudaErrorInvalidValue;
  static PerDeviceFlag smem_set;
  if (cudaError_t e = ensure_dynamic_smem(prefill_attention_kernel, kAttnSmem, smem_set); e != cudaSuccess) return e;
  dim3 grid((p.q_len + kQRows - 1) / kQRows, p.num_heads, p.batch);
  return launch_pdl(prefill_attention_kernel, grid, dim3(224), static_cast<size_t>(kAttnSmem), stream, qn, qr, kv, cm, page_table,
                    seqlens, out, lse, dev_status, p.q_len, p.num_heads, p.num_pages, p.max_pages_per_seq,
                    p.softmax_scale * kLog2e);
}
}  // namespace transmla
