// Decompression of the latent cache for prefill in the MHA form (Eq. 8): k^C_{j,h} = W_UK_h c_j, v_{j,h} = W_UV_h c_j.
//
// A GEMM [tokens x 512] x [512 x H*256] on the Blackwell tensor path.  One CTA = 128 tokens (two pages of one
// sequence, fetched through the page table) x all heads: the latent tile stays in shared memory (8 sub-tiles of
// 128 rows x 128 bytes, 128-byte swizzle), the weights of head h ([W_UK_h ; W_UV_h] = 256 rows x 512) stream
// through a three-stage ring 64 columns at a time, and D [128 x 256] alternates between two halves of the tensor
// memory so that the write-out of head h runs under the products of head h+1.
// Rows of tokens at or beyond the sequence length are stored as zeros: a probability of zero times such a value
// row must stay zero in the attention kernel.
// Warps 0-3 write out (thread = token row), warp 4 issues TMA, warp 5 issues the products.  Bounded waits.
#include "prefill.cuh"
#include "sm100_ptx.cuh"

namespace transmla {
namespace prefill {

using namespace sm100;

constexpr int R = 512, DR = 64, DN = 128, DV = 128;
constexpr int kTok = 128;                       // tokens per CTA
constexpr int kHeadCols = DN + DV;              // 256
constexpr int kASub = kTok * 128;               // 16384: 128 tokens x 64 latent columns
constexpr int kABytes = (R / 64) * kASub;       // 131072
constexpr int kBStage = kHeadCols * 128;        // 32768: 256 weight rows x 64 columns
constexpr int kBStages = 3;
constexpr int kOffA = 0, kOffB = kABytes, kOffBar = kOffB + kBStages * kBStage, kOffMisc = kOffBar + 128;
constexpr int kDecompSmem = kOffMisc + 64 + 1024;
static_assert(kOffBar % 256 == 0 && kDecompSmem <= 232448, "shared memory map");
enum { BAR_A_FULL = 0, BAR_B_FULL = 1, BAR_B_EMPTY = 1 + kBStages, BAR_D_FULL = 1 + 2 * kBStages, BAR_D_FREE = 3 + 2 * kBStages };

__host__ __device__ constexpr uint32_t instr_desc_mn(int m, int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

__global__ void __launch_bounds__(192, 1)
decompress_kernel(const __grid_constant__ CUtensorMap cache_map, const __grid_constant__ CUtensorMap wuk_map,
                  const __grid_constant__ CUtensorMap wuv_map, const int32_t* page_table, const int32_t* seqlens,
                  __nv_bfloat16* kv_dec, int32_t* dev_status, int H, int num_pages, int max_pages) {
  extern __shared__ unsigned char smem_unaligned[];
  const uint32_t raw = smem_u32(smem_unaligned);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_unaligned + (base - raw);
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(sm + kOffMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);
  auto bar = [&](int i) -> uint32_t { return base + kOffBar + 8 * i; };
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int jp = blockIdx.x, b = blockIdx.y;
  pdl_trigger();
  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&cache_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&wuk_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&wuv_map)) : "memory");
    mbar_init(bar(BAR_A_FULL), 1);
    for (int i = 0; i < kBStages; ++i) { mbar_init(bar(BAR_B_FULL + i), 1); mbar_init(bar(BAR_B_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar(BAR_D_FULL + i), 1); mbar_init(bar(BAR_D_FREE + i), 128); }
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
  const int L = clamped_len(seqlens[b], max_pages, tid == 0 ? dev_status : nullptr);
  const int n_pages = (L + kPage - 1) / kPage;
  const bool work = 2 * jp < n_pages;  // block-uniform
  if (work) {
    const bool two = 2 * jp + 1 < n_pages;
    int p0 = page_table[static_cast<size_t>(b) * max_pages + 2 * jp];
    int p1 = two ? page_table[static_cast<size_t>(b) * max_pages + 2 * jp + 1] : 0;
    const bool ok0 = p0 >= 0 && p0 < num_pages, ok1 = two && p1 >= 0 && p1 < num_pages;
    if ((!ok0 || (two && !ok1)) && tid == 0) set_status(dev_status, TRANSMLA_DEV_BAD_PAGE);
    if (!ok0) p0 = 0;
    if (!ok1) p1 = 0;
    if (warp == 4) {
      // ------------------------------------------------------------------ TMA: the latent tile once, then weights
      if (elect_one()) {
        mbar_arrive_expect_tx(bar(BAR_A_FULL), (two ? 2 : 1) * (R / 64) * kPage * 128);
        for (int c = 0; c < R / 64; ++c) {
          tma_load_2d(base + kOffA + c * kASub, &cache_map, c * 64, p0 * kPage, bar(BAR_A_FULL));
          if (two) tma_load_2d(base + kOffA + c * kASub + kPage * 128, &cache_map, c * 64, p1 * kPage, bar(BAR_A_FULL));
        }
      }
      __syncwarp();
      for (int it = 0; it < H * (R / 64); ++it) {
        const int h = it / (R / 64), kc = it % (R / 64), stage = it % kBStages, use = it / kBStages;
        mbar_wait(bar(BAR_B_EMPTY + stage), (use & 1) ^ 1, abort_flag, dev_status);
        if (!*abort_flag && elect_one()) {
          mbar_arrive_expect_tx(bar(BAR_B_FULL + stage), kBStage);
          const uint32_t dst = base + kOffB + stage * kBStage;
          tma_load_2d(dst, &wuk_map, kc * 64, h * DN, bar(BAR_B_FULL + stage));
          tma_load_2d(dst + DN * 128, &wuv_map, kc * 64, h * DV, bar(BAR_B_FULL + stage));
        }
        __syncwarp();
      }
    } else if (warp == 5) {
      // ------------------------------------------------------------------ products
      constexpr uint32_t idesc = instr_desc_mn(kTok, kHeadCols, false, false);
      const uint64_t a0 = smem_desc(base + kOffA, 16, 1024);
      mbar_wait(bar(BAR_A_FULL), 0, abort_flag, dev_status);
      for (int h = 0; h < H; ++h) {
        const int buf = h & 1;
        if (h >= 2) mbar_wait(bar(BAR_D_FREE + buf), ((h >> 1) - 1) & 1, abort_flag, dev_status);
        for (int kc = 0; kc < R / 64; ++kc) {
          const int it = h * (R / 64) + kc, stage = it % kBStages, use = it / kBStages;
          mbar_wait(bar(BAR_B_FULL + stage), use & 1, abort_flag, dev_status);
          tc_fence_after();
          const uint64_t b0 = smem_desc(base + kOffB + stage * kBStage, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            if (elect_one())
              mma_ss(tmem + buf * kHeadCols, desc_advance(a0, kc * kASub + kk * 32), desc_advance(b0, kk * 32), idesc,
                     (kc | kk) ? 1u : 0u);
          }
          if (elect_one()) tc_commit(bar(BAR_B_EMPTY + stage));
          __syncwarp();
        }
        if (elect_one()) tc_commit(bar(BAR_D_FULL + buf));
        __syncwarp();
      }
    } else if (warp < 4) {
      // ------------------------------------------------------------------ write-out: thread = token row
      const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
      const int row = warp * 32 + lane;
      const bool second = row >= kPage;
      const bool stored = !second || two;                         // the second page may not exist
      const int tok = (2 * jp + (second ? 1 : 0)) * kPage + (row & (kPage - 1));
      const bool real = tok < L;                                  // otherwise zeros
      const size_t row_elems = static_cast<size_t>(H) * kHeadCols;
      __nv_bfloat16* dst = kv_dec + (static_cast<size_t>(second ? p1 : p0) * kPage + (row & (kPage - 1))) * row_elems;
      for (int h = 0; h < H; ++h) {
        const int buf = h & 1;
        mbar_wait(bar(BAR_D_FULL + buf), (h >> 1) & 1, abort_flag, dev_status);
        tc_fence_after();
#pragma unroll 1
        for (int g = 0; g < kHeadCols / 32; ++g) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_base + buf * kHeadCols + g * 32, v);
          tc_wait_ld();
          if (stored) {
            uint4* d4 = reinterpret_cast<uint4*>(dst + h * kHeadCols + g * 32);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint4 o;
              o.x = real ? pack_bf16(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1])) : 0u;
              o.y = real ? pack_bf16(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])) : 0u;
              o.z = real ? pack_bf16(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])) : 0u;
              o.w = real ? pack_bf16(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])) : 0u;
              d4[q] = o;
            }
          }
        }
        tc_fence_before();
        mbar_arrive(bar(BAR_D_FREE + buf));
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

}  // namespace prefill

bool prefill_supported(const transmla_params_t& p) {
  return p.kv_lora_rank == prefill::R && p.qk_rope_dim == prefill::DR && p.qk_nope_dim == prefill::DN && p.v_dim == prefill::DV;
}

cudaError_t launch_prefill_decompress(const transmla_params_t& p, const __nv_bfloat16* cache, const int32_t* page_table,
                                      const int32_t* seqlens, const __nv_bfloat16* w_uk, const __nv_bfloat16* w_uv,
                                      __nv_bfloat16* kv_dec, int32_t* dev_status, cudaStream_t stream) {
  using namespace prefill;
  CUtensorMap cmap, kmap, vmap;
  if (!sm100::tensor_map_2d(&cmap, cache, static_cast<uint64_t>(p.num_pages) * kPage, R + DR, kPage) ||
      !sm100::tensor_map_2d(&kmap, w_uk, static_cast<uint64_t>(p.num_heads) * DN, R, DN) ||
      !sm100::tensor_map_2d(&vmap, w_uv, static_cast<uint64_t>(p.num_heads) * DV, R, DV))
    return cudaErrorInvalidValue;
  static PerDeviceFlag smem_set;
  if (cudaError_t e = ensure_dynamic_smem(decompress_kernel, kDecompSmem, smem_set); e != cudaSuccess) return e;
  dim3 grid((p.max_pages_per_seq + 1) / 2, p.batch);
  return launch_pdl(decompress_kernel, grid, dim3(192), static_cast<size_t>(kDecompSmem), stream, cmap, kmap, vmap, page_table,
                    seqlens, kv_dec, dev_status, p.num_heads, p.num_pages, p.max_pages_per_seq);
}

}  // namespace transmla
