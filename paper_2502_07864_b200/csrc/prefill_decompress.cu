// Decompression of the latent cache for prefill in the MHA form (Eq. 8): k^C_{j,h} = W_UK_h c_j, v_{j,h} = W_UV_h c_j.
//
// A GEMM [tokens x 512] x [512 x H*256] on the Blackwell tensor path.  One CTA = 128 tokens (two pages of one
// sequence, fetched through the page table) x all heads.  The latent tile lives in tensor memory (256 columns of
// packed bf16 pairs, the A operand of every instruction); the weights of head h ([W_UK_h ; W_UV_h] = 256 rows x 512)
// stream through a four-stage ring 64 columns at a time; D [128 x 256] takes the other 256 columns.  The tile reaches
// tensor memory through the four ring stages before the first weights.
// Write-out: D goes to a 64 KB staging tile in shared memory as bf16 (the layout of the store's tensor map) and from
// there to the store by TMA, whole 128-byte lines at a time; thread-per-row stores straight from registers (16 bytes
// per lane, rows 16 KB apart) took longer than the head's products.  Tensor memory is released as soon as it has
// been read, so the next head's products run under the conversion and the store.
// Rows of tokens at or beyond the sequence length are stored as zeros: a probability of zero times such a value
// row must stay zero in the attention kernel.
// Warps 0-7 move the tile and write out (warp w: tensor-memory lanes 32 (w % 4).., columns 128 (w / 4)..), warp 8
// issues TMA, warp 9 issues the products.  Bounded waits.
#include "prefill.cuh"
#include "sm100_ptx.cuh"

namespace transmla {
namespace prefill {

using namespace sm100;

constexpr int R = 512, DR = 64, DN = 128, DV = 128;
constexpr int kTok = 128;                       // tokens per CTA
constexpr int kHeadCols = DN + DV;              // 256
constexpr int kASub = kTok * 128;               // 16384: 128 tokens x 64 latent columns
constexpr int kBStage = kHeadCols * 128;        // 32768: 256 weight rows x 64 columns, or two 64-column pieces of the tile
constexpr int kBStages = 4;
constexpr int kAStages = (R / 64) * kASub / kBStage;  // 4: ring stages the latent tile passes through
constexpr int kOutBytes = kTok * kHeadCols * 2;  // 65536: the staging tile, 2 pages x 4 boxes of 64 rows x 128 bytes
constexpr int kOffB = 0, kOffOut = kOffB + kBStages * kBStage, kOffBar = kOffOut + kOutBytes, kOffMisc = kOffBar + 256;
constexpr int kDecompSmem = kOffMisc + 64 + 1024;
constexpr int kDecompThreads = 320;
constexpr uint32_t kColA = 0, kColD = 256;
static_assert(kOffBar % 256 == 0 && kDecompSmem <= 232448, "shared memory map");
enum { BAR_B_FULL = 0, BAR_B_EMPTY = kBStages, BAR_A_READY = 2 * kBStages, BAR_D_FULL, BAR_D_FREE };

__host__ __device__ constexpr uint32_t instr_desc_mn(int m, int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

__global__ void __launch_bounds__(kDecompThreads, 1)
decompress_kernel(const __grid_constant__ CUtensorMap cache_map, const __grid_constant__ CUtensorMap wuk_map,
                  const __grid_constant__ CUtensorMap wuv_map, const __grid_constant__ CUtensorMap out_map,
                  const int32_t* page_table, const int32_t* seqlens,
                  int32_t* dev_status, int H, int num_pages, int max_pages) {
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
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&out_map)) : "memory");
    for (int i = 0; i < kBStages; ++i) { mbar_init(bar(BAR_B_FULL + i), 1); mbar_init(bar(BAR_B_EMPTY + i), 1); }
    mbar_init(bar(BAR_A_READY), 256);
    mbar_init(bar(BAR_D_FULL), 1);
    mbar_init(bar(BAR_D_FREE), 256);
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
    if (warp == 8) {
      // ------------------------------------------------------------------ TMA: the latent tile, then the weights
      // Ring item g: items 0..3 carry the tile (two 64-column pieces each, 128 rows x 128 bytes per piece),
      // items 4.. the weights; item g uses stage g % 4.
      if (elect_one()) {
        for (int g = 0; g < kAStages; ++g) {
          mbar_arrive_expect_tx(bar(BAR_B_FULL + g), 2 * (two ? 2 : 1) * kPage * 128);
          for (int u = 0; u < 2; ++u) {
            const uint32_t dst = base + kOffB + g * kBStage + u * kASub;
            tma_load_2d(dst, &cache_map, (2 * g + u) * 64, p0 * kPage, bar(BAR_B_FULL + g));
            if (two) tma_load_2d(dst + kPage * 128, &cache_map, (2 * g + u) * 64, p1 * kPage, bar(BAR_B_FULL + g));
          }
        }
      }
      __syncwarp();
      for (int it = 0; it < H * (R / 64); ++it) {
        const int h = it / (R / 64), kc = it % (R / 64), g = it + kAStages, stage = g % kBStages, use = g / kBStages;
        mbar_wait(bar(BAR_B_EMPTY + stage), (use & 1) ^ 1, abort_flag, dev_status);
        if (!*abort_flag && elect_one()) {
          mbar_arrive_expect_tx(bar(BAR_B_FULL + stage), kBStage);
          const uint32_t dst = base + kOffB + stage * kBStage;
          tma_load_2d(dst, &wuk_map, kc * 64, h * DN, bar(BAR_B_FULL + stage));
          tma_load_2d(dst + DN * 128, &wuv_map, kc * 64, h * DV, bar(BAR_B_FULL + stage));
        }
        __syncwarp();
      }
    } else if (warp == 9) {
      // ------------------------------------------------------------------ products
      constexpr uint32_t idesc = instr_desc_mn(kTok, kHeadCols, false, false);
      mbar_wait(bar(BAR_A_READY), 0, abort_flag, dev_status);
      for (int h = 0; h < H; ++h) {
        if (h >= 1) mbar_wait(bar(BAR_D_FREE), (h - 1) & 1, abort_flag, dev_status);
        for (int kc = 0; kc < R / 64; ++kc) {
          const int g = h * (R / 64) + kc + kAStages, stage = g % kBStages, use = g / kBStages;
          mbar_wait(bar(BAR_B_FULL + stage), use & 1, abort_flag, dev_status);
          tc_fence_after();
          const uint64_t b0 = smem_desc(base + kOffB + stage * kBStage, 16, 1024);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            if (elect_one())
              mma_ts(tmem + kColD, tmem + kColA + kc * 32 + kk * 8, desc_advance(b0, kk * 32), idesc, (kc | kk) ? 1u : 0u);
          }
          if (elect_one()) tc_commit(bar(BAR_B_EMPTY + stage));
          __syncwarp();
        }
        if (elect_one()) tc_commit(bar(BAR_D_FULL));
        __syncwarp();
      }
    } else {
      // ------------------------------------------------------------------ warps 0-7: thread = token row
      const int quarter = warp & 3, half = warp >> 2;
      const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
      const int row = quarter * 32 + lane;
      // the latent tile, shared memory (swizzled pieces of 128 rows x 128 bytes) -> tensor memory: the warps of half 0
      // move ring items 0 and 1, those of half 1 items 2 and 3
      for (int g = 2 * half; g < 2 * half + 2; ++g) {
        mbar_wait(bar(BAR_B_FULL + g), 0, abort_flag, dev_status);
#pragma unroll 1
        for (int u = 0; u < 2; ++u) {
          const unsigned char* prow = sm + kOffB + g * kBStage + u * kASub + row * 128;
          uint32_t v[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(prow + ((j ^ (row & 7)) << 4));
            v[4 * j] = x.x; v[4 * j + 1] = x.y; v[4 * j + 2] = x.z; v[4 * j + 3] = x.w;
          }
          tmem_st32(tmem + lane_base + kColA + (2 * g + u) * 32, v);
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_A_READY));
      if (half == 0) asm volatile("bar.sync 1, 128;" ::: "memory"); else asm volatile("bar.sync 2, 128;" ::: "memory");
      if ((tid & 127) == 0) { mbar_arrive(bar(BAR_B_EMPTY + 2 * half)); mbar_arrive(bar(BAR_B_EMPTY + 2 * half + 1)); }
      // write-out of D, columns 128 * half .. + 127 of every head
      const bool second = row >= kPage;
      const int slot = row & (kPage - 1);
      const int tok = (2 * jp + (second ? 1 : 0)) * kPage + slot;
      const bool real = tok < L;                                  // otherwise zeros
      // staging: box (page p, 64-column piece c) at ((p * 4 + c) * 8192), row `slot` at 128 bytes, 16-byte unit j at j ^ (slot & 7)
      unsigned char* stage_row = sm + kOffOut + ((second ? 4 : 0) + 2 * half) * 8192 + slot * 128;
      for (int h = 0; h < H; ++h) {
        mbar_wait(bar(BAR_D_FULL), h & 1, abort_flag, dev_status);
        tc_fence_after();
        uint32_t v[128];
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) tmem_ld32(tmem + lane_base + kColD + half * 128 + gq * 32, v + 32 * gq);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(bar(BAR_D_FREE));                             // the next head's products may start
        // the TMA store of the head before must have finished reading the staging tile
        if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        asm volatile("bar.sync 3, 256;" ::: "memory");
#pragma unroll
        for (int c = 0; c < 2; ++c) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t* x = v + c * 64 + j * 8;
            uint4 o;
            o.x = real ? pack_bf16(__uint_as_float(x[0]), __uint_as_float(x[1])) : 0u;
            o.y = real ? pack_bf16(__uint_as_float(x[2]), __uint_as_float(x[3])) : 0u;
            o.z = real ? pack_bf16(__uint_as_float(x[4]), __uint_as_float(x[5])) : 0u;
            o.w = real ? pack_bf16(__uint_as_float(x[6]), __uint_as_float(x[7])) : 0u;
            *reinterpret_cast<uint4*>(stage_row + c * 8192 + ((j ^ (slot & 7)) << 4)) = o;
          }
        }
        fence_proxy_async();
        asm volatile("bar.sync 3, 256;" ::: "memory");
        if (tid == 0) {
          for (int pg = 0; pg < (two ? 2 : 1); ++pg) {
            if (!(pg ? ok1 : ok0)) continue;   // a page the table does not name validly is reported, not written
            for (int c = 0; c < 4; ++c)
              asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                           ::"l"(reinterpret_cast<uint64_t>(&out_map)), "r"(h * kHeadCols + c * 64), "r"((pg ? p1 : p0) * kPage),
                             "r"(base + kOffOut + (pg * 4 + c) * 8192)
                           : "memory");
          }
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // the last stores have left shared memory and landed
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
  CUtensorMap cmap, kmap, vmap, omap;
  if (!sm100::tensor_map_2d(&cmap, cache, static_cast<uint64_t>(p.num_pages) * kPage, R + DR, kPage) ||
      !sm100::tensor_map_2d(&kmap, w_uk, static_cast<uint64_t>(p.num_heads) * DN, R, DN) ||
      !sm100::tensor_map_2d(&vmap, w_uv, static_cast<uint64_t>(p.num_heads) * DV, R, DV) ||
      !sm100::tensor_map_2d(&omap, kv_dec, static_cast<uint64_t>(p.num_pages) * kPage, p.num_heads * kHeadCols, kPage))
    return cudaErrorInvalidValue;
  static PerDeviceFlag smem_set;
  if (cudaError_t e = ensure_dynamic_smem(decompress_kernel, kDecompSmem, smem_set); e != cudaSuccess) return e;
  dim3 grid((p.max_pages_per_seq + 1) / 2, p.batch);
  return launch_pdl(decompress_kernel, grid, dim3(kDecompThreads), static_cast<size_t>(kDecompSmem), stream, cmap, kmap, vmap, omap, page_table,
                    seqlens, dev_status, p.num_heads, p.num_pages, p.max_pages_per_seq);
}

}  // namespace transmla
