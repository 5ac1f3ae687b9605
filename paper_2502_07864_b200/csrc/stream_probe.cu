// Read-only streaming probe: what the split-KV kernel's access pattern costs when nothing is computed.
//
// Same grid (one CTA per partition and block of 32 query rows), same split plan, same ring of three 73 728-byte
// stages filled by the same TMA boxes (nine 64-token x 64-column boxes per page, 128-byte swizzle, evict-first),
// but the consumer is a single warp that hands every stage back as soon as it has landed: no tensor-core work,
// no softmax, no output.  Its duration is the ceiling that launch, ramp-up and the memory system put on any kernel
// that streams the latent cache this way; the split-KV kernel's own time is to be read against it.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace transmla {
namespace sm100 {

constexpr int kProbeK = 576;
constexpr int kProbeChunks = kProbeK / 64;
constexpr int kProbeSubTile = kPage * 128;
constexpr int kProbeStage = kProbeChunks * kProbeSubTile;  // 73728
constexpr int kProbeStages = 3;
constexpr int kProbeSmem = kProbeStages * kProbeStage + 1024 + 256;

__global__ void __launch_bounds__(64, 1)
stream_probe_kernel(const __grid_constant__ CUtensorMap cache_map, const int32_t* page_table, const int32_t* cum,
                    const int32_t* plan, int32_t* dev_status, int num_pages, int max_pages) {
  extern __shared__ unsigned char smem_unaligned[];
  const uint32_t raw = smem_u32(smem_unaligned);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_unaligned + (base - raw);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + kProbeStages * kProbeStage + 128);
  auto full = [&](int i) -> uint32_t { return base + kProbeStages * kProbeStage + 8 * i; };
  auto empty = [&](int i) -> uint32_t { return base + kProbeStages * kProbeStage + 8 * (kProbeStages + i); };
  const int tid = threadIdx.x, warp = tid >> 5;
  pdl_trigger();
  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&cache_map)) : "memory");
    for (int i = 0; i < kProbeStages; ++i) { mbar_init(full(i), 1); mbar_init(empty(i), 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  pdl_wait();
  const int4 pl = reinterpret_cast<const int4*>(plan)[blockIdx.x];
  if (pl.y <= pl.x) return;
  int total = 0;  // pages of this partition (both warps count them the same way)
  for (int b = pl.z; b <= pl.w; ++b) {
    const int c0 = cum[b] + kSegCost;
    total += max(0, min(pl.y, cum[b + 1]) - max(pl.x, c0));
  }
  if (warp == 0) {  // producer
    const uint64_t policy = l2_evict_first_policy();
    int g = 0;
    for (int b = pl.z; b <= pl.w; ++b) {
      const int c0 = cum[b] + kSegCost;
      const int lo = max(pl.x, c0) - c0, hi = min(pl.y, cum[b + 1]) - c0;
      for (int pj = lo; pj < hi; ++pj, ++g) {
        int idx = pj < max_pages ? page_table[static_cast<size_t>(b) * max_pages + pj] : -1;
        if (idx < 0 || idx >= num_pages) { if ((tid & 31) == 0) set_status(dev_status, TRANSMLA_DEV_BAD_PAGE); idx = 0; }
        const int stage = g % kProbeStages, use = g / kProbeStages;
        mbar_wait(empty(stage), (use & 1) ^ 1, abort_flag, dev_status);
        if (!*abort_flag && elect_one()) {
          mbar_arrive_expect_tx(full(stage), kProbeStage);
#pragma unroll
          for (int c = 0; c < kProbeChunks; ++c)
            tma_load_2d_hint(base + stage * kProbeStage + c * kProbeSubTile, &cache_map, c * 64, idx * kPage, full(stage), policy);
        }
        __syncwarp();
      }
    }
  } else {  // consumer: every stage goes back at once
    for (int g = 0; g < total; ++g) {
      const int stage = g % kProbeStages, use = g / kProbeStages;
      mbar_wait(full(stage), use & 1, abort_flag, dev_status);
      if (elect_one()) mbar_arrive(empty(stage));
      __syncwarp();
    }
  }
}

}  // namespace sm100

cudaError_t launch_stream_probe(const transmla_params_t& p, int G, const __nv_bfloat16* cache, const int32_t* page_table,
                                const int32_t* cum, const int32_t* plan, int32_t* dev_status, cudaStream_t stream) {
  using namespace sm100;
  CUtensorMap map;
  if (!tensor_map_2d(&map, cache, static_cast<uint64_t>(p.num_pages) * kPage, kProbeK, kPage)) return cudaErrorInvalidValue;
  static PerDeviceFlag smem_set;
  if (cudaError_t e = ensure_dynamic_smem(stream_probe_kernel, kProbeSmem, smem_set); e != cudaSuccess) return e;
  const int SH = p.q_len * p.num_heads;
  dim3 grid(G, (SH + kRowBlock - 1) / kRowBlock);
  return launch_pdl(stream_probe_kernel, grid, dim3(64), static_cast<size_t>(kProbeSmem), stream, map, page_table, cum, plan,
                    dev_status, p.num_pages, p.max_pages_per_seq);
}

}  // namespace transmla
