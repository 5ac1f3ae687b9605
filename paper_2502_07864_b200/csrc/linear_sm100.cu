// Weight-streaming linear maps on the Blackwell tensor path: y[M, N] = x[M, K] w[N, K]^T for the few tokens of a
// decode step (Eq. 8 right column: c^Q, q^C, q^R; Eq. 9 last line: W_O).
//
// The weights are the large operand (tens of MB, read once), the activations the small one.  A CTA owns 128
// output features and one slice of K:
//   D^T[128 features x T tokens] += W_tile[128 x 64] (A, shared memory, K-major) x X_tile[T x 64]^T (B, K-major)
// with the accumulator in tensor memory, so that the 128 lanes of the MMA are always full whatever the number of
// tokens (16 <= T <= 256, tokens padded to a multiple of 16; rows beyond M read as zero through the tensor map).
// Per CTA the shared-memory traffic is (128 + T) x K_slice x 2 bytes, i.e. the activations are re-read once per
// 128 features, not once per 8 or 32 as in the mma.sync tiles of skinny_gemm.cuh.
// K is cut into `splits` slices so that every SM streams weights (N / 128 tiles alone would occupy 32-48 SMs).
// The slices of a tile are the CTAs of one thread-block cluster: each leaves its fp32 partial in its own shared
// memory (the ring is free by then), and after a cluster barrier every CTA adds the slices of its share of the
// tokens in slice order, reading the others' shared memory directly, applies RoPE where asked and writes bf16 (no
// float atomics: reruns give the same bits).  If the clusters do not all fit on the device at once, or there are
// more than 8 slices, the partials go through a scratch buffer instead and the CTA that arrives last at the tile's
// counter adds them.
//
// Warps: 0 TMA producer, 1 MMA issuer, 2-5 epilogue (each owns the 32 tensor-memory lanes of its quadrant).
#include "common.cuh"
#include "linear_args.cuh"
#include "sm100_ptx.cuh"

namespace transmla {
namespace sm100 {

constexpr int kLinBM = 128;                      // output features per CTA
constexpr int kLinBK = 64;                       // contracted elements per ring stage (128 bytes per row)
constexpr int kLinMaxT = 256;                    // tokens per CTA at most (MMA N)
constexpr int kLinMaxStages = 12;
constexpr int kLinWBytes = kLinBM * 128;         // 16384
constexpr int kLinRingBytes = 196608;            // stages of (weight tile + activation tile); as many as fit, at most 12
constexpr int kLinThreads = 192;
constexpr int kLinSmemBytes = kLinRingBytes + 256 + 1024;
enum { LB_FULL = 0, LB_EMPTY = kLinMaxStages, LB_DONE = 2 * kLinMaxStages };

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// fp32 at the same shared-memory offset in the CTA of rank `rank` of this cluster
__device__ __forceinline__ float ld_cluster_f32(const float* local, uint32_t rank) {
  uint32_t remote;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}

struct LinSm100Params {
  __nv_bfloat16* out[2];   // [M, N_j]
  int N[2];                // output features of job j (multiples of 128)
  int rope_d[2];           // > 0: consecutive blocks of rope_d features are rotated (Eq. 1, d := rope_d)
  int n_jobs, M, S, K, splits;
  int stages;              // ring depth: as many (weight tile + activation box) stages as fit
  int cluster;             // 1: the slices of a tile are the CTAs of one cluster and meet through distributed shared memory
  int x_box_rows;          // rows of the activation box (tokens of a full block, padded to 16); also the row stride of `partial`
  const int32_t* pos_base; // position of token (b, s) = pos_base[b] + pos_shift + s (rotated jobs only)
  int pos_shift;
  float theta;
  float* partial;          // [token block][tile][split][T][128] fp32 (splits > 1)
  int32_t* counters;       // [token block][tile], zero before the launch; left at zero
};

// RoPE of Eq. 1 in the epilogue, rounding and the store.  The even lane of a pair holds the real part, the odd one
// the imaginary part.  Angle = position x theta^(-2l/d), reduced to [-pi, pi] before sine and cosine.  The
// reduction runs in fp32 with the frequency as a (hi, lo) pair and 2*pi as three constants whose products with the
// turn count are formed exactly inside the fused multiply-adds (positions up to 2^20 keep an angle error below
// 1e-5 rad); the double-precision units of this chip are too slow to do it for every (token, pair).  Tokens are
// taken two at a time: the even lane works out the angle of the first, the odd lane that of the second, and they
// swap.
struct LinRope {
  float f_hi = 0.f, f_lo = 0.f;
  int rope_d, S, pos_shift;
  const int32_t* pos_base;
  __device__ LinRope(const LinSm100Params& p, int feature, int rope_d_)
      : rope_d(rope_d_), S(p.S), pos_shift(p.pos_shift), pos_base(p.pos_base) {
    if (rope_d > 0) {
      const double inv_freq = exp2(-2.0 * ((feature % rope_d) >> 1) / rope_d * log2(static_cast<double>(p.theta)));
      f_hi = static_cast<float>(inv_freq);
      f_lo = static_cast<float>(inv_freq - static_cast<double>(f_hi));
    }
  }
  __device__ void sincos_at(int tok, float& sn, float& cs) const {
    const float pos = static_cast<float>(pos_base[tok / S] + pos_shift + tok % S);
    const float a = pos * f_hi;
    const float e = fmaf(pos, f_hi, -a) + pos * f_lo;          // what the rounded product left out
    const float k = rintf(a * 0.15915494309189535f);          // whole turns
    float r = fmaf(-k, 6.28125f, a);                           // 2*pi = 6.28125 + 0.001934051513671875 + 1.2556659146e-6
    r = fmaf(-k, 0.001934051513671875f, r);
    r = fmaf(-k, 1.2556659146e-6f, r) + e;
    sincosf(r, &sn, &cs);
  }
  // values of `feature` for tokens t0 + t and t0 + t + 1 (the second only if has_b): rotate, round, store.
  // Called by all 32 lanes of a warp together.
  __device__ void finish2(__nv_bfloat16* out, int N, int feature, int t0, int t, float va, float vb, bool has_b, int lane) const {
    const float oa = __shfl_xor_sync(0xffffffffu, va, 1), ob = __shfl_xor_sync(0xffffffffu, vb, 1);
    const bool odd = (lane & 1) != 0;
    float re_a = odd ? oa : va, im_a = odd ? va : oa, re_b = odd ? ob : vb, im_b = odd ? vb : ob;
    if (rope_d > 0) {
      float sn = 0.f, cs = 1.f;
      sincos_at(t0 + t + ((odd && has_b) ? 1 : 0), sn, cs);    // even lane: first token; odd lane: second
      const float sn_o = __shfl_xor_sync(0xffffffffu, sn, 1), cs_o = __shfl_xor_sync(0xffffffffu, cs, 1);
      const float sn_a = odd ? sn_o : sn, cs_a = odd ? cs_o : cs;
      const float sn_b = (odd || !has_b) ? sn : sn_o, cs_b = (odd || !has_b) ? cs : cs_o;
      const float ra = re_a * cs_a - im_a * sn_a, ia = im_a * cs_a + re_a * sn_a;
      const float rb = re_b * cs_b - im_b * sn_b, ib = im_b * cs_b + re_b * sn_b;
      re_a = ra; im_a = ia; re_b = rb; im_b = ib;
    }
    if (!odd) {
      *reinterpret_cast<uint32_t*>(out + static_cast<size_t>(t0 + t) * N + feature) = pack_bf16(re_a, im_a);
      if (has_b) *reinterpret_cast<uint32_t*>(out + static_cast<size_t>(t0 + t + 1) * N + feature) = pack_bf16(re_b, im_b);
    }
  }
};

__global__ void __launch_bounds__(kLinThreads, 1)
linear_sm100_kernel(const __grid_constant__ CUtensorMap w_map0, const __grid_constant__ CUtensorMap w_map1,
                    const __grid_constant__ CUtensorMap x_map, const LinSm100Params p, int32_t* dev_status) {
  extern __shared__ unsigned char smem_unaligned[];
  const uint32_t raw = smem_u32(smem_unaligned);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_unaligned + (base - raw);
  const uint32_t bar_base = base + kLinRingBytes;
  auto bar = [&](int i) -> uint32_t { return bar_base + 8 * i; };
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(sm + kLinRingBytes + 8 * (2 * kLinMaxStages + 1));
  const int kLinStages = p.stages;
  const uint32_t kLinStageBytes = kLinWBytes + static_cast<uint32_t>(p.x_box_rows) * 128u;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);
  volatile int* last_flag = abort_flag + 1;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tiles0 = p.N[0] / kLinBM, tiles = tiles0 + (p.n_jobs > 1 ? p.N[1] / kLinBM : 0);
  const int tile = blockIdx.x / p.splits, split = blockIdx.x % p.splits;
  const int job = tile >= tiles0 ? 1 : 0;
  const int f0 = (job ? tile - tiles0 : tile) * kLinBM;       // first output feature of the tile within its job
  const int t0 = blockIdx.y * kLinMaxT;                        // first token of the block
  const int T = min(kLinMaxT, p.M - t0);                       // tokens of this block
  const int TP = (T + 15) & ~15;                               // MMA N
  const int ktiles = p.K / kLinBK;
  const int kt0 = static_cast<int>(static_cast<long long>(split) * ktiles / p.splits);
  const int kt1 = static_cast<int>(static_cast<long long>(split + 1) * ktiles / p.splits);
  const CUtensorMap* w_map = job ? &w_map1 : &w_map0;
  uint32_t tmem_cols = 32;
  while (tmem_cols < static_cast<uint32_t>(TP)) tmem_cols <<= 1;
  pdl_trigger();

  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(w_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&x_map)) : "memory");
    for (int i = 0; i < kLinMaxStages; ++i) { mbar_init(bar(LB_FULL + i), 1); mbar_init(bar(LB_EMPTY + i), 1); }
    mbar_init(bar(LB_DONE), 1);
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  const uint32_t stage_tx = kLinStageBytes;  // rows of the activation box beyond M arrive as zeros

  if (warp == 0) {
    // ======================================================================== TMA producer
    // Weights do not depend on earlier kernels of the stream: the first stages' weight tiles are requested before
    // the dependency wait, their activation tiles after it.
    const int n_it = kt1 - kt0, early = min(n_it, kLinStages);
    for (int i = 0; i < early; ++i) {
      if (elect_one()) {
        mbar_arrive_expect_tx(bar(LB_FULL + i), stage_tx);
        tma_load_2d(base + i * kLinStageBytes, w_map, (kt0 + i) * kLinBK, f0, bar(LB_FULL + i));
      }
      __syncwarp();
    }
    pdl_wait();
    for (int i = 0; i < early; ++i) {
      if (elect_one()) tma_load_2d(base + i * kLinStageBytes + kLinWBytes, &x_map, (kt0 + i) * kLinBK, t0, bar(LB_FULL + i));
      __syncwarp();
    }
    for (int i = early; i < n_it; ++i) {
      const int stage = i % kLinStages, use = i / kLinStages;
      mbar_wait(bar(LB_EMPTY + stage), (use & 1) ^ 1, abort_flag, dev_status);
      if (!*abort_flag && elect_one()) {
        mbar_arrive_expect_tx(bar(LB_FULL + stage), stage_tx);
        tma_load_2d(base + stage * kLinStageBytes, w_map, (kt0 + i) * kLinBK, f0, bar(LB_FULL + stage));
        tma_load_2d(base + stage * kLinStageBytes + kLinWBytes, &x_map, (kt0 + i) * kLinBK, t0, bar(LB_FULL + stage));
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ======================================================================== MMA issuer
    const uint32_t idesc = instr_desc(TP, false);
    const int n_it = kt1 - kt0;
    for (int i = 0; i < n_it; ++i) {
      const int stage = i % kLinStages, use = i / kLinStages;
      mbar_wait(bar(LB_FULL + stage), use & 1, abort_flag, dev_status);
      tc_fence_after();
      const uint64_t a0 = smem_desc(base + stage * kLinStageBytes, 16, 1024);
      const uint64_t b0 = smem_desc(base + stage * kLinStageBytes + kLinWBytes, 16, 1024);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        if (elect_one()) mma_ss(tmem, desc_advance(a0, kk * 32), desc_advance(b0, kk * 32), idesc, (i | kk) ? 1u : 0u);
      }
      if (elect_one()) tc_commit(bar(LB_EMPTY + stage));
      __syncwarp();
    }
    if (elect_one()) tc_commit(bar(LB_DONE));
    __syncwarp();
  } else {
    // ======================================================================== epilogue (warps 2-5)
    const int quad = warp & 3;                                 // tensor-memory lanes 32*quad .. 32*quad+31
    const int fl = quad * 32 + lane;                           // feature of this thread within the tile
    const uint32_t lane_base = static_cast<uint32_t>(quad * 32) << 16;
    const int N = p.N[job], rope_d = p.rope_d[job];
    __nv_bfloat16* out = p.out[job];
    pdl_wait();  // the scratch buffer, the counters and the output may still be in use by earlier kernels
    mbar_wait(bar(LB_DONE), 0, abort_flag, dev_status);
    tc_fence_after();
    LinRope rope(p, f0 + fl, rope_d);
    auto finish2 = [&](int t, float va, float vb, bool has_b) { rope.finish2(out, N, f0 + fl, t0, t, va, vb, has_b, lane); };
    const size_t tile_id = static_cast<size_t>(blockIdx.y) * tiles + tile;
    const size_t slice_elems = static_cast<size_t>(p.x_box_rows) * kLinBM;
    float* my_partial = p.partial + (tile_id * p.splits + split) * slice_elems;
    for (int c = 0; c < TP; c += 32) {
      uint32_t v[32];
      tmem_ld32(tmem + lane_base + c, v);
      tc_wait_ld();
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        if (c + j < T) {  // uniform over the warp
          const bool has_b = c + j + 1 < T;
          if (p.splits == 1) {
            finish2(c + j, __uint_as_float(v[j]), __uint_as_float(v[j + 1]), has_b);
          } else if (p.cluster) {  // the ring is free: every MMA of this CTA has retired
            float* part_s = reinterpret_cast<float*>(sm);
            part_s[(c + j) * kLinBM + fl] = __uint_as_float(v[j]);
            if (has_b) part_s[(c + j + 1) * kLinBM + fl] = __uint_as_float(v[j + 1]);
          } else {
            my_partial[static_cast<size_t>(c + j) * kLinBM + fl] = __uint_as_float(v[j]);
            if (has_b) my_partial[static_cast<size_t>(c + j + 1) * kLinBM + fl] = __uint_as_float(v[j + 1]);
          }
        }
      }
    }
    if (p.splits > 1 && !p.cluster) {
      // the slice that arrives last at the tile's counter adds all slices, in slice order
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (tid == 64) {
        const int old = atomicAdd(p.counters + tile_id, 1);
        *last_flag = (old == p.splits - 1) ? 1 : 0;
        if (old == p.splits - 1) p.counters[tile_id] = 0;  // ready for the next launch
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (*last_flag) {
        __threadfence();
        const float* tile_partial = p.partial + tile_id * p.splits * slice_elems;
        for (int tb = 0; tb < T; tb += 8) {  // eight tokens' slices in flight together
          float acc[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) acc[u] = 0.f;
          for (int s = 0; s < p.splits; ++s) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
              v[u] = tb + u < T ? __ldcg(tile_partial + s * slice_elems + static_cast<size_t>(tb + u) * kLinBM + fl) : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) acc[u] += v[u];
          }
#pragma unroll
          for (int u = 0; u < 8; u += 2)
            if (tb + u < T) finish2(tb + u, acc[u], acc[u + 1], tb + u + 1 < T);
        }
      }
    }
    tc_fence_before();
  }

  if (p.cluster && p.splits > 1) {
    // ---- the slices of the tile meet: every CTA of the cluster has its partial [T][128] in its own shared memory;
    // CTA `split` adds the slices of its share of the tokens in slice order, reading the others' memory directly
    cluster_sync_all();
    if (warp >= 2) {
      const int quad = warp & 3, fl = quad * 32 + lane;
      const int N = p.N[job], rope_d = p.rope_d[job];
      __nv_bfloat16* out = p.out[job];
      const float* part_s = reinterpret_cast<const float*>(sm);
      const int share = (((T + p.splits - 1) / p.splits) + 1) & ~1;  // even, so that token pairs stay together
      const int ts = split * share, te = min(T, ts + share);
      LinRope rope(p, f0 + fl, rope_d);
      for (int tb = ts; tb < te; tb += 8) {
        float acc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) acc[u] = 0.f;
        for (int s = 0; s < p.splits; ++s) {
          float v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) v[u] = tb + u < te ? ld_cluster_f32(part_s + (tb + u) * kLinBM + fl, s) : 0.f;
#pragma unroll
          for (int u = 0; u < 8; ++u) acc[u] += v[u];
        }
#pragma unroll
        for (int u = 0; u < 8; u += 2)
          if (tb + u < te) rope.finish2(out, N, f0 + fl, t0, tb + u, acc[u], acc[u + 1], tb + u + 1 < te, lane);
      }
    }
    cluster_sync_all();  // nobody leaves while its memory may still be read
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

static bool encode_2d(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows) {
  return tensor_map_2d(map, ptr, static_cast<uint64_t>(rows), static_cast<uint32_t>(cols), static_cast<uint32_t>(box_rows), kLinBK);
}

}  // namespace sm100

// Slices of K per 128-feature tile: enough CTAs for every SM to stream weights, at least 4 stages of K per slice.
int linear_sm100_splits(int n_tiles, int K) {
  // one CTA per SM (the ring takes the whole shared memory) and one wave: as many slices as keep tiles x slices
  // within the SM count of a B200, each at least four ring stages long
  const int ktiles = K / sm100::kLinBK;
  int s = 148 / n_tiles;
  if (s > 12) s = 12;
  if (s > ktiles / 4) s = ktiles / 4;
  return s < 1 ? 1 : s;
}

// Where this kernel is used.  Its CTAs take the whole shared memory, so they cannot start while blocks of the kernel
// before them are still resident, and the slices of a tile have to meet at the end; the mma.sync tiles of linear.cu
// have neither cost but re-read the activations once per 32 features.  Measured on the LLaMA-2-7B shape (layer
// step, pipelined) the tcgen05 kernel wins from about 48 tokens on, with long rows of weights (K >= 2048) and at
// least 24 tiles of 128 features: B = 128: 108 -> 70 us for the layer's two large maps; at 16 tokens it is level
// with the mma.sync tiles and at 1 token 13 us slower.
bool linear_sm100_supported(const LinearArgs& a) {
  if (a.n_jobs < 1 || a.n_jobs > 2 || a.M < 48 || a.job[0].K < 2048) return false;
  int tiles = 0;
  for (int j = 0; j < a.n_jobs; ++j) tiles += a.job[j].N / sm100::kLinBM;
  if (tiles < 24) return false;
  for (int j = 0; j < a.n_jobs; ++j) {
    if (a.job[j].N % sm100::kLinBM || a.job[j].K % sm100::kLinBK || a.job[j].K != a.job[0].K || a.job[j].x != a.job[0].x) return false;
    if (a.job[j].rope_d % 2) return false;
  }
  return true;
}

size_t linear_sm100_partial_bytes(int n_tiles, int K, int M) {
  const int splits = linear_sm100_splits(n_tiles, K);
  if (splits == 1) return 0;
  const size_t blocks = (M + sm100::kLinMaxT - 1) / sm100::kLinMaxT;
  const size_t rows = ((M < sm100::kLinMaxT ? M : sm100::kLinMaxT) + 15) & ~15;
  return blocks * n_tiles * splits * rows * sm100::kLinBM * sizeof(float);
}

size_t linear_sm100_counter_bytes(int n_tiles, int M) {
  return static_cast<size_t>((M + sm100::kLinMaxT - 1) / sm100::kLinMaxT) * n_tiles * sizeof(int32_t);
}

cudaError_t launch_linear_sm100(const LinearArgs& a, float* partial, int32_t* counters, int32_t* dev_status,
                                cudaStream_t stream) {
  using namespace sm100;
  LinSm100Params p = {};
  CUtensorMap wmap[2], xmap;
  int tiles = 0;
  for (int j = 0; j < a.n_jobs; ++j) {
    p.out[j] = a.job[j].out; p.N[j] = a.job[j].N; p.rope_d[j] = a.job[j].rope_d;
    if (!encode_2d(&wmap[j], a.job[j].w, a.job[j].N, a.job[j].K, kLinBM)) return cudaErrorInvalidValue;
    tiles += a.job[j].N / kLinBM;
  }
  if (a.n_jobs == 1) wmap[1] = wmap[0];
  const int T = a.M < kLinMaxT ? a.M : kLinMaxT;
  p.x_box_rows = (T + 15) & ~15;
  p.stages = kLinRingBytes / (kLinWBytes + p.x_box_rows * 128);
  if (p.stages > kLinMaxStages) p.stages = kLinMaxStages;
  if (!encode_2d(&xmap, a.job[0].x, a.M, a.job[0].K, p.x_box_rows)) return cudaErrorInvalidValue;
  p.n_jobs = a.n_jobs; p.M = a.M; p.S = a.S; p.K = a.job[0].K;
  p.splits = linear_sm100_splits(tiles, p.K);
  p.pos_base = a.pos_base; p.pos_shift = a.pos_shift; p.theta = a.theta;
  p.partial = partial; p.counters = counters;
  static PerDeviceFlag smem_set;  // zero-initialised; one slot per device
  if (cudaError_t e = ensure_dynamic_smem(linear_sm100_kernel, kLinSmemBytes, smem_set); e != cudaSuccess) return e;
  const int token_blocks = (a.M + kLinMaxT - 1) / kLinMaxT;
  // The K slices of a tile are launched as one thread-block cluster (they are neighbours in blockIdx.x); they then
  // meet through distributed shared memory and need neither the scratch buffer nor the counters.  All clusters have
  // to fit on the device at once (a cluster lives inside one GPC, so fewer fit than SMs / size suggests): the
  // slice count is lowered until they do; if no size from 2 to 8 fits, the wanted count runs through the scratch.
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kLinThreads);
  cfg.dynamicSmemBytes = kLinSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  p.cluster = 0;
  static PerDeviceFlag max_clusters[9];  // co-resident clusters of each size on each device, asked once (0 = not yet)
  const int slot = current_device_slot();
  for (int s = p.splits < 8 ? p.splits : 8; s >= 2 && !p.cluster; --s) {
    attr[1].val.clusterDim.x = s;
    cfg.gridDim = dim3(tiles * s, token_blocks);
    cfg.numAttrs = 2;
    int fit = slot >= 0 ? max_clusters[s].value[slot].load(std::memory_order_acquire) : 0;
    if (fit == 0) {
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, linear_sm100_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = -1; }
      fit = n > 0 ? n : -1;
      if (slot >= 0) max_clusters[s].value[slot].store(fit, std::memory_order_release);
    }
    if (fit >= tiles * token_blocks) { p.cluster = 1; p.splits = s; }
  }
  if (!p.cluster) {
    cfg.gridDim = dim3(tiles * p.splits, token_blocks);
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, linear_sm100_kernel, wmap[0], wmap[1], xmap, p, dev_status);
}

}  // namespace transmla
