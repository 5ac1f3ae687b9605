// Split-KV absorbed-MLA decode (Eq. 9 right, second line) over an FP8 latent cache, r = 512, dR = 64.
//
// Stored row of a token (656 bytes instead of 1152): 512 e4m3 codes of c / scale, 64 bf16 values k^R / scale,
// the fp32 scale, 12 bytes of padding.  (The paper only names FP8; the format is this library's own.)  The kernel
// is the bf16 split-KV kernel with three differences:
//   - scores: the page's codes are the B operand of native FP8 products (kind::f8f6f4, K = 32).  The absorbed
//     queries are split, row by row, into two e4m3 terms q ~ sq * (hi + lo) when they are moved into tensor memory
//     (two terms carry about the 8 bits a bf16 query has); the rope part runs as bf16 products on k^R / scale and
//     q^R / sq.  All of it lands in one accumulator and a score is sq * scale_j times that sum.
//   - products: four more warps turn the codes of a page into scale_j * code as fp16 (the code's fp16 image is exact,
//     the product with the fp16-rounded scale is rounded once more) in a second buffer with the layout the bf16 kernel reads its pages in, and
//     zero-fill the rows beyond the sequence; P is fp16 too (operands of one product must agree in type).
//   - a page's stage goes back to the TMA warp when three parties are done with it: the scores, the converters,
//     and the softmax warps (they read the scales).
// Tensor-memory map: Q hi 0-127, Q lo 128-255 (four codes a column), q^R / sq 256-287, S 288-351, O^T 352-479.
//
// Warp roles: warps 0-3 softmax + epilogue, warp 4 TMA, warp 5 score products, warp 6 PV products, warps 7-10
// converters.  All waits are bounded as in the bf16 kernel.
#include <cuda_fp16.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace transmla {
namespace fp8 {

using namespace sm100;

constexpr int R = 512, DR = 64, K = R + DR;
constexpr int kRowBytes = TRANSMLA_FP8_ROW_BYTES;     // 656
constexpr int kCodeTiles = R / 128;                   // 4 sub-tiles of 64 tokens x 128 codes
constexpr int kSubTileBytes = kPage * 128;            // 8192
constexpr int kOffRope = kCodeTiles * kSubTileBytes;  // 32768: 64 tokens x 64 bf16
constexpr int kOffScale = kOffRope + kSubTileBytes;   // 40960: 64 tokens x 16 bytes (the scale is the first 4)
constexpr int kStageBytes = kOffScale + kPage * 16;   // 41984
constexpr int kStages = 3;
constexpr int kVBytes = 8 * kSubTileBytes;            // 65536: the page's latent part as fp16, 8 sub-tiles of 64 x 64
constexpr int kPBytes = kRowBlock * 128;              // 4096: P[32 rows][64 tokens] fp16
constexpr int kQTileBytes = kRowBlock * 128;          // 4096: one 64-column sub-tile of the 32 query rows (bf16)
constexpr int kQChunks = K / 64;                      // 9
constexpr int kThreads = 352;
constexpr uint32_t kTmemCols = 512;
constexpr int kMetaRing = 16;
enum { ITEM_QUERIES = 1, ITEM_PAGE = 2, ITEM_END = 3 };
constexpr uint32_t kColQhi = 0, kColQlo = 128, kColQr = 256, kColS = 288, kColO = 352;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int kOffStage = 0;
constexpr int kOffV = kStages * kStageBytes;      // 125952 (a multiple of 1024)
constexpr int kOffP = kOffV + kVBytes;            // 2 buffers
constexpr int kOffBar = kOffP + 2 * kPBytes;      // mbarriers (8 bytes each)
constexpr int kOffMisc = kOffBar + 128;
// misc: pmax_s[2][4][32] f32, alpha_s[32] f32, inv_l[32] f32, meta[16] int4, tmem base, abort, ring_done
constexpr int kMiscBytes = 1024 + 128 + 128 + 16 * kMetaRing + 16;
constexpr int kSmemBytes = kOffMisc + kMiscBytes + 1024;  // + slack for the 1024-byte alignment
static_assert(kSmemBytes <= 232448, "shared memory budget");
static_assert(kStageBytes % 1024 == 0 && kQChunks * kQTileBytes <= kStageBytes, "stage layout");

enum { BAR_KV_FULL = 0, BAR_KV_EMPTY = kStages, BAR_Q_READY = 2 * kStages, BAR_S_FULL, BAR_S_FREE, BAR_P_READY0, BAR_P_READY1,
       BAR_PV_DONE0, BAR_PV_DONE1, BAR_V_FULL, BAR_V_EMPTY };

// D[tmem] (+)= A[tmem] * B[smem desc], both operands e4m3 (K = 32 per instruction)
__device__ __forceinline__ void mma_ts_f8(uint32_t d, uint32_t a, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d), "r"(a), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Instruction descriptors: fp32 accumulator, M = 128; e4m3 x e4m3 (both K-major), and fp16 x fp16 with A MN-major.
__host__ __device__ constexpr uint32_t instr_desc_e4m3(int n) {
  return (1u << 4) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
}
__host__ __device__ constexpr uint32_t instr_desc_f16_a_mn(int n) {
  return (1u << 4) | (1u << 15) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
}
// Two floats -> two e4m3 codes (nearest, ties to even, saturating), first argument in the low byte.
__device__ __forceinline__ uint32_t pack_e4m3x2(float lo, float hi) {
  uint16_t r;
  asm volatile("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
// Two e4m3 codes (low 16 bits) -> two fp16 values, exactly.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t v) {
  uint32_t r;
  asm volatile("{\n.reg .b16 t;\nmov.b32 {t, _}, %1;\ncvt.rn.f16x2.e4m3x2 %0, t;\n}" : "=r"(r) : "r"(v));
  return r;
}
__device__ __forceinline__ __half2 as_half2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
decode_fp8_kernel(const __grid_constant__ CUtensorMap cache_map, const __grid_constant__ CUtensorMap scale_map,
                  const __grid_constant__ CUtensorMap q_map,
                    const int32_t* page_table, const int32_t* seqlens,
                    const int32_t* cum, const int32_t* plan, float* partial_o,
                    float* partial_lse, int32_t* dev_status, int S, int H, int num_pages, int max_pages,
                    float scale_log2, int B, int dynamic, int32_t* next) {
  extern __shared__ unsigned char smem_unaligned[];
  const uint32_t raw = smem_u32(smem_unaligned);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_unaligned + (base - raw);
  float* pmax_s = reinterpret_cast<float*>(sm + kOffMisc);         // [2][4][32]: per page parity, warp, row
  float* alpha_s = pmax_s + 256;                                   // [32]
  float* inv_l = alpha_s + 32;                                     // [32]
  int4* meta = reinterpret_cast<int4*>(inv_l + 32);                // [kMetaRing]: what each ring item is
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(meta + kMetaRing);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);
  volatile int* ring_done = abort_flag + 1;
  auto bar = [&](int i) -> uint32_t { return base + kOffBar + 8 * i; };

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int part = blockIdx.x, rb = blockIdx.y;
  const int SH = S * H;
  pdl_trigger();

  if (tid == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&cache_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&q_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&scale_map)) : "memory");
    for (int i = 0; i < kStages; ++i) { mbar_init(bar(BAR_KV_FULL + i), 1); mbar_init(bar(BAR_KV_EMPTY + i), 3); }
    mbar_init(bar(BAR_V_FULL), 1);
    mbar_init(bar(BAR_V_EMPTY), 1);
    mbar_init(bar(BAR_Q_READY), 128);
    mbar_init(bar(BAR_S_FULL), 1);
    mbar_init(bar(BAR_S_FREE), 128);
    mbar_init(bar(BAR_P_READY0), 128);
    mbar_init(bar(BAR_P_READY1), 128);
    mbar_init(bar(BAR_PV_DONE0), 1);
    mbar_init(bar(BAR_PV_DONE1), 1);
    *abort_flag = 0;
    *ring_done = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_base_s)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_base_s;
  pdl_wait();  // the plan, the absorbed queries and the appended cache rows come from the kernel before this one
  const int4 pl = reinterpret_cast<const int4*>(plan)[part];
  const bool has_home = pl.y > pl.x;

  if (has_home) {
    if (warp == 4) {
      // ======================================================================== TMA producer
      // The ring carries, per segment, one item with the 32 absorbed query rows followed by the segment's pages,
      // and one closing item when the CTA has nothing more to do.  What an item is goes into `meta`.
      int g = 0;  // ring items issued by this CTA so far
      const uint64_t stream_policy = l2_evict_first_policy();
      auto acquire = [&](int gi) -> uint32_t {  // waits for the stage of ring item gi; returns its index
        const int stage = gi % kStages, use = gi / kStages;
        mbar_wait(bar(BAR_KV_EMPTY + stage), (use & 1) ^ 1, abort_flag, dev_status);
        return stage;
      };
      auto issue_queries = [&](int b, int slot_code, int L) {
        const uint32_t stage = acquire(g);
        if (!*abort_flag && elect_one()) {
          meta[g & (kMetaRing - 1)] = make_int4(ITEM_QUERIES, b, slot_code, L);
          mbar_arrive_expect_tx(bar(BAR_KV_FULL + stage), kQChunks * kQTileBytes);
          const uint32_t dst = base + kOffStage + stage * kStageBytes;
#pragma unroll
          for (int c = 0; c < kQChunks; ++c)
            tma_load_2d(dst + c * kQTileBytes, &q_map, c * 64, b * SH + rb * kRowBlock, bar(BAR_KV_FULL + stage));
        }
        __syncwarp();
        ++g;
      };
      auto issue_page = [&](int b, int pj, bool first, bool last) {
        int idx = page_table[static_cast<size_t>(b) * max_pages + pj];
        const bool ok = idx >= 0 && idx < num_pages;
        if (!ok) { if (lane == 0) set_status(dev_status, TRANSMLA_DEV_BAD_PAGE); idx = 0; }
        const uint32_t stage = acquire(g);
        if (!*abort_flag && elect_one()) {
          meta[g & (kMetaRing - 1)] = make_int4(ITEM_PAGE, pj, ok ? 1 : 0, (first ? 1 : 0) | (last ? 2 : 0));
          // the pool as bytes [num_pages * 64 rows, 656]: four boxes of 128 codes, one of 128 bytes (64 bf16) and,
          // through a map without swizzle, one of 16 bytes that holds the scale
          mbar_arrive_expect_tx(bar(BAR_KV_FULL + stage), kStageBytes);
          const uint32_t dst = base + kOffStage + stage * kStageBytes;
#pragma unroll
          for (int c = 0; c <= kCodeTiles; ++c)
            tma_load_2d_hint(dst + c * kSubTileBytes, &cache_map, c * 128, idx * kPage, bar(BAR_KV_FULL + stage), stream_policy);
          tma_load_2d_hint(dst + kOffScale, &scale_map, R + 2 * DR, idx * kPage, bar(BAR_KV_FULL + stage), stream_policy);
        }
        __syncwarp();
        ++g;
      };
      // ---- the partition's sequences in turn
      // Page-table entries [lo, hi) of sequence b are asked into L1 ahead of their use (one 128-byte line per lane
      // and round), so that the look-up in front of every page load does not cost a trip to L2.
      auto prefetch_table = [&](int b, int lo, int hi) {
        const int32_t* row = page_table + static_cast<size_t>(b) * max_pages;
        for (int i = (lo & ~31) + lane * 32; i < hi; i += 32 * 32)
          asm volatile("prefetch.global.L1 [%0];" ::"l"(row + max(i, lo)));
      };
      // The last sequence in which this partition owns pages: there it claims until the counter runs dry.  In the
      // sequences before it (a partition that straddles two or more) it takes no more pages than the plan gave it,
      // so that every sequence gets the share of CTA time that the plan meant it to have.
      int last_home = pl.w;
      if (dynamic) {
        const int cw = cum[pl.w], cw1 = cum[pl.w + 1];
        if (min(pl.y, cw1) <= max(pl.x, cw + kSegCost)) --last_home;
      }
      for (int b = pl.z; b <= pl.w; ++b) {
        const int cb = cum[b], cb1 = cum[b + 1];  // one round trip for the three of them
        const int L = clamped_len(seqlens[b], max_pages, nullptr);  // the plan block has already reported a bad length
        const int c0s = cb + kSegCost;  // slot of page 0 of sequence b
        const int pg_lo = max(pl.x, c0s) - c0s, pg_hi = min(pl.y, cb1) - c0s;
        if (pg_hi <= pg_lo) continue;
        if (!dynamic) {  // exactly the plan's range
          prefetch_table(b, pg_lo, pg_hi);
          issue_queries(b, part + b, L);
          for (int pj = pg_lo; pj < pg_hi; ++pj) issue_page(b, pj, pj == pg_lo, pj == pg_hi - 1);
          continue;
        }
        // Pages of sequence b from its counter until it runs dry.  Three are claimed in one go (one atomic
        // instruction, lanes 0..2) so that the stages fill at once.  After that the next two page numbers are
        // always in hand and the claim behind them is in flight while a page waits for its stage, which keeps the
        // counter's round trip off the critical path and tells at issue time whether a page is the segment's
        // last one: it is exactly when the claim behind it is past the end (claims only grow).
        const int n_b = cb1 - c0s;
        int32_t* counter = next + static_cast<size_t>(rb) * B + b;
        int left = b < last_home ? pg_hi - pg_lo : 0x7fffffff;  // claims this partition may still make here
        const int take = min(kStages, left);
        left -= take;
        int head = 0x7fffffff;
        if (lane < take) head = atomicAdd(counter, 1);
        prefetch_table(b, 0, n_b);  // in flight together with the claim
        int c0 = __shfl_sync(0xffffffffu, head, 0), c1 = __shfl_sync(0xffffffffu, head, 1), c2 = __shfl_sync(0xffffffffu, head, 2);
        { int t; if (c0 > c1) { t = c0; c0 = c1; c1 = t; } if (c1 > c2) { t = c1; c1 = c2; c2 = t; } if (c0 > c1) { t = c0; c0 = c1; c1 = t; } }
        if (c0 >= n_b) {  // the others have taken everything: the combine still expects a partial from this slot
          if (rb * kRowBlock + lane < SH) partial_lse[static_cast<size_t>(part + b) * SH + rb * kRowBlock + lane] = -INFINITY;
          continue;
        }
        issue_queries(b, part + b, L);
        bool first = true;
        while (c0 < n_b) {
          int pend = 0x7fffffff;
          const bool ahead = c2 < n_b && left > 0;
          if (ahead) { --left; if (lane == 0) pend = atomicAdd(counter, 1); }
          issue_page(b, c0, first, c1 >= n_b);
          first = false;
          c0 = c1;
          c1 = c2;
          c2 = ahead ? __shfl_sync(0xffffffffu, pend, 0) : 0x7fffffff;
        }
      }
      {  // closing item
        const uint32_t stage = acquire(g);
        if (elect_one()) {
          meta[g & (kMetaRing - 1)] = make_int4(ITEM_END, 0, 0, 0);
          mbar_arrive(bar(BAR_KV_FULL + stage));
        }
        __syncwarp();
      }
    } else if (warp == 5) {
      // ======================================================================== MMA issuer, scores
      // Follows the ring: skips query items (the softmax warps move them to tensor memory and report through
      // Q_READY, which also tells when the ring has ended) and runs the score products of a page as soon as it has
      // landed: per 32 codes two e4m3 products (the queries' high and low term) on the page's codes as they came
      // from memory, then four bf16 products on the rope part, all into one accumulator.
      constexpr uint32_t idesc_f8 = instr_desc_e4m3(kPage);
      constexpr uint32_t idesc_rope = instr_desc(kPage, false);
      int g = 0, n = 0, seg = 0;  // ring items, pages, segments handled so far
      while (true) {
        // a segment begins (or the ring ends): the softmax warps say which
        mbar_wait(bar(BAR_Q_READY), seg & 1, abort_flag, dev_status);
        ++seg;
        if (__any_sync(0xffffffffu, *abort_flag != 0) || *ring_done != 0) break;
        if (elect_one()) mbar_arrive(bar(BAR_KV_EMPTY + g % kStages));  // this warp's share of handing the query item back
        __syncwarp();
        ++g;
        while (true) {
          const int stage = g % kStages, use = g / kStages;
          mbar_wait(bar(BAR_KV_FULL + stage), use & 1, abort_flag, dev_status);
          const int4 m = meta[g & (kMetaRing - 1)];
          if (n > 0) mbar_wait(bar(BAR_S_FREE), (n - 1) & 1, abort_flag, dev_status);
          tc_fence_after();
          const uint64_t k0 = smem_desc(base + kOffStage + stage * kStageBytes, 16, 1024);
#pragma unroll
          for (int c = 0; c < kCodeTiles; ++c) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const uint64_t bd = desc_advance(k0, c * kSubTileBytes + kk * 32);
              if (elect_one()) mma_ts_f8(tmem + kColS, tmem + kColQhi + c * 32 + kk * 8, bd, idesc_f8, (c | kk) ? 1u : 0u);
              if (elect_one()) mma_ts_f8(tmem + kColS, tmem + kColQlo + c * 32 + kk * 8, bd, idesc_f8, 1u);
            }
          }
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            if (elect_one())
              mma_ts(tmem + kColS, tmem + kColQr + kk * 8, desc_advance(k0, kOffRope + kk * 32), idesc_rope, 1u);
          }
          if (elect_one()) {
            tc_commit(bar(BAR_KV_EMPTY + stage));  // one of the three parties that hand the stage back
            tc_commit(bar(BAR_S_FULL));
          }
          __syncwarp();
          ++g; ++n;
          if ((m.w & 2) != 0 || m.x != ITEM_PAGE || __any_sync(0xffffffffu, *abort_flag != 0)) break;
        }
      }
    } else if (warp == 6) {
      // ======================================================================== MMA issuer, products
      // O^T += V^T P^T for a page as soon as its probabilities and its fp16 copy are there.  It follows the ring only
      // to learn where segments begin and end.
      constexpr uint32_t idesc_pv = instr_desc_f16_a_mn(kRowBlock);
      int g = 0, n = 0, seg = 0;
      while (true) {
        mbar_wait(bar(BAR_Q_READY), seg & 1, abort_flag, dev_status);
        ++seg;
        if (__any_sync(0xffffffffu, *abort_flag != 0) || *ring_done != 0) break;
        ++g;
        while (true) {
          const int stage = g % kStages, use = g / kStages;
          mbar_wait(bar(BAR_KV_FULL + stage), use & 1, abort_flag, dev_status);
          const int4 m = meta[g & (kMetaRing - 1)];
          mbar_wait(bar(BAR_V_FULL), n & 1, abort_flag, dev_status);
          mbar_wait(bar(BAR_P_READY0 + (n & 1)), (n >> 1) & 1, abort_flag, dev_status);
          tc_fence_after();
          const uint64_t a0 = smem_desc(base + kOffV, kSubTileBytes, 1024);
          const uint64_t b0 = smem_desc(base + kOffP + (n & 1) * kPBytes, 16, 1024);
          const uint32_t acc0 = (m.w & 1) != 0 ? 0u : 1u;  // the segment's first page starts the accumulator afresh
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              if (elect_one())
                mma_ss(tmem + kColO + t * 32, desc_advance(a0, (2 * t) * kSubTileBytes + kk * 2048),
                       desc_advance(b0, kk * 32), idesc_pv, kk == 0 ? acc0 : 1u);
            }
          }
          if (elect_one()) {
            tc_commit(bar(BAR_V_EMPTY));
            tc_commit(bar(BAR_PV_DONE0 + (n & 1)));
          }
          __syncwarp();
          ++g; ++n;
          if ((m.w & 2) != 0 || m.x != ITEM_PAGE || __any_sync(0xffffffffu, *abort_flag != 0)) break;
        }
      }
    } else if (warp >= 7) {
      // ======================================================================== converters (warps 7-10)
      // Per page: scale_j * code -> fp16 into the V buffer, in the layout of a bf16 page's latent sub-tiles (64
      // tokens x 64 columns, 128-byte rows, 128-byte swizzle); rows beyond the sequence become zeros.  They hand a
      // query item back too (their third of it), so that no stage can be
      // used twice before they have seen it.
      const int c = tid - 224;
      int g = 0, n = 0, L_seg = 0;
      while (true) {
        const int stage = g % kStages, use = g / kStages;
        mbar_wait(bar(BAR_KV_FULL + stage), use & 1, abort_flag, dev_status);
        const int4 m = meta[g & (kMetaRing - 1)];
        int stop;
        asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 q, %1, 0;\nbar.red.or.pred p, 3, 128, q;\nselp.s32 %0, 1, 0, p;\n}"
                     : "=r"(stop) : "r"(static_cast<int>(*abort_flag != 0 || m.x == ITEM_END)) : "memory");
        if (stop) break;
        if (m.x == ITEM_QUERIES) {
          L_seg = m.w;  // the sequence's length, for the pages that follow
          if (c == 0) mbar_arrive(bar(BAR_KV_EMPTY + stage));
          ++g;
          continue;
        }
        if (n > 0) mbar_wait(bar(BAR_V_EMPTY), (n - 1) & 1, abort_flag, dev_status);
        const unsigned char* st = sm + kOffStage + stage * kStageBytes;
        unsigned char* vb = sm + kOffV;
        const int valid = m.z != 0 ? min(kPage, L_seg - m.y * kPage) : 0;  // rows [valid, 64) must read as zero
        // 16 rounds; in a round a warp takes 4 consecutive rows x the 8 16-byte chunks of one 128-code sub-tile, so that
        // its loads sweep whole 128-byte rows (the swizzle only permutes the chunks inside a row)
#pragma unroll 1
        for (int rblk = 0; rblk < 4; ++rblk) {
          const int r = rblk * 16 + (c >> 3), j = c & 7;
          const __half2 sc2 = __half2half2(__float2half_rn(r < valid ? *reinterpret_cast<const float*>(st + kOffScale + r * 16) : 0.f));
#pragma unroll
          for (int ct = 0; ct < kCodeTiles; ++ct) {  // code sub-tile: columns 128 ct .. 128 ct + 127
            const uint4 x = *reinterpret_cast<const uint4*>(st + ct * kSubTileBytes + r * 128 + ((j ^ (r & 7)) << 4));
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            uint32_t o[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const __half2 lo = __hmul2(as_half2(e4m3x2_to_f16x2(w[k] & 0xffffu)), sc2);
              const __half2 hi = __hmul2(as_half2(e4m3x2_to_f16x2(w[k] >> 16)), sc2);
              o[2 * k] = r < valid ? as_u32(lo) : 0u;  // (a NaN code times a zero scale would still be NaN)
              o[2 * k + 1] = r < valid ? as_u32(hi) : 0u;
            }
            // columns 128 ct + 16 j .. + 15 -> V sub-tile 2 ct + j / 4, 16-byte chunks 2 (j % 4) and 2 (j % 4) + 1
            unsigned char* dst = vb + (2 * ct + (j >> 2)) * kSubTileBytes + r * 128;
            const int ch = 2 * (j & 3);
            *reinterpret_cast<uint4*>(dst + ((ch ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            *reinterpret_cast<uint4*>(dst + (((ch + 1) ^ (r & 7)) << 4)) = make_uint4(o[4], o[5], o[6], o[7]);
          }
        }
        fence_proxy_async();
        asm volatile("bar.sync 3, 128;" ::: "memory");
        if (c == 0) {
          mbar_arrive(bar(BAR_V_FULL));
          mbar_arrive(bar(BAR_KV_EMPTY + stage));
        }
        ++g; ++n;
      }
    } else if (warp < 4) {
      // ======================================================================== softmax + epilogue (warps 0-3)
      const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
      const int my_row = rb * kRowBlock + lane;  // query row of this thread (same in all four replicas)
      int g = 0, n = 0;  // ring items and pages handled so far
      float sq_row = 1.f;  // scale of this thread's query row (see open_segment)
      // Looks at ring item g.  Queries: moves the 32 rows from shared memory (swizzled sub-tiles of 32 rows x
      // 128 bytes) to this warp's replica in tensor memory, 32 columns (64 elements) at a time, hands the stage
      // back and returns the item's description.  Closing item: marks the ring as ended.  Either way the MMA
      // warp is told through Q_READY.  All 128 threads take the same path (the description is the same for all).
      auto open_segment = [&]() -> int4 {
        const int stage = g % kStages, use = g / kStages;
        mbar_wait(bar(BAR_KV_FULL + stage), use & 1, abort_flag, dev_status);
        int4 m = meta[g & (kMetaRing - 1)];
        int aborted;
        asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 q, %1, 0;\nbar.red.or.pred p, 1, 128, q;\nselp.s32 %0, 1, 0, p;\n}"
                     : "=r"(aborted) : "r"(*abort_flag) : "memory");
        if (aborted || m.x != ITEM_QUERIES) {
          m.x = ITEM_END;
          if (tid == 0) *ring_done = 1;
          asm volatile("bar.sync 1, 128;" ::: "memory");
          mbar_arrive(bar(BAR_Q_READY));
          return m;
        }
        const unsigned char* qrow = sm + kOffStage + stage * kStageBytes + lane * 128;
        // This row's absorbed query q (512 bf16): q ~ sq * (hi + lo) with hi, lo e4m3 and sq = max|q| / 448.
        float amax = 0.f;
#pragma unroll 1
        for (int c = 0; c < kCodeTiles * 2; ++c) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(qrow + c * kQTileBytes + ((j ^ (lane & 7)) << 4));
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) amax = fmaxf(amax, fmaxf(fabsf(bf16_lo(w[k])), fabsf(bf16_hi(w[k]))));
          }
        }
        sq_row = amax > 0.f ? amax * (1.f / 448.f) : 1.f;
        const float inv_sq = 1.f / sq_row;
#pragma unroll 1
        for (int c = 0; c < kCodeTiles * 2; ++c) {  // 64 query values -> 16 columns of four codes, high and low term
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(qrow + c * kQTileBytes + ((j ^ (lane & 7)) << 4));
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            uint32_t h2[4], l2[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const float a = bf16_lo(w[k]) * inv_sq, b = bf16_hi(w[k]) * inv_sq;
              h2[k] = pack_e4m3x2(a, b);
              const float2 back = __half22float2(as_half2(e4m3x2_to_f16x2(h2[k])));
              l2[k] = pack_e4m3x2(a - back.x, b - back.y);
            }
            hi[2 * j] = h2[0] | (h2[1] << 16); hi[2 * j + 1] = h2[2] | (h2[3] << 16);
            lo[2 * j] = l2[0] | (l2[1] << 16); lo[2 * j + 1] = l2[2] | (l2[3] << 16);
          }
          tmem_st16(tmem + lane_base + kColQhi + c * 16, hi);
          tmem_st16(tmem + lane_base + kColQlo + c * 16, lo);
        }
        {  // the rope part, divided by sq, stays bf16
          uint32_t v[32];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 x = *reinterpret_cast<const uint4*>(qrow + 8 * kQTileBytes + ((j ^ (lane & 7)) << 4));
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) v[4 * j + k] = pack_bf16(bf16_lo(w[k]) * inv_sq, bf16_hi(w[k]) * inv_sq);
          }
          tmem_st32(tmem + lane_base + kColQr, v);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_Q_READY));
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (tid == 0) mbar_arrive(bar(BAR_KV_EMPTY + stage));  // one of three: the score warp and the converters see it too
        ++g;
        return m;
      };
      int4 seg_meta = open_segment();
      while (seg_meta.x == ITEM_QUERIES) {
        const int L = seg_meta.w;
        float* o_rows = partial_o + (static_cast<size_t>(seg_meta.z) * SH + rb * kRowBlock) * R;
        float* lse_rows = partial_lse + static_cast<size_t>(seg_meta.z) * SH + rb * kRowBlock;
        const int n_vis = my_row < SH ? L - (S - 1 - my_row / H) : 0;

        float m_used = -INFINITY, l_run = 0.f;
        bool more = true;
        while (more) {
          const int stage = g % kStages;
          mbar_wait(bar(BAR_KV_FULL + stage), (g / kStages) & 1, abort_flag, dev_status);
          const int4 pm = meta[g & (kMetaRing - 1)];
          const int pj = pm.y;
          const bool page_ok = pm.z != 0;
          const int tok_end = page_ok ? n_vis - pj * kPage : 0;           // tokens [0, tok_end) of the page are visible
          const bool first = (pm.w & 1) != 0;
          const int buf = n & 1;

          mbar_wait(bar(BAR_S_FULL), n & 1, abort_flag, dev_status);
          tc_fence_after();
          uint32_t sq[16];  // this warp's 16 tokens of its row
          tmem_ld16(tmem + lane_base + kColS + warp * 16, sq);
          tc_wait_ld();
          tc_fence_before();
          mbar_arrive(bar(BAR_S_FREE));
          {
            // a score is sq (row) * scale_j (token) * the accumulated sum; tokens beyond the visible range are dropped
            // by selection, so whatever their scale holds does not matter
            const unsigned char* scl = sm + kOffStage + stage * kStageBytes + kOffScale + warp * 16 * 16;
            const float row_factor = sq_row * scale_log2;
            float pmax = -INFINITY;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float x = warp * 16 + j < tok_end
                                  ? __uint_as_float(sq[j]) * (row_factor * *reinterpret_cast<const float*>(scl + j * 16))
                                  : -INFINITY;
              sq[j] = __float_as_uint(x);
              pmax = fmaxf(pmax, x);
            }
            pmax_s[(buf * 4 + warp) * 32 + lane] = pmax;
          }
          // one barrier per page: the row maxima meet, and all 128 threads learn together whether the CTA gave up
          int aborted;
          asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 q, %1, 0;\nbar.red.or.pred p, 1, 128, q;\nselp.s32 %0, 1, 0, p;\n}"
                       : "=r"(aborted) : "r"(*abort_flag) : "memory");
          more = (pm.w & 2) == 0 && pm.x == ITEM_PAGE && !aborted;
          if (tid == 0) mbar_arrive(bar(BAR_KV_EMPTY + stage));  // the scales have been read: the softmax warps' share
          const float rowmax = fmaxf(fmaxf(pmax_s[(buf * 4 + 0) * 32 + lane], pmax_s[(buf * 4 + 1) * 32 + lane]),
                                     fmaxf(pmax_s[(buf * 4 + 2) * 32 + lane], pmax_s[(buf * 4 + 3) * 32 + lane]));
          // Lazy rescale: the reference maximum only moves when some row's new maximum exceeds it by 2^8.  Every
          // warp holds all 32 rows, so the four warps take the same decision without talking to each other.
          float alpha = 1.f;
          bool rescale = false;
          if (first) {
            m_used = rowmax;
          } else {
            rescale = __any_sync(0xffffffffu, rowmax > m_used + 8.f);
            if (rescale) {
              const float m_new = fmaxf(m_used, rowmax);
              alpha = (m_new == -INFINITY) ? 1.f : exp2f(m_used - m_new);
              m_used = m_new;
              l_run *= alpha;
            }
          }
          const float m_ref = m_used;

          // ---- probabilities of tokens 16*warp .. 16*warp+15
          uint32_t pk[8];
          float psum = 0.f;
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const int t0 = warp * 16 + j;
            const float p0 = t0 < tok_end ? exp2f(__uint_as_float(sq[j]) - m_ref) : 0.f;
            const float p1 = t0 + 1 < tok_end ? exp2f(__uint_as_float(sq[j + 1]) - m_ref) : 0.f;
            psum += p0 + p1;
            pk[j >> 1] = pack_f16(p0, p1);
          }
          l_run += psum;

          // ---- P buffer `buf` is free once PV of CTA page n-2 is done
          if (n >= 2) mbar_wait(bar(BAR_PV_DONE0 + buf), ((n >> 1) - 1) & 1, abort_flag, dev_status);
          {
            unsigned char* prow = sm + kOffP + buf * kPBytes + lane * 128;
            const int c0w = 2 * warp, sw = lane & 7;
            *reinterpret_cast<uint4*>(prow + ((c0w ^ sw) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            *reinterpret_cast<uint4*>(prow + (((c0w + 1) ^ sw) << 4)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
          }
          // ---- rescale O^T by alpha (columns = query rows) once the previous PV has landed
          if (rescale) {
            if (warp == 0) alpha_s[lane] = alpha;
            asm volatile("bar.sync 1, 128;" ::: "memory");  // a later rescale is at least one page barrier away
            if (n >= 1) mbar_wait(bar(BAR_PV_DONE0 + ((n - 1) & 1)), ((n - 1) >> 1) & 1, abort_flag, dev_status);
            tc_fence_after();
#pragma unroll 1
            for (int t = 0; t < 4; ++t) {
              uint32_t ov[32];
              tmem_ld32(tmem + lane_base + kColO + t * 32, ov);
              tc_wait_ld();
#pragma unroll
              for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha_s[j]);
              tmem_st32(tmem + lane_base + kColO + t * 32, ov);
            }
            tc_wait_st();
          }
          fence_proxy_async();
          tc_fence_before();
          mbar_arrive(bar(BAR_P_READY0 + buf));
          ++g; ++n;
        }

        // ---- epilogue of the segment: wait for the last PV, normalise, store O (transposed back) and lse.
        // The row sums meet in the half of pmax_s that the last page did not use (its readers are behind the
        // last page's barrier; the next page writes it only after the barrier at the end of this epilogue).
        float* l_part = pmax_s + (n & 1) * 128;
        l_part[warp * 32 + lane] = l_run;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const float l_tot = l_part[lane] + l_part[32 + lane] + l_part[64 + lane] + l_part[96 + lane];
        if (warp == 0) {
          inv_l[lane] = l_tot > 0.f ? 1.f / l_tot : 0.f;
          if (my_row < SH) lse_rows[lane] = l_tot > 0.f ? (m_used + log2f(l_tot)) * kLn2 : -INFINITY;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        // The queries of the next segment go to tensor memory now (every QK^T of this segment has completed), so
        // that its first QK^T runs while this segment's result is written out.
        seg_meta = open_segment();
        const int n_last = n - 1;
        mbar_wait(bar(BAR_PV_DONE0 + (n_last & 1)), (n_last >> 1) & 1, abort_flag, dev_status);
        tc_fence_after();
        float* dst = o_rows + warp * 32 + lane;
#pragma unroll 1
        for (int t = 0; t < 4; t += 2) {  // two 128-row tiles per round trip to tensor memory
          uint32_t ov[64];
          tmem_ld32(tmem + lane_base + kColO + t * 32, ov);
          tmem_ld32(tmem + lane_base + kColO + (t + 1) * 32, ov + 32);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (rb * kRowBlock + j < SH) {
              const float sc = inv_l[j];
              dst[static_cast<size_t>(j) * R + t * 128] = __uint_as_float(ov[j]) * sc;
              dst[static_cast<size_t>(j) * R + (t + 1) * 128] = __uint_as_float(ov[32 + j]) * sc;
            }
          }
        }
        tc_fence_before();
        asm volatile("bar.sync 1, 128;" ::: "memory");  // inv_l and the row sums are reused by the next segment
      }
    }
  }

  // ---- teardown: everyone arrives, tensor memory is returned
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------- host
}  // namespace fp8

bool decode_fp8_supported(const transmla_params_t& p) {
  return p.kv_lora_rank == fp8::R && p.qk_rope_dim == fp8::DR && p.q_len * p.num_heads <= 1024;
}

cudaError_t launch_decode_fp8(const transmla_params_t& p, int G, const __nv_bfloat16* q_hat, const void* cache_fp8,
                              const int32_t* page_table, const int32_t* seqlens, const int32_t* cum, const int32_t* plan,
                              float* partial_o, float* partial_lse, int32_t* dev_status, cudaStream_t stream) {
  using namespace fp8;
  // The pool as bytes [num_pages * 64 rows, 656]: boxes of 64 rows x 128 bytes with the 128-byte swizzle (codes and
  // rope part), and of 64 rows x 16 bytes without swizzle (scales).  The absorbed queries as in the bf16 kernel.
  CUtensorMap map, smap, qmap;
  const int SH = p.q_len * p.num_heads;
  const uint64_t rows = static_cast<uint64_t>(p.num_pages) * kPage;
  if (!tensor_map_2d(&map, cache_fp8, rows, kRowBytes, kPage, 128, TMAP_U8_SW128) ||
      !tensor_map_2d(&smap, cache_fp8, rows, kRowBytes, kPage, 16, TMAP_U8_PLAIN) ||
      !tensor_map_2d(&qmap, q_hat, static_cast<uint64_t>(p.batch) * SH, K, kRowBlock))
    return cudaErrorInvalidValue;
  static PerDeviceFlag smem_set;
  if (cudaError_t e = ensure_dynamic_smem(decode_fp8_kernel, kSmemBytes, smem_set); e != cudaSuccess) return e;
  dim3 grid(G, (SH + kRowBlock - 1) / kRowBlock);
  int32_t* next = const_cast<int32_t*>(cum) + 3 * p.batch + 1;  // page counters, zeroed by the plan
  return launch_pdl(decode_fp8_kernel, grid, dim3(kThreads), static_cast<size_t>(kSmemBytes), stream, map, smap, qmap,
                    page_table, seqlens, cum, plan, partial_o, partial_lse, dev_status, p.q_len, p.num_heads,
                    p.num_pages, p.max_pages_per_seq, p.softmax_scale * kLog2e, p.batch, dynamic_claims(p, G) ? 1 : 0, next);
}

}  // namespace transmla
