// Plan, absorb, append and combine kernels of the absorbed-MLA decode step.
//
// These touch a few MB (weights, queries, split partials) against the hundreds of MB the split-KV
// kernel streams.  They are small GEMMs with M = number of query rows or new tokens, latency bound
// rather than bandwidth bound, so they run on mma.sync tensor-core tiles, keep many independent
// 16-byte loads in flight, and are fused into as few launches as the data dependencies allow: one
// "prologue" launch holds the append blocks, the absorb blocks and the plan block.
//
// 16-byte operand loads: a lane (g, t) of an m16n8k16 tile needs k = 2t, 2t+1, 2t+8, 2t+9 of its row.
// A dot product does not care in which order k is visited as long as both operands agree, so both
// sides load the 8 consecutive elements 8t .. 8t+7 of a 32-wide k window with one uint4 and feed words
// (x, y) to one MMA and (z, w) to the next.  Where one operand comes from shared memory instead, it
// is stored there in the matching order (kperm below).
#include "append_block.cuh"
#include "common.cuh"
#include "skinny_gemm.cuh"

namespace transmla {

// Position, inside its 32-wide window, at which element p must sit in shared memory so that ldmatrix
// hands out the fragment that pairs with a uint4 global load of the other operand.
__device__ __forceinline__ int kperm(int p) { return ((p & 7) >> 1) * 8 + (p >> 3) * 2 + (p & 1); }

// ------------------------------------------------------------------------------------------------
// Split plan.  Every non-empty sequence owns ceil(L_b/P) page slots preceded by kSegCost virtual slots (the
// price of opening a sequence); cum[b] = slots before sequence b; partition i owns slots
// [floor(i*T/G), floor((i+1)*T/G)); plan row = (begin, end, sequence of first slot, of last slot).
// One block of 256 threads; the scan runs in chunks of 256 sequences; the prefix sums are kept in
// shared memory (when they fit) for the binary searches.
// ------------------------------------------------------------------------------------------------
constexpr int kPlanSmemSeqs = 4096;

__device__ __forceinline__ int seq_of_page(const int32_t* cum, int B, int x) {
  // the b in [0, B) with cum[b] <= x < cum[b+1]  ==  (first index with cum > x) - 1
  int lo = 0, hi = B + 1;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (cum[mid] > x) hi = mid; else lo = mid + 1;
  }
  return lo - 1;
}

__device__ void plan_block(const int32_t* seqlens, int B, int G, int RB, int max_pages, int32_t* cum, int32_t* plan,
                           int32_t* dev_status, unsigned char* smem_raw) {
  __shared__ int warp_sums[8];
  __shared__ int carry;
  int32_t* cum_s = reinterpret_cast<int32_t*>(smem_raw);  // [B+1] when B < kPlanSmemSeqs
  const bool in_smem = B < kPlanSmemSeqs;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  if (tid == 0) { carry = 0; cum[0] = 0; if (in_smem) cum_s[0] = 0; }
  __syncthreads();
  for (int base = 0; base < B; base += 256) {
    const int b = base + tid;
    int n = 0;
    if (b < B) { const int L = clamped_len(seqlens[b], max_pages, dev_status); n = L > 0 ? (L + kPage - 1) / kPage + kSegCost : 0; }
    int v = n;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += t; }
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    const int incl = v + before;
    if (b < B) { cum[b + 1] = incl; if (in_smem) cum_s[b + 1] = incl; }
    __syncthreads();
    if (tid == 255) carry = incl;
    __syncthreads();
  }
  const int32_t* cs = in_smem ? cum_s : cum;
  const long long T = cs[B];
  for (int i = tid; i < G; i += 256) {
    const int p0 = static_cast<int>((static_cast<long long>(i) * T) / G);
    const int p1 = static_cast<int>((static_cast<long long>(i + 1) * T) / G);
    int b0 = -1, b1 = -1;
    if (p1 > p0) { b0 = seq_of_page(cs, B, p0); b1 = seq_of_page(cs, B, p1 - 1); }
    reinterpret_cast<int4*>(plan)[i] = make_int4(p0, p1, b0, b1);
  }
  // Partitions that hold pages of sequence b: first and last index (0, -1 for an empty sequence), stored behind
  // the prefix sums so that the combine does not repeat the 64-bit divisions for every row and head.
  int32_t* seq_parts = cum + B + 1;
  for (int b = tid; b < B; b += 256) {
    const long long c0 = static_cast<long long>(cs[b]) + kSegCost, c1 = cs[b + 1];
    int i_first = 0, i_last = -1;
    if (c1 > c0) {
      i_first = static_cast<int>(((c0 + 1) * G - 1) / T);
      i_last = static_cast<int>((c1 * G - 1) / T);
    }
    seq_parts[2 * b] = i_first;
    seq_parts[2 * b + 1] = i_last;
  }
  // The page counters of the split-KV kernel start at zero.  Every earlier kernel of the stream has completed
  // here (the dependency wait above), so nobody is still counting.
  int32_t* next = cum + 3 * B + 1;
  for (int i = tid; i < RB * B; i += 256) next[i] = 0;
}

// ------------------------------------------------------------------------------------------------
// Absorb (Eq. 9 right, first line): q_hat[bs,h,:r] = W_UK_h^T q_nope[bs,h,:], q_hat[bs,h,r:] = q_pe[bs,h,:].
// A block owns nt consecutive 128-column tiles of one head's latent columns (nt = 1, or 2 when that brings the
// launch down to one wave): it stages W_UK_h[:, tiles] and the head's query rows (128 at a time) in shared
// memory with asynchronous 16-byte copies, all in flight together, and walks the rows in 16-row tiles, so W_UK
// is read once.  The block that owns a head's first tile also copies the rope part of the rows.
// ------------------------------------------------------------------------------------------------
constexpr int kAbsorbRows = 128;  // query rows staged per pass

__device__ void absorb_block(const __nv_bfloat16* q_nope, const __nv_bfloat16* q_pe,
                             const __nv_bfloat16* __restrict__ w_uk, __nv_bfloat16* q_hat, int BS, int H,
                             int dn, int dR, int r, int h, int rt0, int nt, unsigned char* smem_raw) {
  const int apitch = dn + 8, wpitch = nt * 128 + 8;
  __nv_bfloat16* w_s = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [dn][wpitch]
  __nv_bfloat16* a_s = w_s + dn * wpitch;                            // [kAbsorbRows][dn + 8]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3, mi = lane >> 3;
  const int n0 = rt0 * 128, K = r + dR, vec_per_row = nt * 16;
  for (int i = tid; i < dn * vec_per_row; i += 256) {  // columns beyond r are zero-filled
    const int k = i / vec_per_row, c = i % vec_per_row;
    const bool in = n0 + c * 8 < r;
    cp_async16(w_s + k * wpitch + c * 8, w_uk + (static_cast<size_t>(h) * dn + k) * r + (in ? n0 + c * 8 : 0), in ? 16 : 0);
  }
  cp_async_commit();
  pdl_wait();  // the queries may come from the kernel before this one; the weights above may not
  const int chunks = dn / 8;
  for (int p0 = 0; p0 < BS; p0 += kAbsorbRows) {
    const int rows = min(kAbsorbRows, BS - p0);
    const int rows16 = (rows + 15) & ~15;
    if (p0 > 0) __syncthreads();  // previous pass has consumed a_s
    for (int i = tid; i < rows16 * chunks; i += 256) {  // rows beyond the last one are zero-filled
      const int rr = i / chunks, c = i % chunks;
      cp_async16(a_s + rr * apitch + c * 8, q_nope + (static_cast<size_t>(p0 + min(rr, rows - 1)) * H + h) * dn + c * 8,
                 rr < rows ? 16 : 0);
    }
    cp_async_commit();
    if (p0 == 0 && rt0 == 0 && dR > 0) {
      // the rope part is a plain copy, made while the operands of the first products are on their way
      if (dR % 8 == 0 && r % 8 == 0) {  // 16 bytes at a time, four copies in flight
        const int vecs = dR / 8;
        for (int i0 = tid; i0 < BS * vecs; i0 += 256 * 4) {
          uint4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * 256, row = i / vecs, c = (i % vecs) * 8;
            v[u] = make_uint4(0, 0, 0, 0);
            if (i < BS * vecs) v[u] = ld_u128(q_pe + (static_cast<size_t>(row) * H + h) * dR + c);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * 256, row = i / vecs, c = (i % vecs) * 8;
            if (i < BS * vecs) *reinterpret_cast<uint4*>(q_hat + (static_cast<size_t>(row) * H + h) * K + r + c) = v[u];
          }
        }
      } else {
        const int pairs = dR / 2;
        for (int i = tid; i < BS * pairs; i += 256) {
          const int row = i / pairs, c = (i % pairs) * 2;
          *reinterpret_cast<uint32_t*>(q_hat + (static_cast<size_t>(row) * H + h) * K + r + c) =
              ld_u32(q_pe + (static_cast<size_t>(row) * H + h) * dR + c);
        }
      }
    }
    cp_async_wait<0>();
    __syncthreads();
    for (int m0 = 0; m0 < rows16; m0 += 16) {
      for (int wc = warp * 16 * nt; wc < (warp + 1) * 16 * nt; wc += 16) {  // this warp's 16-column steps
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll 4
        for (int ks = 0; ks < dn / 16; ++ks) {
          uint32_t a[4], bf[4];
          ldmatrix_x4(a, a_s + (m0 + (mi & 1) * 8 + (lane & 7)) * apitch + ks * 16 + (mi >> 1) * 8);
          ldmatrix_x4_trans(bf, w_s + (ks * 16 + (mi & 1) * 8 + (lane & 7)) * wpitch + wc + (mi >> 1) * 8);
          mma_bf16_16816(acc[0], a, bf[0], bf[1]);
          mma_bf16_16816(acc[1], a, bf[2], bf[3]);
        }
        const int r0 = p0 + m0 + g, r1 = r0 + 8;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int col = n0 + wc + j * 8 + t4 * 2;
          if (col < r) {
            if (r0 < BS) *reinterpret_cast<uint32_t*>(q_hat + (static_cast<size_t>(r0) * H + h) * K + col) = pack_bf16(acc[j][0], acc[j][1]);
            if (r1 < BS) *reinterpret_cast<uint32_t*>(q_hat + (static_cast<size_t>(r1) * H + h) * K + col) = pack_bf16(acc[j][2], acc[j][3]);
          }
        }
      }
    }
  }
}

static size_t absorb_smem(int dn, int nt) {
  return (static_cast<size_t>(dn) * (nt * 128 + 8) + static_cast<size_t>(kAbsorbRows) * (dn + 8)) * sizeof(__nv_bfloat16);
}

// Tiles per absorb block: two when the prologue launch would otherwise not fit the device in one wave of one block
// per SM (the append's accumulators allow no more), the tile count is even and the pair's weights fit.
static int absorb_tiles_per_block(const transmla_params_t& p, int other_blocks) {
  static PerDeviceFlag sms_of;  // SM count per device, asked once
  const int slot = current_device_slot();
  int sms = slot >= 0 ? sms_of.value[slot].load(std::memory_order_acquire) : 0;
  if (sms == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      return 1;
    }
    if (slot >= 0) sms_of.value[slot].store(sms, std::memory_order_release);
  }
  const int r_tiles = (p.kv_lora_rank + 127) / 128;
  const bool fits_one = other_blocks + p.num_heads * r_tiles <= sms;
  return (!fits_one && r_tiles % 2 == 0 && p.qk_nope_dim <= 128) ? 2 : 1;
}

__global__ void __launch_bounds__(256) append_kernel(const __nv_bfloat16* x,
                                                     const __nv_bfloat16* __restrict__ w,
                                                     const int32_t* positions,
                                                     const int32_t* page_table,
                                                     __nv_bfloat16* cache, int32_t* dev_status, int B,
                                                     int S, int D, int r, int dR, int num_pages, int max_pages,
                                                     float theta, int t_splits, int wide) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_trigger();
  if (wide)
    append_block<1, 4>(x, w, positions, 0, page_table, cache, dev_status, B, S, D, r, dR, num_pages, max_pages, theta,
                       blockIdx.x, t_splits, smem_raw);
  else
    append_block<kAppendMaxMT, 1>(x, w, positions, 0, page_table, cache, dev_status, B, S, D, r, dR, num_pages, max_pages,
                                  theta, blockIdx.x, t_splits, smem_raw);
}

// Absorb blocks followed by one plan block: everything transmla_mla_decode needs before the split-KV kernel.
__global__ void __launch_bounds__(256) absorb_plan_kernel(const __nv_bfloat16* q_nope,
                                                          const __nv_bfloat16* q_pe,
                                                          const __nv_bfloat16* __restrict__ w_uk,
                                                          __nv_bfloat16* q_hat,
                                                          const int32_t* seqlens, int32_t* cum,
                                                          int32_t* plan, int32_t* dev_status, int B, int S, int H,
                                                          int dn, int dR, int r, int G, int max_pages, int nt) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_trigger();
  const int per_head = (r + 127) / 128 / nt;  // absorb blocks per head, nt tiles each
  const int n_absorb = H * per_head;
  if (static_cast<int>(blockIdx.x) < n_absorb) {
    absorb_block(q_nope, q_pe, w_uk, q_hat, B * S, H, dn, dR, r, blockIdx.x / per_head, blockIdx.x % per_head * nt, nt, smem_raw);
  } else {
    plan_block(seqlens, B, G, (S * H + kRowBlock - 1) / kRowBlock, max_pages, cum, plan, dev_status, smem_raw);
  }
}

// The whole prologue of a decode step in one launch: plan block, append blocks, absorb blocks.
// The appended token of sequence b sits at seqlens[b] - S + s.
__global__ void __launch_bounds__(256) prologue_kernel(
    const __nv_bfloat16* x, const __nv_bfloat16* __restrict__ w_dkv_kr,
    const int32_t* page_table, __nv_bfloat16* cache, const __nv_bfloat16* q_nope,
    const __nv_bfloat16* q_pe, const __nv_bfloat16* __restrict__ w_uk, __nv_bfloat16* q_hat,
    const int32_t* seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status, int B, int S, int H, int D,
    int dn, int dR, int r, int num_pages, int max_pages, float theta, int G, int t_splits, int wide, int nt) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_trigger();
  const int n_append = (r + dR) / (wide ? 32 : 8) * t_splits;
  const int per_head = (r + 127) / 128 / nt;  // absorb blocks per head, nt tiles each
  const int bid = static_cast<int>(blockIdx.x) - 1;
  if (bid < 0) {
    plan_block(seqlens, B, G, (S * H + kRowBlock - 1) / kRowBlock, max_pages, cum, plan, dev_status, smem_raw);
  } else if (bid < n_append) {
    if (wide)
      append_block<1, 4>(x, w_dkv_kr, seqlens, -S, page_table, cache, dev_status, B, S, D, r, dR, num_pages, max_pages,
                         theta, bid, t_splits, smem_raw);
    else
      append_block<kAppendMaxMT, 1>(x, w_dkv_kr, seqlens, -S, page_table, cache, dev_status, B, S, D, r, dR, num_pages,
                                    max_pages, theta, bid, t_splits, smem_raw);
  } else {
    const int a = bid - n_append;
    absorb_block(q_nope, q_pe, w_uk, q_hat, B * S, H, dn, dR, r, a / per_head, a % per_head * nt, nt, smem_raw);
  }
}

constexpr int kPrologueMaxSmem = 144 * 1024;

// Token splits of the append: one per 64 new tokens, at most 4.
// With many new tokens a block takes 32 output features and 16 tokens (activations re-read a quarter as often
// per feature, weights four times as often per token: 384 KB per block instead of 576 KB at 128 tokens).
bool append_wide(const transmla_params_t& p) {
  return p.batch * p.q_len > 32 && (p.kv_lora_rank + p.qk_rope_dim) % 32 == 0 && p.kv_lora_rank % 2 == 0;
}
int append_token_splits(const transmla_params_t& p) {
  const int T = p.batch * p.q_len;
  if (append_wide(p)) return (T + 15) / 16 > 32 ? 32 : (T + 15) / 16;
  return T <= 64 ? 1 : (T + 63) / 64 > 4 ? 4 : (T + 63) / 64;
}

cudaError_t launch_append(const transmla_params_t& p, const __nv_bfloat16* x, const __nv_bfloat16* w,
                          const int32_t* positions, const int32_t* page_table, __nv_bfloat16* cache,
                          int32_t* dev_status, cudaStream_t stream) {
  const int K = p.kv_lora_rank + p.qk_rope_dim;
  const int ts = append_token_splits(p);
  const int wide = append_wide(p) ? 1 : 0;
  return launch_pdl(append_kernel, dim3(K / (wide ? 32 : 8) * ts), dim3(256), kAppendSmem, stream, x, w, positions, page_table,
                    cache, dev_status, p.batch, p.q_len, p.hidden_dim, p.kv_lora_rank, p.qk_rope_dim, p.num_pages,
                    p.max_pages_per_seq, p.rope_theta, ts, wide);
}

cudaError_t launch_absorb_plan(const transmla_params_t& p, int G, const __nv_bfloat16* q_nope,
                               const __nv_bfloat16* q_pe, const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat,
                               const int32_t* seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status,
                               cudaStream_t stream) {
  const int nt = absorb_tiles_per_block(p, 1);
  size_t smem = absorb_smem(p.qk_nope_dim, nt);
  if (smem < kPlanSmemSeqs * sizeof(int32_t)) smem = kPlanSmemSeqs * sizeof(int32_t);
  static PerDeviceFlag smem_set;  // zero-initialised; one slot per device
  if (cudaError_t e = ensure_dynamic_smem(absorb_plan_kernel, kPrologueMaxSmem, smem_set); e != cudaSuccess) return e;
  const int blocks = p.num_heads * ((p.kv_lora_rank + 127) / 128 / nt) + 1;
  return launch_pdl(absorb_plan_kernel, dim3(blocks), dim3(256), smem, stream, q_nope, q_pe, w_uk, q_hat, seqlens, cum,
                    plan, dev_status, p.batch, p.q_len, p.num_heads, p.qk_nope_dim, p.qk_rope_dim, p.kv_lora_rank, G,
                    p.max_pages_per_seq, nt);
}

cudaError_t launch_prologue(const transmla_params_t& p, int G, const __nv_bfloat16* x, const __nv_bfloat16* w_dkv_kr,
                            const int32_t* page_table, __nv_bfloat16* cache, const __nv_bfloat16* q_nope,
                            const __nv_bfloat16* q_pe, const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat,
                            const int32_t* seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status,
                            cudaStream_t stream) {
  const int ts = append_token_splits(p);
  const int wide = append_wide(p) ? 1 : 0;
  const int n_append = (p.kv_lora_rank + p.qk_rope_dim) / (wide ? 32 : 8) * ts;
  const int nt = absorb_tiles_per_block(p, 1 + n_append);
  size_t smem = absorb_smem(p.qk_nope_dim, nt);
  if (smem < kAppendSmem) smem = kAppendSmem;
  static PerDeviceFlag smem_set;  // zero-initialised; one slot per device
  if (cudaError_t e = ensure_dynamic_smem(prologue_kernel, kPrologueMaxSmem, smem_set); e != cudaSuccess) return e;
  const int blocks = 1 + n_append + p.num_heads * ((p.kv_lora_rank + 127) / 128 / nt);
  return launch_pdl(prologue_kernel, dim3(blocks), dim3(256), smem, stream, x, w_dkv_kr, page_table, cache, q_nope, q_pe,
                    w_uk, q_hat, seqlens, cum, plan, dev_status, p.batch, p.q_len, p.num_heads, p.hidden_dim,
                    p.qk_nope_dim, p.qk_rope_dim, p.kv_lora_rank, p.num_pages, p.max_pages_per_seq, p.rope_theta, G, ts, wide, nt);
}

// ------------------------------------------------------------------------------------------------
// Combine + up-projection (Eq. 9 right, last line before W_O).  Block = one head x 8 or 16 query rows
// x (optionally) one half of the dv output columns.
// Phase 1: each warp merges the split partials of its rows by their lse (segments of sequence b live
// in slots i + b for the partitions i that overlap its pages) into shared memory as a bf16 hi/lo
// pair, so that the tensor-core product of phase 2 carries fp32-like precision of o_hat.  The merged
// row is stored in kperm order.
// Phase 2: out[rows, h, :] = o_hat W_UV_h^T with W_UV_h read straight from global memory, 16 bytes per
// lane and all loads of a tile in flight together.
// ------------------------------------------------------------------------------------------------
constexpr int kCombineRows = 16;

// kPrefetch: hold the first weight tile in registers from before the dependency wait (few blocks, latency
// matters); otherwise load weights window by window and keep the register count low enough for two blocks per SM.
template <bool kPrefetch>
__global__ void __launch_bounds__(256, kPrefetch ? 1 : 2) combine_kernel(const int32_t* cum,
                                                      const float* partial_o,
                                                      const float* partial_lse,
                                                      const __nv_bfloat16* __restrict__ w_uv,
                                                      __nv_bfloat16* out, float* lse_out,
                                                      int B, int S, int H, int r, int dv, int G, int rows_per_block) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch = r + 8;
  __nv_bfloat16* o_hi = reinterpret_cast<__nv_bfloat16*>(smem_raw);  // [16][pitch]
  __nv_bfloat16* o_lo = o_hi + kCombineRows * pitch;                 // [16][pitch]
  pdl_trigger();
  const int h = blockIdx.x, bs0 = blockIdx.y * rows_per_block;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int SH = S * H, BS = B * S;
  const int g = lane >> 2, t4 = lane & 3, mi = lane >> 3;
  const int tiles = dv / 8, tiles_per_z = (tiles + gridDim.z - 1) / gridDim.z;
  const int nt_lo = blockIdx.z * tiles_per_z, nt_hi = min(tiles, nt_lo + tiles_per_z);
  // The weights do not depend on the merge: the first tile's 16-byte loads are issued now and land while
  // the partials are merged.
  constexpr int kWin = kPrefetch ? 16 : 4;  // windows of 32 columns held in registers per round
  uint4 wv[kWin];
  if (kPrefetch) {
    const int nt = nt_lo + warp;
    const __nv_bfloat16* wrow = w_uv + (static_cast<size_t>(h) * dv + min(nt, tiles - 1) * 8 + g) * r + t4 * 8;
#pragma unroll
    for (int u = 0; u < kWin; ++u) wv[u] = (nt < nt_hi && u * 32 < r) ? ld_u128(wrow + u * 32) : make_uint4(0, 0, 0, 0);
  }
  pdl_wait();  // the partials and the prefix sums come from the kernels before this one
  const long long T = cum[B];

  for (int rr = warp; rr < kCombineRows; rr += 8) {
    const int bs = bs0 + rr;
    float acc[4][4];
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[c][0] = acc[c][1] = acc[c][2] = acc[c][3] = 0.f;
    float lse = -INFINITY, inv = 0.f;
    if (rr < rows_per_block && bs < BS) {
      const int b = bs / S, s = bs % S, row = s * H + h;
      const int32_t* seq_parts = cum + B + 1;  // only 4-byte aligned: B + 1 may be odd
      const int i_first = seq_parts[2 * b], nseg = seq_parts[2 * b + 1] - i_first + 1;
      const bool dense = T >= G;  // then every partition owns at least one slot
      if (nseg > 0) {
        auto seg_lse = [&](int j) -> float {  // lse of the j-th candidate partition, -inf if it is empty or absent
          if (j >= nseg) return -INFINITY;
          const int pi = i_first + j;
          if (!dense) {
            const long long p0 = (static_cast<long long>(pi) * T) / G, p1 = (static_cast<long long>(pi + 1) * T) / G;
            if (p1 <= p0) return -INFINITY;
          }
          return partial_lse[static_cast<size_t>(pi + b) * SH + row];
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
            const float* po0 = partial_o + (static_cast<size_t>(i_first + base + b) * SH + row) * r + lane * 4;
            const size_t seg_stride = static_cast<size_t>(SH) * r;
            // four segments per round so that their loads overlap; a zero weight skips the (unwritten) slot
            for (int j0 = 0; j0 < cnt; j0 += 4) {
              float wj[4];
              float4 v[4][4];
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                wj[u] = (j0 + u < cnt) ? __shfl_sync(0xffffffffu, wgt, (j0 + u) & 31) : 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  v[u][c] = make_float4(0.f, 0.f, 0.f, 0.f);
                  if (wj[u] != 0.f && c * 128 + lane * 4 < r)
                    v[u][c] = *reinterpret_cast<const float4*>(po0 + (j0 + u) * seg_stride + c * 128);
                }
              }
#pragma unroll
              for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  acc[c][0] = fmaf(wj[u], v[u][c].x, acc[c][0]); acc[c][1] = fmaf(wj[u], v[u][c].y, acc[c][1]);
                  acc[c][2] = fmaf(wj[u], v[u][c].z, acc[c][2]); acc[c][3] = fmaf(wj[u], v[u][c].w, acc[c][3]);
                }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
          inv = 1.f / den;
          lse = m + __logf(den);
        }
      }
      if (lse_out != nullptr && lane == 0 && blockIdx.z == 0) lse_out[(static_cast<size_t>(b) * S + s) * H + h] = lse;
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
        const int win = k & ~31, p = k & 31;  // elements p..p+3 of the window: two pairs, each stays adjacent
        const int q0 = win + kperm(p), q1 = win + kperm(p + 2);
        *reinterpret_cast<uint32_t*>(o_hi + rr * pitch + q0) = pack_bf16(v[0], v[1]);
        *reinterpret_cast<uint32_t*>(o_hi + rr * pitch + q1) = pack_bf16(v[2], v[3]);
        *reinterpret_cast<uint32_t*>(o_lo + rr * pitch + q0) = pack_bf16(lo[0], lo[1]);
        *reinterpret_cast<uint32_t*>(o_lo + rr * pitch + q1) = pack_bf16(lo[2], lo[3]);
      }
    }
  }
  __syncthreads();

  for (int nt = nt_lo + warp; nt < nt_hi; nt += 8) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const __nv_bfloat16* wrow = w_uv + (static_cast<size_t>(h) * dv + nt * 8 + g) * r + t4 * 8;
    for (int w0 = 0; w0 < r; w0 += kWin * 32) {  // kWin windows per round, all their loads in flight together
      if (!kPrefetch || nt != nt_lo + warp || w0 != 0) {
#pragma unroll
        for (int u = 0; u < kWin; ++u)
          wv[u] = (w0 + u * 32 < r) ? ld_u128(wrow + w0 + u * 32) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < kWin; ++u) {
        if (w0 + u * 32 < r) {
          uint32_t ah[4], al[4];
          const int off = ((mi & 1) * 8 + (lane & 7)) * pitch + w0 + u * 32 + (mi >> 1) * 8;
          ldmatrix_x4(ah, o_hi + off);
          ldmatrix_x4(al, o_lo + off);
          mma_bf16_16816(acc, ah, wv[u].x, wv[u].y);
          mma_bf16_16816(acc, al, wv[u].x, wv[u].y);
          ldmatrix_x4(ah, o_hi + off + 16);
          ldmatrix_x4(al, o_lo + off + 16);
          mma_bf16_16816(acc, ah, wv[u].z, wv[u].w);
          mma_bf16_16816(acc, al, wv[u].z, wv[u].w);
        }
      }
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
                           int32_t* dev_status, cudaStream_t stream) {
  (void)dev_status;
  const int BS = p.batch * p.q_len;
  // 8 rows per block while the register-prefetching variant runs (few query rows, more parallelism), 16 beyond:
  // at 64 query rows that is 256 blocks, one wave at two blocks per SM, instead of 512
  const int rows = BS <= 32 ? 8 : 16;
  const int zsplit = (BS <= 64 && p.v_dim >= 128) ? 2 : 1;
  dim3 grid(p.num_heads, (BS + rows - 1) / rows, zsplit);
  const size_t smem = 2 * kCombineRows * (p.kv_lora_rank + 8) * sizeof(__nv_bfloat16);
  if (BS <= 32)
    return launch_pdl(combine_kernel<true>, grid, dim3(256), smem, stream, cum, partial_o, partial_lse, w_uv, out, lse_out,
                      p.batch, p.q_len, p.num_heads, p.kv_lora_rank, p.v_dim, G, rows);
  return launch_pdl(combine_kernel<false>, grid, dim3(256), smem, stream, cum, partial_o, partial_lse, w_uv, out, lse_out,
                    p.batch, p.q_len, p.num_heads, p.kv_lora_rank, p.v_dim, G, rows);
}

}  // namespace transmla
