// Linear maps either side of the attention (Eq. 8 right column: queries; Eq. 9 last line: W_O), as skinny GEMMs
// y[M, N] = x[M, K] w[N, K]^T with M = the step's new tokens.  They stream their weights once; a block owns 8
// output features (see skinny_gemm.cuh).  One launch may hold two jobs (q^C and q^R share their input).
#include <algorithm>

#include "append_block.cuh"
#include "common.cuh"
#include "linear_args.cuh"
#include "skinny_gemm.cuh"

namespace transmla {

// MAXMT x 16 tokens per pass, NT x 8 output features per block.
template <int MAXMT, int NT>
__global__ void __launch_bounds__(256, 1) linear_kernel(LinearArgs a, int32_t* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  pdl_trigger();
  int nb = blockIdx.x, j = 0;
  const int blocks0 = a.job[0].N / (8 * NT) * a.t_splits;
  const int blocks1 = a.n_jobs > 1 ? a.job[1].N / (8 * NT) * a.t_splits : 0;
  if (nb >= blocks0 + blocks1) {  // the step's append: token (b, s) sits at pos_base[b] + pos_shift + s
    const AppendJob& ap = a.append;
    nb -= blocks0 + blocks1;
    if (ap.wide)
      append_block<1, 4>(ap.x, ap.w, a.pos_base, a.pos_shift, ap.page_table, ap.cache, dev_status, ap.B, a.S, ap.D, ap.r, ap.dR,
                         ap.num_pages, ap.max_pages, a.theta, nb, ap.t_splits, smem_raw);
    else
      append_block<kAppendMaxMT, 1>(ap.x, ap.w, a.pos_base, a.pos_shift, ap.page_table, ap.cache, dev_status, ap.B, a.S, ap.D,
                                    ap.r, ap.dR, ap.num_pages, ap.max_pages, a.theta, nb, ap.t_splits, smem_raw);
    return;
  }
  if (nb >= blocks0) { nb -= blocks0; j = 1; }
  const LinearJob job = a.job[j];
  const int f_tiles = job.N / (8 * NT), f0 = (nb % f_tiles) * 8 * NT;
  const int t_chunk = (((a.M + a.t_splits - 1) / a.t_splits) + 15) & ~15;
  const int t_begin = (nb / f_tiles) * t_chunk, t_end = min(a.M, t_begin + t_chunk);
  skinny_gemm_tile<MAXMT, NT>(job.x, job.w, job.K, f0, t_begin, t_end, smem_raw, [&](int t, int pr, float re, float im) {
    const int f = f0 + pr * 2;
    if (job.rope_d > 0) {
      const int pos = a.pos_base[t / a.S] + a.pos_shift + t % a.S;
      rope_pair(re, im, pos, (f % job.rope_d) >> 1, job.rope_d, a.theta);
    }
    *reinterpret_cast<uint32_t*>(job.out + static_cast<size_t>(t) * job.N + f) = pack_bf16(re, im);
  });
}

cudaError_t launch_linear(const LinearArgs& args, int32_t* dev_status, cudaStream_t stream) {
  // 32 features per block when every job allows it (the activations are then read a quarter as often)
  bool wide = true;
  for (int j = 0; j < args.n_jobs; ++j) wide = wide && args.job[j].N % 32 == 0;
  const int per_block = wide ? 32 : 8;
  int blocks = 0;
  for (int j = 0; j < args.n_jobs; ++j) blocks += args.job[j].N / per_block * args.t_splits;
  blocks += args.append.blocks;  // short blocks at the end of the grid: they fill the last wave
  static_assert(skinny_gemm_smem(8, 1) >= kAppendBlockSmem && skinny_gemm_smem(4, 4) >= kAppendBlockSmem, "append blocks fit");
  if (!wide) return launch_pdl(linear_kernel<8, 1>, dim3(blocks), dim3(256), skinny_gemm_smem(8, 1), stream, args, dev_status);
  constexpr size_t smem = skinny_gemm_smem(4, 4);  // 64 KB: above the default limit
  static PerDeviceFlag smem_set;  // zero-initialised; one slot per device
  if (cudaError_t e = ensure_dynamic_smem(linear_kernel<4, 4>, static_cast<int>(smem), smem_set); e != cudaSuccess) return e;
  return launch_pdl(linear_kernel<4, 4>, dim3(blocks), dim3(256), smem, stream, args, dev_status);
}

}  // namespace transmla

using namespace transmla;

namespace {
constexpr size_t kAlign = 256;
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline int token_splits(int M) { return M <= 64 ? 1 : (M + 63) / 64 > 4 ? 4 : (M + 63) / 64; }
}  // namespace

extern "C" {

size_t transmla_layer_scratch_bytes(const transmla_params_t* p, int32_t q_lora_rank) {
  if (p == nullptr || q_lora_rank < 0) return 0;
  const size_t M = static_cast<size_t>(p->batch) * p->q_len, H = p->num_heads;
  size_t off = 0;
  off = round_up(off + M * q_lora_rank * 2, kAlign);
  off = round_up(off + M * H * p->qk_nope_dim * 2, kAlign);
  off = round_up(off + M * H * p->qk_rope_dim * 2 + 16, kAlign);
  off = round_up(off + M * H * p->v_dim * 2, kAlign);
  // tcgen05 linear maps: partial results of the K slices (largest of the three launches) and arrival counters
  const int Mi = static_cast<int>(M), D = p->hidden_dim, Kq = q_lora_rank ? q_lora_rank : D;
  const int tiles_dq = q_lora_rank / 128, tiles_q = static_cast<int>(H) * (p->qk_nope_dim + p->qk_rope_dim) / 128, tiles_o = D / 128;
  size_t partial = 0;
  if (tiles_dq > 0) partial = std::max(partial, linear_sm100_partial_bytes(tiles_dq, D, Mi));
  if (tiles_q > 0) partial = std::max(partial, linear_sm100_partial_bytes(tiles_q, Kq, Mi));
  if (tiles_o > 0) partial = std::max(partial, linear_sm100_partial_bytes(tiles_o, static_cast<int>(H) * p->v_dim, Mi));
  off = round_up(off + partial, kAlign);
  off = round_up(off + linear_sm100_counter_bytes(std::max(tiles_dq, std::max(tiles_q, tiles_o)) + 1, Mi), kAlign);
  return off;
}

transmla_status_t transmla_layer_decode_step(const transmla_params_t* p, const transmla_layer_weights_t* w,
                                             const void* x, const int32_t* page_table, const int32_t* seqlens,
                                             void* cache, void* workspace, size_t workspace_bytes, void* scratch,
                                             size_t scratch_bytes, void* y, int32_t* dev_status, void* stream) {
  if (p == nullptr || w == nullptr) return TRANSMLA_ERR_NULL;
  if (!x || !seqlens || !scratch || !y || !w->w_uq || !w->w_o || !w->w_dkv_kr || !w->w_uk || !w->w_uv) return TRANSMLA_ERR_NULL;
  if (p->qk_rope_dim > 0 && !w->w_qr) return TRANSMLA_ERR_NULL;
  const bool low_rank = w->w_dq != nullptr;
  const int H = p->num_heads, D = p->hidden_dim, rq = low_rank ? w->q_lora_rank : 0;
  const int Kq = low_rank ? rq : D, Ko = H * p->v_dim;
  if (p->batch < 1 || p->q_len < 1 || D < 256 || D % 256 || Ko % 256 || (low_rank && (rq < 256 || rq % 256)) ||
      (H * p->qk_nope_dim) % 8 || (H * p->qk_rope_dim) % 8 || p->qk_rope_dim % 2)
    return TRANSMLA_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(y) || !aligned16(w->w_dq) || !aligned16(w->w_uq) || !aligned16(w->w_qr) ||
      !aligned16(w->w_o) || (reinterpret_cast<uintptr_t>(scratch) & (kAlign - 1)))
    return TRANSMLA_ERR_ALIGN;
  if (scratch_bytes < transmla_layer_scratch_bytes(p, rq)) return TRANSMLA_ERR_WORKSPACE;

  const int M = p->batch * p->q_len;
  char* base = static_cast<char*>(scratch);
  size_t off = 0;
  auto* cq = reinterpret_cast<__nv_bfloat16*>(base + off);      off = round_up(off + static_cast<size_t>(M) * rq * 2, kAlign);
  auto* q_nope = reinterpret_cast<__nv_bfloat16*>(base + off);  off = round_up(off + static_cast<size_t>(M) * H * p->qk_nope_dim * 2, kAlign);
  auto* q_pe = reinterpret_cast<__nv_bfloat16*>(base + off);    off = round_up(off + static_cast<size_t>(M) * H * p->qk_rope_dim * 2 + 16, kAlign);
  auto* attn = reinterpret_cast<__nv_bfloat16*>(base + off);                          off = round_up(off + static_cast<size_t>(M) * H * p->v_dim * 2, kAlign);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // tcgen05 linear maps (feature counts that are multiples of 128): scratch for the K slices and their counters
  const int tiles_dq = rq / 128, tiles_q = H * (p->qk_nope_dim + p->qk_rope_dim) / 128, tiles_o = D / 128;
  size_t partial_bytes = 0;
  if (tiles_dq > 0) partial_bytes = std::max(partial_bytes, linear_sm100_partial_bytes(tiles_dq, D, M));
  if (tiles_q > 0) partial_bytes = std::max(partial_bytes, linear_sm100_partial_bytes(tiles_q, Kq, M));
  if (tiles_o > 0) partial_bytes = std::max(partial_bytes, linear_sm100_partial_bytes(tiles_o, Ko, M));
  auto* lin_partial = reinterpret_cast<float*>(base + off);                          off = round_up(off + partial_bytes, kAlign);
  auto* lin_counters = reinterpret_cast<int32_t*>(base + off);
  const size_t counter_bytes = linear_sm100_counter_bytes(std::max(tiles_dq, std::max(tiles_q, tiles_o)) + 1, M);
  bool counters_cleared = false;
  // One linear launch: the tcgen05 kernel where the shapes allow it, the mma.sync tiles otherwise.  The counters
  // of the tcgen05 kernel must be zero before its first launch of this call; every launch leaves them at zero.
  auto run_linear = [&](const LinearArgs& la) -> cudaError_t {
    if (!linear_sm100_supported(la)) return launch_linear(la, dev_status, s);
    if (!counters_cleared) {
      cudaError_t e = cudaMemsetAsync(lin_counters, 0, counter_bytes, s);
      if (e != cudaSuccess) return e;
      counters_cleared = true;
    }
    return launch_linear_sm100(la, lin_partial, lin_counters, dev_status, s);
  };
  const auto* xin = static_cast<const __nv_bfloat16*>(x);

  transmla_status_t st = validate_step_args(p, x, q_nope, q_pe, w->w_dkv_kr, w->w_uk, w->w_uv, cache, page_table, seqlens,
                                            workspace, workspace_bytes, attn, dev_status);
  if (st != TRANSMLA_OK) return st;

  LinearArgs a = {};
  a.M = M; a.S = p->q_len; a.t_splits = token_splits(M); a.pos_base = seqlens; a.pos_shift = -p->q_len; a.theta = p->rope_theta;
  // The append (Eq. 7 left) is one more linear map of x: where the layer's first launch runs on the mma.sync tiles
  // its blocks ride in that launch, off the chain queries -> absorb -> attention; otherwise it stays in the
  // attention step's prologue.
  AppendJob ap = {};
  ap.x = xin; ap.w = static_cast<const __nv_bfloat16*>(w->w_dkv_kr); ap.page_table = page_table;
  ap.cache = static_cast<__nv_bfloat16*>(cache);
  ap.B = p->batch; ap.D = D; ap.r = p->kv_lora_rank; ap.dR = p->qk_rope_dim; ap.num_pages = p->num_pages;
  ap.max_pages = p->max_pages_per_seq; ap.t_splits = append_token_splits(*p); ap.wide = append_wide(*p) ? 1 : 0;
  ap.blocks = (ap.r + ap.dR) / (ap.wide ? 32 : 8) * ap.t_splits;
  bool appended = false;
  auto with_append = [&](LinearArgs& la) {  // the first launch takes the append along if it can
    if (!appended && !linear_sm100_supported(la)) { la.append = ap; appended = true; }
  };
  if (low_rank) {  // c^Q = W_DQ x
    a.n_jobs = 1;
    a.job[0] = {xin, static_cast<const __nv_bfloat16*>(w->w_dq), cq, rq, D, 0};
    with_append(a);
    if (run_linear(a) != cudaSuccess) return TRANSMLA_ERR_CUDA;
    a.append = AppendJob{};
  }
  const __nv_bfloat16* qin = low_rank ? cq : xin;
  a.n_jobs = p->qk_rope_dim > 0 ? 2 : 1;  // q^C = W_UQ c^Q and q^R = RoPE(W_QR c^Q, t) in one launch
  a.job[0] = {qin, static_cast<const __nv_bfloat16*>(w->w_uq), q_nope, H * p->qk_nope_dim, Kq, 0};
  a.job[1] = {qin, static_cast<const __nv_bfloat16*>(w->w_qr), q_pe, H * p->qk_rope_dim, Kq, p->qk_rope_dim};
  if (!low_rank) with_append(a);
  if (run_linear(a) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  a.append = AppendJob{};

  if (appended) {  // the new tokens' rows are in the cache (or on their way, earlier in the stream): attention only
    st = transmla_mla_decode(p, q_nope, q_pe, w->w_uk, cache, page_table, seqlens, workspace, workspace_bytes, dev_status, stream);
    if (st == TRANSMLA_OK)
      st = transmla_mla_combine(p, workspace, workspace_bytes, w->w_uv, attn, nullptr, dev_status, stream);
  } else {
    st = transmla_decode_step(p, x, q_nope, q_pe, page_table, seqlens, w->w_dkv_kr, w->w_uk, w->w_uv, cache,
                              workspace, workspace_bytes, attn, nullptr, dev_status, stream);
  }
  if (st != TRANSMLA_OK) return st;

  a.n_jobs = 1;  // y = W_O [o_1; ...; o_h]
  a.job[0] = {attn, static_cast<const __nv_bfloat16*>(w->w_o), static_cast<__nv_bfloat16*>(y), D, Ko, 0};
  if (run_linear(a) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  return TRANSMLA_OK;
}

}  // extern "C"
