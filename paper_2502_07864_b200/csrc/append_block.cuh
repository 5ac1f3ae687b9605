// The append's block routine, shared by the kernels that hold append blocks (the prologue launches and, in the
// layer step, the launch of the query maps).
#pragma once
#include "common.cuh"
#include "skinny_gemm.cuh"

namespace transmla {

// ------------------------------------------------------------------------------------------------
// Latent append (Eq. 7 left): y = [W_DKV; W_KR] x, RoPE (Eq. 1) on y[r:], bf16, scatter to the page slot.
// One block owns 8 consecutive output features (a RoPE pair never straddles blocks); its 8 warps
// split the hidden dimension and meet in shared memory.  Tokens are the M dimension of the tiles.
// Token (b, s) sits at position pos_base[b] + pos_shift + s.
// ------------------------------------------------------------------------------------------------
template <int MAXMT, int NT>
__device__ void append_block(const __nv_bfloat16* x, const __nv_bfloat16* __restrict__ w,
                             const int32_t* pos_base, int pos_shift,
                             const int32_t* page_table, __nv_bfloat16* cache,
                             int32_t* dev_status, int B, int S, int D, int r, int dR, int num_pages, int max_pages,
                             float theta, int nb, int t_splits, unsigned char* smem_raw) {
  // block nb = (token split, feature tile): with many tokens the token range is cut so that more SMs take part
  const int K = r + dR, f_tiles = K / (8 * NT), f0 = (nb % f_tiles) * 8 * NT;
  const int t_chunk = (((B * S + t_splits - 1) / t_splits) + 15) & ~15;
  const int t_begin = (nb / f_tiles) * t_chunk, t_end = min(B * S, t_begin + t_chunk);
  skinny_gemm_tile<MAXMT, NT>(x, w, D, f0, t_begin, t_end, smem_raw, [&](int t, int pr, float re, float im) {
    const int b = t / S, s = t % S;
    const int pos = pos_base[b] + pos_shift + s;
    const int pj = pos / kPage;
    int page = -1;
    if (pos >= 0 && pj < max_pages) page = page_table[static_cast<size_t>(b) * max_pages + pj];
    if (page < 0 || page >= num_pages) {
      set_status(dev_status, TRANSMLA_DEV_BAD_PAGE);
      return;
    }
    const int f = f0 + pr * 2;
    if (f >= r) rope_pair(re, im, pos, (f - r) >> 1, dR, theta);  // RoPE pair l of the decoupled key (Eq. 1)
    *reinterpret_cast<uint32_t*>(cache + (static_cast<size_t>(page) * kPage + pos % kPage) * K + f) = pack_bf16(re, im);
  });
}

// Shared memory an append block needs, and how the host cuts the append into blocks.
constexpr size_t kAppendBlockSmem = kAppendSmem;
bool append_wide(const transmla_params_t& p);        // 32 features x 16 tokens per block instead of 8 x 64
int append_token_splits(const transmla_params_t& p);

}  // namespace transmla
