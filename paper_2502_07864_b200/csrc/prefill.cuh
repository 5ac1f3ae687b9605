// Prefill in the MHA form (Sec. 3.3, Eq. 8 and Eq. 9 left): launchers of its two kernels.
#pragma once
#include "common.cuh"

namespace transmla {

// dn = dv = 128, r = 512, dR = 64: the shape the tensor-path kernels are built for.
bool prefill_supported(const transmla_params_t& p);
// One row of the decompressed store holds, for every head, k^C (dn) followed by v (dv), in bf16.
inline size_t prefill_row_elems(const transmla_params_t& p) {
  return static_cast<size_t>(p.num_heads) * (p.qk_nope_dim + p.v_dim);
}
// kv_dec[num_pages * 64, H * 256]: row page*64 + slot of every page the page table names for tokens < L_b.
cudaError_t launch_prefill_decompress(const transmla_params_t& p, const __nv_bfloat16* cache, const int32_t* page_table,
                                      const int32_t* seqlens, const __nv_bfloat16* w_uk, const __nv_bfloat16* w_uv,
                                      __nv_bfloat16* kv_dec, int32_t* dev_status, cudaStream_t stream);
// out[B, S, H, dv], lse[B, S, H] (may be null): causal attention of the chunk's S query positions over kv_dec and k^R.
cudaError_t launch_prefill_attention(const transmla_params_t& p, const __nv_bfloat16* q_nope, const __nv_bfloat16* q_pe,
                                     const __nv_bfloat16* cache, const __nv_bfloat16* kv_dec, const int32_t* page_table,
                                     const int32_t* seqlens, __nv_bfloat16* out, float* lse, int32_t* dev_status,
                                     cudaStream_t stream);

}  // namespace transmla
