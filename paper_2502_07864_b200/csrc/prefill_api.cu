// C ABI of prefill in the MHA form (Sec. 3.3): decompress the latent cache once (Eq. 8), then ordinary causal
// attention of the chunk's query positions over the decompressed keys and values (Eq. 9 left).
#include "prefill.cuh"

using namespace transmla;

namespace {
inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

transmla_status_t check_prefill_shape(const transmla_params_t* p) {
  if (p == nullptr) return TRANSMLA_ERR_NULL;
  if (p->page_size != kPage || !prefill_supported(*p)) return TRANSMLA_ERR_SHAPE;
  if (p->num_heads < 1 || p->num_heads > 1024 || p->q_len < 1 || p->q_len > (1 << 20)) return TRANSMLA_ERR_SHAPE;
  if (p->batch < 1 || p->batch > 65535 || p->num_pages < 1 || p->max_pages_per_seq < 1) return TRANSMLA_ERR_SHAPE;
  if (static_cast<long long>(p->batch) * p->q_len > 0x7fffffffLL) return TRANSMLA_ERR_SHAPE;
  return TRANSMLA_OK;
}
transmla_status_t on_blackwell() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return TRANSMLA_ERR_CUDA; }
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  return major == 10 ? TRANSMLA_OK : TRANSMLA_ERR_ARCH;
}
}  // namespace

extern "C" {

size_t transmla_prefill_scratch_bytes(const transmla_params_t* p) {
  if (check_prefill_shape(p) != TRANSMLA_OK) return 0;
  return static_cast<size_t>(p->num_pages) * kPage * prefill_row_elems(*p) * sizeof(__nv_bfloat16);
}

transmla_status_t transmla_prefill_decompress(const transmla_params_t* p, const void* cache, const int32_t* page_table,
                                              const int32_t* seqlens, const void* w_uk, const void* w_uv, void* scratch,
                                              size_t scratch_bytes, int32_t* dev_status, void* stream) {
  transmla_status_t st = check_prefill_shape(p);
  if (st != TRANSMLA_OK) return st;
  if (!cache || !page_table || !seqlens || !w_uk || !w_uv || !scratch) return TRANSMLA_ERR_NULL;
  if (!aligned_to(cache, 128) || !aligned_to(w_uk, 16) || !aligned_to(w_uv, 16) || !aligned_to(scratch, 128) ||
      !aligned_to(page_table, 4) || !aligned_to(seqlens, 4) || !aligned_to(dev_status, 4))
    return TRANSMLA_ERR_ALIGN;
  if (scratch_bytes < transmla_prefill_scratch_bytes(p)) return TRANSMLA_ERR_WORKSPACE;
  if ((st = on_blackwell()) != TRANSMLA_OK) return st;
  const cudaError_t e = launch_prefill_decompress(*p, static_cast<const __nv_bfloat16*>(cache), page_table, seqlens,
                                                  static_cast<const __nv_bfloat16*>(w_uk), static_cast<const __nv_bfloat16*>(w_uv),
                                                  static_cast<__nv_bfloat16*>(scratch), dev_status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

transmla_status_t transmla_prefill_attention(const transmla_params_t* p, const void* q_nope, const void* q_pe, const void* cache,
                                             const void* scratch, size_t scratch_bytes, const int32_t* page_table,
                                             const int32_t* seqlens, void* out, float* lse, int32_t* dev_status, void* stream) {
  transmla_status_t st = check_prefill_shape(p);
  if (st != TRANSMLA_OK) return st;
  if (!q_nope || !q_pe || !cache || !scratch || !page_table || !seqlens || !out) return TRANSMLA_ERR_NULL;
  if (!aligned_to(q_nope, 16) || !aligned_to(q_pe, 16) || !aligned_to(cache, 128) || !aligned_to(scratch, 128) ||
      !aligned_to(out, 16) || !aligned_to(lse, 4) || !aligned_to(page_table, 4) || !aligned_to(seqlens, 4) ||
      !aligned_to(dev_status, 4))
    return TRANSMLA_ERR_ALIGN;
  if (scratch_bytes < transmla_prefill_scratch_bytes(p)) return TRANSMLA_ERR_WORKSPACE;
  if ((st = on_blackwell()) != TRANSMLA_OK) return st;
  const cudaError_t e = launch_prefill_attention(*p, static_cast<const __nv_bfloat16*>(q_nope), static_cast<const __nv_bfloat16*>(q_pe),
                                                 static_cast<const __nv_bfloat16*>(cache), static_cast<const __nv_bfloat16*>(scratch),
                                                 page_table, seqlens, static_cast<__nv_bfloat16*>(out), lse, dev_status,
                                                 static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

transmla_status_t transmla_mla_prefill(const transmla_params_t* p, const void* q_nope, const void* q_pe, const void* w_uk,
                                       const void* w_uv, const void* cache, const int32_t* page_table, const int32_t* seqlens,
                                       void* scratch, size_t scratch_bytes, void* out, float* lse, int32_t* dev_status,
                                       void* stream) {
  transmla_status_t st = transmla_prefill_decompress(p, cache, page_table, seqlens, w_uk, w_uv, scratch, scratch_bytes, dev_status, stream);
  if (st != TRANSMLA_OK) return st;
  return transmla_prefill_attention(p, q_nope, q_pe, cache, scratch, scratch_bytes, page_table, seqlens, out, lse, dev_status, stream);
}

}  // extern "C"
