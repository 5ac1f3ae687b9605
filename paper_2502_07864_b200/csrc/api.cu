// C ABI of the absorbed-MLA decode library: argument checks, workspace layout, launches.
#include <cstdio>
#include <cstring>
#include <unordered_set>
#include <vector>

#include "common.cuh"

using namespace transmla;

namespace {

constexpr size_t kAlign = 256;
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

bool supported_latent(int r, int dR) {
  return (r == 512 && dR == 64) || (r == 128 && dR == 0) || (r == 64 && dR == 16);
}

transmla_status_t check_shape(const transmla_params_t* p, bool need_hidden) {
  if (p == nullptr) return TRANSMLA_ERR_NULL;
  if (p->page_size != kPage) return TRANSMLA_ERR_SHAPE;
  if (!supported_latent(p->kv_lora_rank, p->qk_rope_dim)) return TRANSMLA_ERR_SHAPE;
  if (p->num_heads < 1 || p->q_len < 1 || p->num_heads * p->q_len > 1024) return TRANSMLA_ERR_SHAPE;
  if (p->qk_nope_dim < 16 || p->qk_nope_dim > 256 || p->qk_nope_dim % 16) return TRANSMLA_ERR_SHAPE;
  if (p->v_dim < 8 || p->v_dim > 256 || p->v_dim % 8) return TRANSMLA_ERR_SHAPE;
  if (p->batch < 1 || p->num_pages < 1 || p->max_pages_per_seq < 1) return TRANSMLA_ERR_SHAPE;
  if (p->num_partitions < 0 || p->num_partitions > (1 << 20)) return TRANSMLA_ERR_SHAPE;
  if (need_hidden && (p->hidden_dim < 256 || p->hidden_dim % 256)) return TRANSMLA_ERR_SHAPE;
  return TRANSMLA_OK;
}

transmla_status_t check_device(int* sm_count) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return TRANSMLA_ERR_CUDA; }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  if (major != 10) return TRANSMLA_ERR_ARCH;
  if (sm_count != nullptr &&
      cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return TRANSMLA_ERR_CUDA;
  return TRANSMLA_OK;
}

thread_local cudaEvent_t tl_prof_start = nullptr, tl_prof_stop = nullptr;

// ---- host <-> device transfers of the host-buffer step done by one kernel each way.
// Pinned host memory is addressable from the device, so a single launch can move all five input arrays (and
// another one the results) instead of one copy-engine operation per array, each with its own start-up latency.
struct CopyJob { const void* src; void* dst; unsigned long long bytes; };
struct CopyList { CopyJob job[6]; int n; int32_t* zero_word; };

__global__ void __launch_bounds__(256) copy_list_kernel(CopyList list) {
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0 && list.zero_word != nullptr) *list.zero_word = 0;
  if (static_cast<int>(blockIdx.y) >= list.n) return;
  const CopyJob j = list.job[blockIdx.y];
  const size_t tid = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x, nthr = static_cast<size_t>(gridDim.x) * blockDim.x;
  if (((reinterpret_cast<uintptr_t>(j.src) | reinterpret_cast<uintptr_t>(j.dst) | j.bytes) & 15) == 0) {
    const uint4* s = static_cast<const uint4*>(j.src);
    uint4* d = static_cast<uint4*>(j.dst);
    for (size_t i = tid; i < j.bytes / 16; i += nthr) d[i] = s[i];
  } else {  // every array of the step is a whole number of 4-byte words
    const uint32_t* s = static_cast<const uint32_t*>(j.src);
    uint32_t* d = static_cast<uint32_t*>(j.dst);
    for (size_t i = tid; i < j.bytes / 4; i += nthr) d[i] = s[i];
  }
}

// Blocks per array for the copy kernel: one per 16 KB of the largest array, between 24 and 128 (a few blocks
// cannot keep enough reads in flight over PCIe once an array reaches a megabyte).
int copy_blocks(const CopyList& l) {
  unsigned long long most = 0;
  for (int i = 0; i < l.n; ++i) most = l.job[i].bytes > most ? l.job[i].bytes : most;
  const unsigned long long b = most / 16384;
  return b < 24 ? 24 : b > 128 ? 128 : static_cast<int>(b);
}

bool is_pinned_host(const void* p) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
  return a.type == cudaMemoryTypeHost && (reinterpret_cast<uintptr_t>(p) & 3) == 0;
}

// One pinned word per calling thread for reading the device status back without a copy-engine operation.
int32_t* pinned_status_word() {
  thread_local int32_t* word = nullptr;
  if (word == nullptr && cudaHostAlloc(reinterpret_cast<void**>(&word), 64, cudaHostAllocPortable) != cudaSuccess) {
    cudaGetLastError();
    word = nullptr;
  }
  return word;
}

}  // namespace

extern "C" {

void transmla_profile_decode_kernel(void* start_event, void* stop_event) {
  tl_prof_start = static_cast<cudaEvent_t>(start_event);
  tl_prof_stop = static_cast<cudaEvent_t>(stop_event);
}

transmla_status_t transmla_workspace_layout(const transmla_params_t* p, transmla_workspace_layout_t* out) {
  if (out == nullptr) return TRANSMLA_ERR_NULL;
  transmla_status_t st = check_shape(p, false);
  if (st != TRANSMLA_OK) return st;
  int G = p->num_partitions;
  if (G == 0) {
    int sms = 0;
    st = check_device(&sms);
    if (st != TRANSMLA_OK) return st;
    const int row_blocks = (p->q_len * p->num_heads + kRowBlock - 1) / kRowBlock;
    G = sms / row_blocks;
    // Small problems: no more partitions than a quarter of the pages the batch can hold, so that a partition
    // keeps at least about four pages and a sequence is not cut into dozens of one-page partials.
    const long long cap = (static_cast<long long>(p->batch) * p->max_pages_per_seq + 3) / 4;
    if (G > cap) G = static_cast<int>(cap);
    if (G < 1) G = 1;
  }
  const size_t B = p->batch, SH = static_cast<size_t>(p->q_len) * p->num_heads;
  const size_t K = p->kv_lora_rank + p->qk_rope_dim;
  const size_t slots = static_cast<size_t>(G) + B - 1;
  size_t off = 0;
  out->num_partitions = G;
  out->num_slots = static_cast<int32_t>(slots);
  out->q_hat_offset = off;       off = round_up(off + B * SH * K * sizeof(__nv_bfloat16), kAlign);
  out->cum_pages_offset = off;   off = round_up(off + (3 * B + 1 + (SH + kRowBlock - 1) / kRowBlock * B) * sizeof(int32_t), kAlign);
  out->plan_offset = off;        off = round_up(off + static_cast<size_t>(G) * 4 * sizeof(int32_t), kAlign);
  out->partial_o_offset = off;   off = round_up(off + slots * SH * p->kv_lora_rank * sizeof(float), kAlign);
  out->partial_lse_offset = off; off = round_up(off + slots * SH * sizeof(float), kAlign);
  out->total_bytes = off;
  return TRANSMLA_OK;
}

transmla_status_t transmla_latent_append(const transmla_params_t* p, const void* x, const void* w_dkv_kr,
                                         const int32_t* positions, const int32_t* page_table, void* cache,
                                         int32_t* dev_status, void* stream) {
  transmla_status_t st = check_shape(p, true);
  if (st != TRANSMLA_OK) return st;
  if (!x || !w_dkv_kr || !positions || !page_table || !cache) return TRANSMLA_ERR_NULL;
  if (!aligned(x, 16) || !aligned(w_dkv_kr, 16) || !aligned(positions, 4) || !aligned(page_table, 4) ||
      !aligned(cache, 128) || !aligned(dev_status, 4))
    return TRANSMLA_ERR_ALIGN;
  st = check_device(nullptr);
  if (st != TRANSMLA_OK) return st;
  cudaError_t e = launch_append(*p, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w_dkv_kr),
                                positions, page_table, static_cast<__nv_bfloat16*>(cache), dev_status,
                                static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

static transmla_status_t check_decode_args(const transmla_params_t* p, const void* q_nope, const void* q_pe,
                                           const void* w_uk, const void* cache, const int32_t* page_table,
                                           const int32_t* seqlens, void* workspace, size_t workspace_bytes,
                                           int32_t* dev_status, transmla_workspace_layout_t* lay) {
  transmla_status_t st = transmla_workspace_layout(p, lay);
  if (st != TRANSMLA_OK) return st;
  if (!q_nope || !w_uk || !cache || !page_table || !seqlens || !workspace) return TRANSMLA_ERR_NULL;
  if (p->qk_rope_dim > 0 && !q_pe) return TRANSMLA_ERR_NULL;
  if (!aligned(q_nope, 16) || !aligned(q_pe, 16) || !aligned(w_uk, 16) || !aligned(cache, 128) ||
      !aligned(page_table, 4) || !aligned(seqlens, 4) || !aligned(workspace, kAlign) || !aligned(dev_status, 4))
    return TRANSMLA_ERR_ALIGN;
  if (workspace_bytes < lay->total_bytes) return TRANSMLA_ERR_WORKSPACE;
  return check_device(nullptr);
}

// Host-side checks of a whole decode step, for callers inside the library that launch other kernels first.
extern "C++" {
namespace transmla {
transmla_status_t validate_step_args(const transmla_params_t* p, const void* x, const void* q_nope, const void* q_pe,
                                     const void* w_dkv_kr, const void* w_uk, const void* w_uv, const void* cache,
                                     const int32_t* page_table, const int32_t* seqlens, void* workspace,
                                     size_t workspace_bytes, const void* out, int32_t* dev_status) {
  transmla_status_t st = check_shape(p, true);
  if (st != TRANSMLA_OK) return st;
  if (!x || !w_dkv_kr || !w_uv || !out) return TRANSMLA_ERR_NULL;
  if (!aligned(x, 16) || !aligned(w_dkv_kr, 16) || !aligned(w_uv, 16) || !aligned(out, 16)) return TRANSMLA_ERR_ALIGN;
  transmla_workspace_layout_t lay;
  return check_decode_args(p, q_nope, q_pe, w_uk, cache, page_table, seqlens, workspace, workspace_bytes, dev_status, &lay);
}
}  // namespace transmla
}  // extern "C++"

// The split-KV kernel, bracketed by the caller's timing events when the profiling hook is armed.
static transmla_status_t launch_split_kv(const transmla_params_t* p, const transmla_workspace_layout_t& lay,
                                         const void* cache, const int32_t* page_table, const int32_t* seqlens,
                                         char* ws, int32_t* dev_status, cudaStream_t s) {
  cudaEvent_t ev0 = tl_prof_start, ev1 = tl_prof_stop;
  tl_prof_start = tl_prof_stop = nullptr;
  if (ev0 != nullptr && cudaEventRecord(ev0, s) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  auto launch = decode_sm100_supported(*p) ? launch_decode_sm100 : launch_decode_generic;
  if (launch(*p, lay.num_partitions, reinterpret_cast<__nv_bfloat16*>(ws + lay.q_hat_offset),
             static_cast<const __nv_bfloat16*>(cache), page_table, seqlens,
             reinterpret_cast<int32_t*>(ws + lay.cum_pages_offset), reinterpret_cast<int32_t*>(ws + lay.plan_offset),
             reinterpret_cast<float*>(ws + lay.partial_o_offset), reinterpret_cast<float*>(ws + lay.partial_lse_offset),
             dev_status, s) != cudaSuccess)
    return TRANSMLA_ERR_CUDA;
  if (ev1 != nullptr && cudaEventRecord(ev1, s) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  return TRANSMLA_OK;
}

transmla_status_t transmla_mla_decode(const transmla_params_t* p, const void* q_nope, const void* q_pe,
                                      const void* w_uk, const void* cache, const int32_t* page_table,
                                      const int32_t* seqlens, void* workspace, size_t workspace_bytes,
                                      int32_t* dev_status, void* stream) {
  transmla_workspace_layout_t lay;
  transmla_status_t st = check_decode_args(p, q_nope, q_pe, w_uk, cache, page_table, seqlens, workspace,
                                           workspace_bytes, dev_status, &lay);
  if (st != TRANSMLA_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  if (launch_absorb_plan(*p, lay.num_partitions, static_cast<const __nv_bfloat16*>(q_nope),
                         static_cast<const __nv_bfloat16*>(q_pe), static_cast<const __nv_bfloat16*>(w_uk),
                         reinterpret_cast<__nv_bfloat16*>(ws + lay.q_hat_offset), seqlens,
                         reinterpret_cast<int32_t*>(ws + lay.cum_pages_offset),
                         reinterpret_cast<int32_t*>(ws + lay.plan_offset), dev_status, s) != cudaSuccess)
    return TRANSMLA_ERR_CUDA;
  return launch_split_kv(p, lay, cache, page_table, seqlens, ws, dev_status, s);
}

transmla_status_t transmla_mla_combine(const transmla_params_t* p, const void* workspace, size_t workspace_bytes,
                                       const void* w_uv, void* out, float* lse_out, int32_t* dev_status,
                                       void* stream) {
  transmla_workspace_layout_t lay;
  transmla_status_t st = transmla_workspace_layout(p, &lay);
  if (st != TRANSMLA_OK) return st;
  if (!workspace || !w_uv || !out) return TRANSMLA_ERR_NULL;
  if (!aligned(workspace, kAlign) || !aligned(w_uv, 16) || !aligned(out, 16) || !aligned(lse_out, 4))
    return TRANSMLA_ERR_ALIGN;
  if (workspace_bytes < lay.total_bytes) return TRANSMLA_ERR_WORKSPACE;
  st = check_device(nullptr);
  if (st != TRANSMLA_OK) return st;
  const char* ws = static_cast<const char*>(workspace);
  cudaError_t e = launch_combine(*p, lay.num_partitions, reinterpret_cast<const int32_t*>(ws + lay.cum_pages_offset),
                                 reinterpret_cast<const float*>(ws + lay.partial_o_offset),
                                 reinterpret_cast<const float*>(ws + lay.partial_lse_offset),
                                 static_cast<const __nv_bfloat16*>(w_uv), static_cast<__nv_bfloat16*>(out), lse_out,
                                 dev_status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

transmla_status_t transmla_latent_append_fp8(const transmla_params_t* p, const void* x, const void* w_dkv_kr,
                                             const int32_t* positions, const int32_t* page_table, void* cache_fp8,
                                             void* scratch, size_t scratch_bytes, int32_t* dev_status, void* stream) {
  transmla_status_t st = check_shape(p, true);
  if (st != TRANSMLA_OK) return st;
  if (!decode_fp8_supported(*p)) return TRANSMLA_ERR_SHAPE;
  if (!x || !w_dkv_kr || !positions || !page_table || !cache_fp8 || !scratch) return TRANSMLA_ERR_NULL;
  if (!aligned(x, 16) || !aligned(w_dkv_kr, 16) || !aligned(positions, 4) || !aligned(page_table, 4) ||
      !aligned(cache_fp8, 128) || !aligned(scratch, 16) || !aligned(dev_status, 4))
    return TRANSMLA_ERR_ALIGN;
  const size_t need = static_cast<size_t>(p->batch) * p->q_len * (p->kv_lora_rank + p->qk_rope_dim) * sizeof(float);
  if (scratch_bytes < need) return TRANSMLA_ERR_WORKSPACE;
  st = check_device(nullptr);
  if (st != TRANSMLA_OK) return st;
  cudaError_t e = launch_append_fp8(*p, static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(w_dkv_kr),
                                    positions, page_table, cache_fp8, static_cast<float*>(scratch), dev_status,
                                    static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

transmla_status_t transmla_mla_decode_fp8(const transmla_params_t* p, const void* q_nope, const void* q_pe,
                                          const void* w_uk, const void* cache_fp8, const int32_t* page_table,
                                          const int32_t* seqlens, void* workspace, size_t workspace_bytes,
                                          int32_t* dev_status, void* stream) {
  transmla_workspace_layout_t lay;
  transmla_status_t st = check_decode_args(p, q_nope, q_pe, w_uk, cache_fp8, page_table, seqlens, workspace,
                                           workspace_bytes, dev_status, &lay);
  if (st != TRANSMLA_OK) return st;
  if (!decode_fp8_supported(*p)) return TRANSMLA_ERR_SHAPE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  if (launch_absorb_plan(*p, lay.num_partitions, static_cast<const __nv_bfloat16*>(q_nope),
                         static_cast<const __nv_bfloat16*>(q_pe), static_cast<const __nv_bfloat16*>(w_uk),
                         reinterpret_cast<__nv_bfloat16*>(ws + lay.q_hat_offset), seqlens,
                         reinterpret_cast<int32_t*>(ws + lay.cum_pages_offset),
                         reinterpret_cast<int32_t*>(ws + lay.plan_offset), dev_status, s) != cudaSuccess)
    return TRANSMLA_ERR_CUDA;
  cudaEvent_t ev0 = tl_prof_start, ev1 = tl_prof_stop;
  tl_prof_start = tl_prof_stop = nullptr;
  if (ev0 != nullptr && cudaEventRecord(ev0, s) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  if (launch_decode_fp8(*p, lay.num_partitions, reinterpret_cast<__nv_bfloat16*>(ws + lay.q_hat_offset), cache_fp8, page_table,
                        seqlens, reinterpret_cast<int32_t*>(ws + lay.cum_pages_offset),
                        reinterpret_cast<int32_t*>(ws + lay.plan_offset), reinterpret_cast<float*>(ws + lay.partial_o_offset),
                        reinterpret_cast<float*>(ws + lay.partial_lse_offset), dev_status, s) != cudaSuccess)
    return TRANSMLA_ERR_CUDA;
  if (ev1 != nullptr && cudaEventRecord(ev1, s) != cudaSuccess) return TRANSMLA_ERR_CUDA;
  return TRANSMLA_OK;
}

int transmla_page_claims_at_run_time(const transmla_params_t* p) {
  transmla_workspace_layout_t lay;
  if (transmla_workspace_layout(p, &lay) != TRANSMLA_OK) return 0;
  return dynamic_claims(*p, lay.num_partitions) ? 1 : 0;
}

transmla_status_t transmla_stream_probe(const transmla_params_t* p, const void* cache, const int32_t* page_table,
                                        const void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                        void* stream) {
  transmla_workspace_layout_t lay;
  transmla_status_t st = transmla_workspace_layout(p, &lay);
  if (st != TRANSMLA_OK) return st;
  if (!decode_sm100_supported(*p)) return TRANSMLA_ERR_SHAPE;
  if (!cache || !page_table || !workspace) return TRANSMLA_ERR_NULL;
  if (!aligned(cache, 128) || !aligned(page_table, 4) || !aligned(workspace, kAlign) || !aligned(dev_status, 4))
    return TRANSMLA_ERR_ALIGN;
  if (workspace_bytes < lay.total_bytes) return TRANSMLA_ERR_WORKSPACE;
  st = check_device(nullptr);
  if (st != TRANSMLA_OK) return st;
  const char* ws = static_cast<const char*>(workspace);
  cudaError_t e = launch_stream_probe(*p, lay.num_partitions, static_cast<const __nv_bfloat16*>(cache), page_table,
                                      reinterpret_cast<const int32_t*>(ws + lay.cum_pages_offset),
                                      reinterpret_cast<const int32_t*>(ws + lay.plan_offset), dev_status,
                                      static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

transmla_status_t transmla_validate_tables(const transmla_params_t* p, const int32_t* page_table,
                                           const int32_t* seqlens) {
  transmla_status_t st = check_shape(p, false);
  if (st != TRANSMLA_OK) return st;
  if (!page_table || !seqlens) return TRANSMLA_ERR_NULL;
  std::vector<bool> used(static_cast<size_t>(p->num_pages), false);
  for (int b = 0; b < p->batch; ++b) {
    const int64_t L = seqlens[b];
    if (L < 0 || L > static_cast<int64_t>(p->max_pages_per_seq) * kPage) return TRANSMLA_ERR_RANGE;
    const int n = static_cast<int>((L + kPage - 1) / kPage);
    for (int j = 0; j < n; ++j) {
      const int32_t idx = page_table[static_cast<size_t>(b) * p->max_pages_per_seq + j];
      if (idx < 0 || idx >= p->num_pages || used[idx]) return TRANSMLA_ERR_RANGE;
      used[idx] = true;
    }
  }
  return TRANSMLA_OK;
}

transmla_status_t transmla_decode_step(const transmla_params_t* p, const void* x, const void* q_nope,
                                       const void* q_pe, const int32_t* page_table, const int32_t* seqlens,
                                       const void* w_dkv_kr, const void* w_uk, const void* w_uv, void* cache,
                                       void* workspace, size_t workspace_bytes, void* out, float* lse_out,
                                       int32_t* dev_status, void* stream) {
  transmla_status_t st = check_shape(p, true);
  if (st != TRANSMLA_OK) return st;
  if (!x || !w_dkv_kr || !w_uv || !out) return TRANSMLA_ERR_NULL;
  if (!aligned(x, 16) || !aligned(w_dkv_kr, 16) || !aligned(w_uv, 16) || !aligned(out, 16) || !aligned(lse_out, 4))
    return TRANSMLA_ERR_ALIGN;
  transmla_workspace_layout_t lay;
  st = check_decode_args(p, q_nope, q_pe, w_uk, cache, page_table, seqlens, workspace, workspace_bytes, dev_status, &lay);
  if (st != TRANSMLA_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  if (launch_prologue(*p, lay.num_partitions, static_cast<const __nv_bfloat16*>(x),
                      static_cast<const __nv_bfloat16*>(w_dkv_kr), page_table, static_cast<__nv_bfloat16*>(cache),
                      static_cast<const __nv_bfloat16*>(q_nope), static_cast<const __nv_bfloat16*>(q_pe),
                      static_cast<const __nv_bfloat16*>(w_uk), reinterpret_cast<__nv_bfloat16*>(ws + lay.q_hat_offset),
                      seqlens, reinterpret_cast<int32_t*>(ws + lay.cum_pages_offset),
                      reinterpret_cast<int32_t*>(ws + lay.plan_offset), dev_status, s) != cudaSuccess)
    return TRANSMLA_ERR_CUDA;
  st = launch_split_kv(p, lay, cache, page_table, seqlens, ws, dev_status, s);
  if (st != TRANSMLA_OK) return st;
  return transmla_mla_combine(p, workspace, workspace_bytes, w_uv, out, lse_out, dev_status, stream);
}

size_t transmla_step_staging_bytes(const transmla_params_t* p) {
  if (check_shape(p, true) != TRANSMLA_OK) return 0;
  const size_t B = p->batch, S = p->q_len, H = p->num_heads;
  size_t off = 0;
  off = round_up(off + B * S * p->hidden_dim * 2, kAlign);                 // x
  off = round_up(off + B * S * H * p->qk_nope_dim * 2, kAlign);            // q_nope
  off = round_up(off + B * S * H * p->qk_rope_dim * 2 + 16, kAlign);       // q_pe
  off = round_up(off + B * p->max_pages_per_seq * 4, kAlign);              // page_table
  off = round_up(off + B * 4, kAlign);                                     // seqlens
  off = round_up(off + B * S * H * p->v_dim * 2, kAlign);                  // out
  off = round_up(off + B * S * H * 4, kAlign);                             // lse
  off = round_up(off + 4, kAlign);                                         // device status word
  return off;
}

transmla_status_t transmla_decode_step_host(const transmla_params_t* p, const void* h_x, const void* h_q_nope,
                                            const void* h_q_pe, const int32_t* h_page_table,
                                            const int32_t* h_seqlens, const void* w_dkv_kr, const void* w_uk,
                                            const void* w_uv, void* cache, void* staging, size_t staging_bytes,
                                            void* workspace, size_t workspace_bytes, void* h_out, float* h_lse,
                                            int32_t* h_dev_status, void* stream) {
  transmla_status_t st = check_shape(p, true);
  if (st != TRANSMLA_OK) return st;
  if (!h_x || !h_q_nope || !h_page_table || !h_seqlens || !w_dkv_kr || !w_uk || !w_uv || !cache || !staging ||
      !workspace || !h_out)
    return TRANSMLA_ERR_NULL;
  if (p->qk_rope_dim > 0 && !h_q_pe) return TRANSMLA_ERR_NULL;
  if (!aligned(staging, kAlign)) return TRANSMLA_ERR_ALIGN;
  if (staging_bytes < transmla_step_staging_bytes(p)) return TRANSMLA_ERR_WORKSPACE;
  const size_t B = p->batch, S = p->q_len, H = p->num_heads;
  const size_t nx = B * S * p->hidden_dim * 2, nqn = B * S * H * p->qk_nope_dim * 2, nqp = B * S * H * p->qk_rope_dim * 2;
  const size_t npt = B * p->max_pages_per_seq * 4, nout = B * S * H * p->v_dim * 2, nlse = B * S * H * 4;
  char* base = static_cast<char*>(staging);
  size_t off = 0;
  char* d_x = base + off;    off = round_up(off + nx, kAlign);
  char* d_qn = base + off;   off = round_up(off + nqn, kAlign);
  char* d_qp = base + off;   off = round_up(off + nqp + 16, kAlign);
  char* d_pt = base + off;   off = round_up(off + npt, kAlign);
  char* d_sl = base + off;   off = round_up(off + B * 4, kAlign);
  char* d_out = base + off;  off = round_up(off + nout, kAlign);
  char* d_lse = base + off;  off = round_up(off + nlse, kAlign);
  char* d_st = base + off;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  bool ok = true;
  const bool in_pinned = is_pinned_host(h_x) && is_pinned_host(h_q_nope) && (nqp == 0 || is_pinned_host(h_q_pe)) &&
                         is_pinned_host(h_page_table) && is_pinned_host(h_seqlens);
  if (in_pinned) {
    CopyList l = {};
    l.job[l.n++] = {h_x, d_x, nx};
    l.job[l.n++] = {h_q_nope, d_qn, nqn};
    if (nqp) l.job[l.n++] = {h_q_pe, d_qp, nqp};
    l.job[l.n++] = {h_page_table, d_pt, npt};
    l.job[l.n++] = {h_seqlens, d_sl, B * 4};
    l.zero_word = reinterpret_cast<int32_t*>(d_st);
    copy_list_kernel<<<dim3(copy_blocks(l), l.n), 256, 0, s>>>(l);
    ok &= cudaGetLastError() == cudaSuccess;
  } else {
    ok &= cudaMemcpyAsync(d_x, h_x, nx, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_qn, h_q_nope, nqn, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (nqp) ok &= cudaMemcpyAsync(d_qp, h_q_pe, nqp, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_pt, h_page_table, npt, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_sl, h_seqlens, B * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok &= cudaMemsetAsync(d_st, 0, 4, s) == cudaSuccess;
  }
  if (!ok) return TRANSMLA_ERR_CUDA;
  // The tables are checked on the host while the device already copies them: a bad table ends the call here,
  // before anything that uses the staged copies is launched.
  st = transmla_validate_tables(p, h_page_table, h_seqlens);
  if (st != TRANSMLA_OK) return st;
  for (int b = 0; b < p->batch; ++b)
    if (h_seqlens[b] < p->q_len) return TRANSMLA_ERR_RANGE;  // the step appends S tokens per sequence
  const bool out_pinned = is_pinned_host(h_out) && (h_lse == nullptr || is_pinned_host(h_lse));
  auto* dst = reinterpret_cast<int32_t*>(d_st);
  st = transmla_decode_step(p, d_x, d_qn, d_qp, reinterpret_cast<int32_t*>(d_pt), reinterpret_cast<int32_t*>(d_sl),
                            w_dkv_kr, w_uk, w_uv, cache, workspace, workspace_bytes,
                            d_out, reinterpret_cast<float*>(d_lse), dst, stream);
  if (st != TRANSMLA_OK) return st;
  int32_t dev_word = 0;
  int32_t* pinned_word = pinned_status_word();
  if (pinned_word != nullptr && out_pinned) {
    CopyList l = {};
    l.job[l.n++] = {d_out, h_out, nout};
    if (h_lse) l.job[l.n++] = {d_lse, h_lse, nlse};
    l.job[l.n++] = {d_st, pinned_word, 4};
    copy_list_kernel<<<dim3(copy_blocks(l), l.n), 256, 0, s>>>(l);
    ok &= cudaGetLastError() == cudaSuccess;
    ok &= cudaStreamSynchronize(s) == cudaSuccess;
    dev_word = *pinned_word;
  } else {
    ok &= cudaMemcpyAsync(h_out, d_out, nout, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    if (h_lse) ok &= cudaMemcpyAsync(h_lse, d_lse, nlse, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok &= cudaMemcpyAsync(&dev_word, d_st, 4, cudaMemcpyDeviceToHost, s) == cudaSuccess;
    ok &= cudaStreamSynchronize(s) == cudaSuccess;
  }
  if (h_dev_status) *h_dev_status = dev_word;
  return ok ? TRANSMLA_OK : TRANSMLA_ERR_CUDA;
}

const char* transmla_status_string(transmla_status_t status) {
  switch (status) {
    case TRANSMLA_OK: return "ok";
    case TRANSMLA_ERR_NULL: return "null pointer";
    case TRANSMLA_ERR_ALIGN: return "misaligned pointer";
    case TRANSMLA_ERR_SHAPE: return "unsupported shape";
    case TRANSMLA_ERR_RANGE: return "sequence length or page index out of range";
    case TRANSMLA_ERR_WORKSPACE: return "workspace too small";
    case TRANSMLA_ERR_CUDA: return "CUDA call failed";
    case TRANSMLA_ERR_ARCH: return "device is not sm_100";
  }
  return "unknown status";
}

}  // extern "C"
