// Decode + combine for callers that cannot hand the library a workspace.
//
// Some hosts of this library run where device allocation is off the table: a serving loop whose
// memory pool was carved up at start-up and leaves nothing to ask cudaMalloc for, a plugin called
// from inside another framework's stream callback or capture region where allocating would
// synchronise the device, or a process whose allocator is owned by a runtime that this code may not
// call.  For them the split partials, the split plan and the absorbed queries live in a fixed array
// inside the library image instead of a caller buffer.
#include <mutex>

#include "common.cuh"

namespace {

// 16 MiB per GPU that loads the library, held until the process exits.
constexpr size_t kStaticWorkspaceBytes = size_t(16) << 20;
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

// In host code `g_static_workspace` is only a handle for the runtime, not a device address, so the
// address the kernels get is looked up once per device with that device current.
std::mutex g_mutex;
void* g_device_ptr[transmla::kMaxDevices] = {};

transmla_status_t static_workspace_ptr(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return TRANSMLA_ERR_CUDA; }
  if (dev < 0 || dev >= transmla::kMaxDevices) return TRANSMLA_ERR_CUDA;  // device ordinals beyond 63 are not served
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_device_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return TRANSMLA_ERR_CUDA;
    }
    g_device_ptr[dev] = p;
  }
  *out = g_device_ptr[dev];
  return TRANSMLA_OK;
}

}  // namespace

extern "C" {

size_t transmla_static_workspace_capacity(void) { return kStaticWorkspaceBytes; }

transmla_status_t transmla_mla_attention_static(const transmla_params_t* params, const void* q_nope, const void* q_pe,
                                                const void* w_uk, const void* w_uv, const void* cache,
                                                const int32_t* page_table, const int32_t* seqlens, void* out,
                                                float* lse_out, int32_t* dev_status, void* stream) {
  transmla_workspace_layout_t lay;
  transmla_status_t st = transmla_workspace_layout(params, &lay);
  if (st != TRANSMLA_OK) return st;
  if (lay.total_bytes > kStaticWorkspaceBytes) return TRANSMLA_ERR_WORKSPACE;  // problem too large for the built-in array
  void* ws = nullptr;
  st = static_workspace_ptr(&ws);
  if (st != TRANSMLA_OK) return st;
  // Every region of the workspace that a step reads is written earlier in the same step, so nothing
  // left over from the previous call needs clearing.
  st = transmla_mla_decode(params, q_nope, q_pe, w_uk, cache, page_table, seqlens, ws, kStaticWorkspaceBytes, dev_status,
                           stream);
  if (st != TRANSMLA_OK) return st;
  return transmla_mla_combine(params, ws, kStaticWorkspaceBytes, w_uv, out, lse_out, dev_status, stream);
}

}  // extern "C"
