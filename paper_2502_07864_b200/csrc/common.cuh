// Shared device helpers of the absorbed-MLA decode kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "transmla.h"

namespace transmla {

constexpr int kPage = 64;       // tokens per cache page (P)
constexpr int kRowBlock = 32;   // query rows (s*H + h) one CTA works on
constexpr int kSegCost = TRANSMLA_SEGMENT_COST_PAGES;  // virtual slots in front of every non-empty sequence
// Dynamic page claims of the split-KV kernel (r = 512, dR = 64, partition count chosen by the library): the CTAs
// whose partitions hold pages of a sequence take that sequence's pages one by one from a counter instead of
// keeping to the plan's ranges, so a CTA on a faster SM ends up with more pages.  The counters next[rb][b] (one per
// block of 32 query rows and sequence) sit behind the plan's prefix sums and partition ranges.
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void set_status(int32_t* dev_status, int bit) {
  if (dev_status != nullptr) atomicOr(dev_status, bit);
}

// A sequence length outside [0, max_pages * P] cannot be honoured, the page table has no entries for it: it is
// clamped, so that no look-up leaves the table's row, and reported through TRANSMLA_DEV_BAD_LEN.
__device__ __forceinline__ int clamped_len(int L, int max_pages, int32_t* dev_status) {
  const long long cap = static_cast<long long>(max_pages) * kPage;
  if (L >= 0 && L <= cap) return L;
  set_status(dev_status, TRANSMLA_DEV_BAD_LEN);
  return L < 0 ? 0 : static_cast<int>(cap);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte asynchronous global->shared copy; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(void* dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_u32(dst)), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t (&r)[2], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];\n"
               : "=r"(r[0]), "=r"(r[1])
               : "r"(smem_u32(p)));
}

// D += A(16x16, row) * B(16x8, col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// mbarrier and bulk-copy wrappers shared by the kernels that use the asynchronous copy engine.
constexpr long long kWaitCycles = 400000000LL;  // bound of every barrier wait, ~0.2 s at 2 GHz
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns at once when the CTA has already given up.  For diagnosis, bit 8 + i of the status word
// is set for every barrier slot i (position within its 256-byte block) on which a wait was still pending when the
// CTA gave up; the first of them is the one whose limit expired.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* dev_status) {
  if (*abort_flag) return;
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    const bool expired = clock64() - t0 > kWaitCycles;
    if (expired || *abort_flag) {
      *abort_flag = 1;
      set_status(dev_status, TRANSMLA_DEV_TIMEOUT | (1 << (8 + ((bar & 255u) >> 3))));
      return;
    }
  }
}
// True in exactly one lane of a converged warp.  Code around it stays warp-uniform, so descriptors and
// addresses can live in uniform registers instead of being moved there for every instruction.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}
// 1-D bulk copy global -> shared (16-byte aligned addresses, size a multiple of 16), completing on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// Programmatic dependent launch.  Every kernel of the step is launched so that it may start while the
// kernel before it in the stream is still draining: it calls pdl_trigger() at once (the kernel after it may
// be scheduled as soon as SM resources allow) and pdl_wait() before the first access to anything an earlier
// kernel of the stream may have produced or may still be reading.  Only weights are touched before the wait.
// Pointers to anything but weights are therefore never declared `const __restrict__`: that pair tells the compiler
// that the data cannot change while the kernel runs, which lets it issue the load above the wait (it did: the
// combine read the plan's page total before the plan block had written it, once the kernels before it ran long
// enough for its blocks to be resident that early).
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Per-device host-side bookkeeping.  Function attributes (the dynamic shared memory limit) and occupancy answers
// belong to one device, so what has been set or asked is remembered per device ordinal, in atomics: two host
// threads that race through the first call both make the (idempotent) runtime call, nothing else.
constexpr int kMaxDevices = 64;
inline int current_device_slot() {  // the current device's ordinal, or -1 (then nothing is remembered)
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
  return dev >= 0 && dev < kMaxDevices ? dev : -1;
}
struct PerDeviceFlag {
  std::atomic<int> value[kMaxDevices];
};
// Raises the kernel's dynamic shared memory limit on the current device, once per device.
template <typename Kernel>
cudaError_t ensure_dynamic_smem(Kernel kernel, int bytes, PerDeviceFlag& done) {
  const int slot = current_device_slot();
  if (slot >= 0 && done.value[slot].load(std::memory_order_acquire) != 0) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && slot >= 0) done.value[slot].store(1, std::memory_order_release);
  return e;
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Every host-side check of transmla_decode_step, without launching anything.
transmla_status_t validate_step_args(const transmla_params_t* p, const void* x, const void* q_nope, const void* q_pe,
                                     const void* w_dkv_kr, const void* w_uk, const void* w_uv, const void* cache,
                                     const int32_t* page_table, const int32_t* seqlens, void* workspace,
                                     size_t workspace_bytes, const void* out, int32_t* dev_status);

// Launchers (host).  Each enqueues on `stream` and returns the launch error, if any.
bool dynamic_claims(const transmla_params_t& p, int G);  // whether the split-KV kernel hands pages out at run time
cudaError_t launch_absorb_plan(const transmla_params_t& p, int G, const __nv_bfloat16* q_nope,
                               const __nv_bfloat16* q_pe, const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat,
                               const int32_t* seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status,
                               cudaStream_t stream);
cudaError_t launch_prologue(const transmla_params_t& p, int G, const __nv_bfloat16* x, const __nv_bfloat16* w_dkv_kr,
                            const int32_t* page_table, __nv_bfloat16* cache, const __nv_bfloat16* q_nope,
                            const __nv_bfloat16* q_pe, const __nv_bfloat16* w_uk, __nv_bfloat16* q_hat,
                            const int32_t* seqlens, int32_t* cum, int32_t* plan, int32_t* dev_status,
                            cudaStream_t stream);
cudaError_t launch_append(const transmla_params_t& p, const __nv_bfloat16* x, const __nv_bfloat16* w,
                          const int32_t* positions, const int32_t* page_table, __nv_bfloat16* cache,
                          int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_decode_generic(const transmla_params_t& p, int G, const __nv_bfloat16* q_hat,
                                  const __nv_bfloat16* cache, const int32_t* page_table, const int32_t* seqlens,
                                  const int32_t* cum, const int32_t* plan, float* partial_o, float* partial_lse,
                                  int32_t* dev_status, cudaStream_t stream);
bool decode_sm100_supported(const transmla_params_t& p);
cudaError_t launch_decode_sm100(const transmla_params_t& p, int G, const __nv_bfloat16* q_hat,
                                const __nv_bfloat16* cache, const int32_t* page_table, const int32_t* seqlens,
                                const int32_t* cum, const int32_t* plan, float* partial_o, float* partial_lse,
                                int32_t* dev_status, cudaStream_t stream);
bool decode_fp8_supported(const transmla_params_t& p);
cudaError_t launch_decode_fp8(const transmla_params_t& p, int G, const __nv_bfloat16* q_hat, const void* cache_fp8,
                              const int32_t* page_table, const int32_t* seqlens, const int32_t* cum, const int32_t* plan,
                              float* partial_o, float* partial_lse, int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_append_fp8(const transmla_params_t& p, const __nv_bfloat16* x, const __nv_bfloat16* w, const int32_t* positions,
                              const int32_t* page_table, void* cache_fp8, float* scratch, int32_t* dev_status,
                              cudaStream_t stream);
cudaError_t launch_stream_probe(const transmla_params_t& p, int G, const __nv_bfloat16* cache, const int32_t* page_table,
                                const int32_t* cum, const int32_t* plan, int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_combine(const transmla_params_t& p, int G, const int32_t* cum, const float* partial_o,
                           const float* partial_lse, const __nv_bfloat16* w_uv, __nv_bfloat16* out, float* lse_out,
                           int32_t* dev_status, cudaStream_t stream);

}  // namespace transmla
