// PTX wrappers shared by the kernels that run on the Blackwell tensor path (TMA loads, tcgen05.mma with
// accumulators in tensor memory), and the host-side look-up of the tensor-map encoder.
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>

#include <mutex>

#include "common.cuh"

namespace transmla {
namespace sm100 {

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// The same with an L2 eviction hint.  Cache pages are read once per step: marking them evict-first keeps the
// few MB of weights and split partials that the neighbouring kernels reuse resident in L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  return policy;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d), "r"(a), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

#define TM_R4(v, i) "=r"(v[i]), "=r"(v[i + 1]), "=r"(v[i + 2]), "=r"(v[i + 3])
#define TM_R16(v, i) TM_R4(v, i), TM_R4(v, i + 4), TM_R4(v, i + 8), TM_R4(v, i + 12)
#define TM_W4(v, i) "r"(v[i]), "r"(v[i + 1]), "r"(v[i + 2]), "r"(v[i + 3])
#define TM_W16(v, i) TM_W4(v, i), TM_W4(v, i + 4), TM_W4(v, i + 8), TM_W4(v, i + 12)

// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp gets lane (base lane + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : TM_R16(v, 0)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : TM_R16(v, 0), TM_R16(v, 16)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::TM_W16(v, 0), "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
      ::TM_W16(v, 0), TM_W16(v, 16), "r"(taddr)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte offsets
// (all in 16-byte units), descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
         (static_cast<uint64_t>(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// The same descriptor `bytes` further on (bytes is a multiple of 16; the tile stays inside the 256 KB window,
// so the 14-bit address field cannot carry).
__device__ __forceinline__ uint64_t desc_advance(uint64_t desc, uint32_t bytes) { return desc + (bytes >> 4); }
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool a_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(128 >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------- host
inline PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  });
  return fn;
}

// Tensor map of a dense row-major matrix [rows, cols] (bf16, or bytes) read in boxes of box_rows x box_cols elements,
// by default 64 bf16 columns (128 bytes) with the 128-byte swizzle.  Encoding one costs a driver call of about a microsecond and a decode step needs the same
// two every time (the cache pool and the workspace do not move), so the last few are kept, keyed by device, base
// address and geometry, behind a mutex.  A tensor map holds nothing but that address and geometry, so a cached one
// stays right for as long as the key matches, whatever has happened to the memory in between.
// kind: what the elements are and how a box is laid out in shared memory.
enum { TMAP_BF16_SW128 = 0, TMAP_U8_SW128 = 1, TMAP_U8_PLAIN = 2 };
struct TensorMapKey {
  int device;
  const void* base;
  uint64_t rows;
  uint32_t cols, box_rows, box_cols, kind;
  bool operator==(const TensorMapKey& o) const {
    return device == o.device && base == o.base && rows == o.rows && cols == o.cols && box_rows == o.box_rows &&
           box_cols == o.box_cols && kind == o.kind;
  }
};
inline bool tensor_map_2d(CUtensorMap* out, const void* base, uint64_t rows, uint32_t cols, uint32_t box_rows,
                          uint32_t box_cols = 64, uint32_t kind = TMAP_BF16_SW128) {
  constexpr int kSlots = 16;
  struct Slot { TensorMapKey key; CUtensorMap map; uint64_t used; };
  static std::mutex mutex;
  static Slot slots[kSlots] = {};
  static uint64_t tick = 0;
  TensorMapKey key = {current_device_slot(), base, rows, cols, box_rows, box_cols, kind};
  std::lock_guard<std::mutex> lock(mutex);
  int victim = 0;
  for (int i = 0; i < kSlots; ++i) {
    if (slots[i].used != 0 && slots[i].key == key) {
      slots[i].used = ++tick;
      *out = slots[i].map;
      return true;
    }
    if (slots[i].used < slots[victim].used) victim = i;
  }
  auto encode = encode_fn();
  if (encode == nullptr) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * (kind == TMAP_BF16_SW128 ? sizeof(__nv_bfloat16) : 1)};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t elem_strides[2] = {1, 1};
  CUtensorMap map;
  if (encode(&map, kind == TMAP_BF16_SW128 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
             const_cast<void*>(base), dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
             kind == TMAP_U8_PLAIN ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  slots[victim].key = key;
  slots[victim].map = map;
  slots[victim].used = ++tick;
  *out = map;
  return true;
}

}  // namespace sm100
}  // namespace transmla
