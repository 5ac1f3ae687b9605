// Arguments of the linear-map launches (shared by the mma.sync and the tcgen05 implementation).
#pragma once
#include "common.cuh"

namespace transmla {

struct LinearJob {
  const __nv_bfloat16* x;   // [M, K]
  const __nv_bfloat16* w;   // [N, K]
  __nv_bfloat16* out;       // [M, N]
  int N, K;
  int rope_d;               // > 0: consecutive blocks of rope_d output features are rotated (Eq. 1, d := rope_d)
};
// Append blocks riding in a launch of linear maps (Eq. 7 left is one more linear map of the same x): blocks
// beyond those of the jobs run append_block.  blocks = 0: none.
struct AppendJob {
  const __nv_bfloat16* x;        // [B*S, D]
  const __nv_bfloat16* w;        // [r + dR, D]
  const int32_t* page_table;
  __nv_bfloat16* cache;
  int B, D, r, dR, num_pages, max_pages, t_splits, wide, blocks;
};
struct LinearArgs {
  LinearJob job[2];
  AppendJob append;
  int n_jobs, M, S, t_splits;
  const int32_t* pos_base;  // position of token (b, s) = pos_base[b] + pos_shift + s (used by rotated jobs only)
  int pos_shift;
  float theta;
};

// tcgen05 implementation (linear_sm100.cu): needs N a multiple of 128 and K a multiple of 64 in every job.
bool linear_sm100_supported(const LinearArgs& a);
int linear_sm100_splits(int n_tiles, int K);
size_t linear_sm100_partial_bytes(int n_tiles, int K, int M);   // scratch for the K slices' partial results
size_t linear_sm100_counter_bytes(int n_tiles, int M);          // per-tile arrival counters (zero before a launch)
cudaError_t launch_linear_sm100(const LinearArgs& a, float* partial, int32_t* counters, int32_t* dev_status,
                                cudaStream_t stream);

}  // namespace transmla
