/*
 * transmla.h - C ABI of the absorbed-MLA decode library for NVIDIA B200 (sm_100a).
 *
 * The library computes one attention layer's decode step for a GQA model converted to
 * Multi-head Latent Attention (TransMLA, arXiv 2502.07864), in the Absorb form (Sec. 3.3, Eq. 9
 * right-hand column) directly over the compressed per-token latent cache
 *     k_hat_t = [ c_t^KV ; k_t^R ]        (r + dR values per token and layer).
 *
 * Symbols follow the paper: D hidden size, H (= h) query heads, dn (= d) per-head no-RoPE key dim,
 * dR (= d^R) decoupled RoPE dim, dv per-head value dim, r (= r_kv) latent rank; B sequences,
 * S new query tokens per sequence, L_b cached tokens of sequence b (the S new ones included),
 * P tokens per cache page.
 *
 * General rules for every entry point
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers are ordinary
 *     host memory.  The caller owns every buffer.  Unless an entry point says otherwise the library
 *     allocates nothing, frees nothing, never synchronises, and enqueues work only on `stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream).
 *   - All floating-point tensors are bfloat16 unless stated, dense, row-major, last index fastest.
 *     Accumulation is fp32; casts to bf16 round to nearest even.
 *   - Tensor bases must be 16-byte aligned; the cache base 128-byte aligned.
 *   - Problems that the host can see (null or misaligned pointer, unsupported shape, workspace too
 *     small, no sm_100 device) return an error code and launch nothing.  Problems only the device can
 *     see set bits in `*dev_status` (device int32, may be NULL; the caller zeroes it and reads it
 *     after synchronising) and never trap: a page-table entry outside [0, num_pages) is skipped
 *     (its tokens contribute nothing) and sets TRANSMLA_DEV_BAD_PAGE; a sequence length outside
 *     [0, max_pages_per_seq * P] is clamped to that range (no look-up leaves the page table's row) and
 *     sets TRANSMLA_DEV_BAD_LEN; a bounded wait that expired sets TRANSMLA_DEV_TIMEOUT and the affected
 *     results are unspecified.
 *   - Thread safety: entry points may be called from several host threads.  The library's own mutable
 *     state is: per-device "already set" flags for kernel attributes and cluster-occupancy answers
 *     (atomics; a race only repeats an idempotent runtime call), a per-device cache of the TMA
 *     descriptors of the cache pool and of the workspace (guarded by a mutex), the per-thread timing
 *     hook of transmla_profile_decode_kernel, a per-thread pinned status word used by
 *     transmla_decode_step_host, and the built-in array of transmla_mla_attention_static, which all
 *     calls on a device share (see the rule there).  Calls that use the same workspace, staging buffer or
 *     output buffers must be ordered by the caller.
 */
#ifndef TRANSMLA_H_
#define TRANSMLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TRANSMLA_OK = 0,
  TRANSMLA_ERR_NULL = 1,      /* a required pointer is NULL */
  TRANSMLA_ERR_ALIGN = 2,     /* a pointer violates the alignment rule */
  TRANSMLA_ERR_SHAPE = 3,     /* unsupported or inconsistent dimensions */
  TRANSMLA_ERR_RANGE = 4,     /* a sequence length or page index is out of range (host validation) */
  TRANSMLA_ERR_WORKSPACE = 5, /* workspace or staging buffer too small */
  TRANSMLA_ERR_CUDA = 6,      /* a CUDA runtime/driver call failed */
  TRANSMLA_ERR_ARCH = 7       /* the current device is not compute capability 10.x */
} transmla_status_t;

/* bytes of one token's row in the FP8 latent cache (r = 512, dR = 64): 512 e4m3 codes, 64 bf16, fp32 scale, padding */
#define TRANSMLA_FP8_ROW_BYTES 656

/* page-equivalents charged to a partition for every sequence it opens (split plan) */
#define TRANSMLA_SEGMENT_COST_PAGES 2

/* bits of the device status word; when TRANSMLA_DEV_TIMEOUT is set, bits 8 and up tell which of the kernel's
 * internal waits were still pending (diagnostic only, no stable meaning) */
#define TRANSMLA_DEV_BAD_PAGE 1
#define TRANSMLA_DEV_TIMEOUT 2
#define TRANSMLA_DEV_BAD_LEN 4
#define TRANSMLA_DEV_NUMERIC 8 /* conversion calls: an eigen-iteration did not converge, or a Gram matrix was singular */

typedef struct {
  int32_t hidden_dim;        /* D; used by the append only */
  int32_t num_heads;         /* H */
  int32_t q_len;             /* S >= 1 */
  int32_t qk_nope_dim;       /* dn */
  int32_t qk_rope_dim;       /* dR, even, may be 0 */
  int32_t v_dim;             /* dv */
  int32_t kv_lora_rank;      /* r */
  int32_t page_size;         /* P; must be 64 */
  int32_t num_pages;         /* pages in the cache pool */
  int32_t max_pages_per_seq; /* row stride of page_table */
  int32_t batch;             /* B */
  int32_t num_partitions;    /* G: how many pieces the batch's pages are split into; 0 = library chooses
                                (SMs / row blocks, at most batch * max_pages_per_seq / 4).  With an explicit G
                                every partition handles exactly the page range of the plan and a rerun gives
                                the same bits.  With 0, r = 512, dR = 64 and at least 8 partitions per
                                sequence, the CTAs that share a sequence take its pages from a counter as they
                                go (a CTA on a faster SM gets more): which pages meet in which partial then
                                depends on timing, and results can differ in the last fp32 bits between runs */
  float softmax_scale;       /* 1/sqrt(dn + dR) for MLA (Eq. 9), 1/sqrt(d) for a lifted GQA layer (Eq. 13) */
  float rope_theta;          /* RoPE base, 10000 in Eq. 1 */
} transmla_params_t;

/* Supported (r, dR) pairs: (512, 64), (128, 0), (64, 16).  dn: multiple of 16, dv: multiple of 8, both up to 256; D: multiple of 256.
 * S*H <= 1024.  page_size == 64. */

/* Byte offsets of the regions inside the workspace that carries results from
 * transmla_mla_decode to transmla_mla_combine.  All regions are written by transmla_mla_decode.
 *   q_hat       bf16  [B, S, H, r+dR]   absorbed queries (Eq. 9 right, first line)
 *   cum_pages   int32 [3B+1 + RB*B]     [0..B]: slot prefix sums (below); [B+1..3B]: per sequence the first and
 *                                       last partition that holds pages of it (0, -1 for an empty sequence);
 *                                       then one page counter per block of 32 query rows (RB = ceil(S*H/32)
 *                                       of them) and sequence, used when pages are handed out at run time.
 *                                       Prefix sums: a sequence with n_b = ceil(L_b/P) > 0 pages owns
 *                                       TRANSMLA_SEGMENT_COST_PAGES virtual slots followed by its n_b page
 *                                       slots; cum[b] = number of slots before sequence b
 *   plan        int32 [G, 4]            per partition: slot begin, end, sequence of first slot, sequence of
 *                                       last slot (-1, -1 for an empty partition); partition i owns slots
 *                                       [floor(i*T/G), floor((i+1)*T/G)), T = cum[B].  The virtual slots make
 *                                       a partition that opens a second sequence shorter by that many pages
 *   partial_o   fp32  [G+B-1, S*H, r]   per segment (partition i, sequence b), slot = i + b:
 *                                       softmax-weighted mean of c_j over the segment's visible tokens
 *   partial_lse fp32  [G+B-1, S*H]      natural-log softmax denominator of the segment (-inf = empty)
 * Row index inside a slot is s*H + h. */
typedef struct {
  int32_t num_partitions;  /* the G actually used */
  int32_t num_slots;       /* G + B - 1 */
  size_t q_hat_offset;
  size_t cum_pages_offset;
  size_t plan_offset;
  size_t partial_o_offset;
  size_t partial_lse_offset;
  size_t total_bytes;
} transmla_workspace_layout_t;

/* Workspace layout and size for `params` (host computation only; needs a CUDA device only when
 * params->num_partitions == 0, to read its SM count).  Returns TRANSMLA_OK or an error. */
transmla_status_t transmla_workspace_layout(const transmla_params_t* params /* host */,
                                            transmla_workspace_layout_t* layout /* host, out */);

/* Latent append (Sec. 3.3, Eq. 7 left column):
 *     c_t = W_DKV x_t,   k_t^R = RoPE(W_KR x_t, t)   (RoPE of Eq. 1: interleaved pairs, angle
 *     t * rope_theta^(-2l/dR) for pair l), rounded to bf16 and stored as the cache row of token t.
 * Token (b, s) has position positions[b] + s and goes to
 *     cache[page_table[b][pos / P]][pos % P][0 .. r+dR).
 *   x          device bf16 [B, S, D]
 *   w_dkv_kr   device bf16 [r+dR, D]: rows 0..r-1 = W_DKV, rows r.. = W_KR
 *   positions  device int32 [B], 0-based position of each sequence's first new token
 *   page_table device int32 [B, max_pages_per_seq]
 *   cache      device bf16 [num_pages, P, r+dR]; only the addressed rows are written
 * A position that maps outside the page table or to a page outside the pool is skipped and sets
 * TRANSMLA_DEV_BAD_PAGE. */
transmla_status_t transmla_latent_append(const transmla_params_t* params /* host */,
                                         const void* x, const void* w_dkv_kr, const int32_t* positions,
                                         const int32_t* page_table, void* cache, int32_t* dev_status,
                                         void* stream);

/* Absorb + split-KV decode (Eq. 9 right column, first and second line):
 *     q_hat[b,s,h] = [ W_UK_h^T q_nope[b,s,h] ; q_pe[b,s,h] ]
 *     o_hat[b,s,h] = sum_j softmax_j( q_hat . k_hat_j * softmax_scale ) c_j
 * over the visible tokens j in [0, L_b - (S-1-s)) of sequence b (the cache already holds the S new
 * tokens; query s sees everything up to and including its own token).  The batch's pages are split
 * into G partitions (see transmla_workspace_layout_t); each segment's normalised partial result and
 * log-sum-exp go to the workspace.  Rows of a page beyond L_b, and page-table entries beyond
 * ceil(L_b/P), are never used and may hold anything (NaN included).
 *   q_nope     device bf16 [B, S, H, dn]
 *   q_pe       device bf16 [B, S, H, dR]  RoPE already applied (ignored when dR == 0; may be NULL then)
 *   w_uk       device bf16 [H, dn, r]     k^C_h = W_UK_h c
 *   cache      device bf16 [num_pages, P, r+dR]
 *   page_table device int32 [B, max_pages_per_seq]
 *   seqlens    device int32 [B], 0 <= L_b <= max_pages_per_seq * P
 *   workspace  device, >= layout.total_bytes, 256-byte aligned */
transmla_status_t transmla_mla_decode(const transmla_params_t* params /* host */, const void* q_nope,
                                      const void* q_pe, const void* w_uk, const void* cache,
                                      const int32_t* page_table, const int32_t* seqlens, void* workspace,
                                      size_t workspace_bytes, int32_t* dev_status, void* stream);

/* Combine + up-projection (Eq. 9 right column, last line, before W_O):
 *     o_hat = sum_k w_k partial_o_k,  w_k = exp(lse_k - lse) with lse = log sum_k exp(lse_k),
 *     out[b,s,h] = W_UV_h o_hat[b,s,h].
 * Reads cum_pages, partial_o and partial_lse from the workspace a preceding transmla_mla_decode
 * with the same `params` filled.
 *   w_uv       device bf16 [H, dv, r]     v_h = W_UV_h c
 *   out        device bf16 [B, S, H, dv]
 *   lse_out    device fp32 [B, S, H] or NULL; natural log of the full softmax denominator
 * A query that sees no token (L_b - (S-1-s) <= 0) gets out = 0 and lse = -inf. */
transmla_status_t transmla_mla_combine(const transmla_params_t* params /* host */, const void* workspace,
                                       size_t workspace_bytes, const void* w_uv, void* out,
                                       float* lse_out, int32_t* dev_status, void* stream);

/* Host-side check of the index tables (host pointers): every L_b in [0, max_pages_per_seq*P], every
 * used page-table entry in [0, num_pages), no page used twice.  Returns TRANSMLA_OK or
 * TRANSMLA_ERR_RANGE.  Launches nothing. */
transmla_status_t transmla_validate_tables(const transmla_params_t* params /* host */,
                                           const int32_t* page_table /* host */,
                                           const int32_t* seqlens /* host */);

/* One whole decode step on device buffers: append the S new tokens of every sequence at positions
 * L_b - S .. L_b - 1 (what transmla_latent_append does with positions[b] = L_b - S), then what
 * transmla_mla_decode and transmla_mla_combine do, in three launches.  Same arguments and rules as
 * those three calls.  Every sequence needs L_b >= S. */
transmla_status_t transmla_decode_step(const transmla_params_t* params /* host */, const void* x,
                                       const void* q_nope, const void* q_pe, const int32_t* page_table,
                                       const int32_t* seqlens, const void* w_dkv_kr, const void* w_uk,
                                       const void* w_uv, void* cache, void* workspace,
                                       size_t workspace_bytes, void* out, float* lse_out, int32_t* dev_status,
                                       void* stream);

/* Weights of one converted attention layer for transmla_layer_decode_step (all device bf16, row-major).
 * Queries follow Eq. 8, right column: c^Q = W_DQ x, q^C = W_UQ c^Q, q^R = RoPE(W_QR c^Q, t).  With
 * w_dq == NULL the compression is skipped (full-rank queries, the other variant the paper runs): w_uq and
 * w_qr then act on x itself. */
typedef struct {
  const void* w_dq;      /* [r_q, D] or NULL */
  int32_t q_lora_rank;   /* r_q (multiple of 256); ignored when w_dq == NULL */
  const void* w_uq;      /* [H*dn, Dq], Dq = r_q or D: rows h*dn .. h*dn+dn-1 give q^C of head h */
  const void* w_qr;      /* [H*dR, Dq]: rows h*dR .. give q^R of head h before RoPE (NULL when dR == 0) */
  const void* w_dkv_kr;  /* [r+dR, D]   as in transmla_latent_append */
  const void* w_uk;      /* [H, dn, r]  as in transmla_mla_decode */
  const void* w_uv;      /* [H, dv, r]  as in transmla_mla_combine */
  const void* w_o;       /* [D, H*dv]:  y = W_O [o_1; ...; o_H]  (Eq. 9, last line) */
} transmla_layer_weights_t;

/* Bytes of device scratch transmla_layer_decode_step needs: c^Q, q^C, q^R and the attention output (bf16), plus
 * the partial sums and arrival counters of the K-sliced linear maps used from 48 new tokens on. */
size_t transmla_layer_scratch_bytes(const transmla_params_t* params /* host */, int32_t q_lora_rank);

/* The whole attention layer for the S newest tokens of every sequence, x [B, S, D] -> y [B, S, D] (device bf16):
 * queries (Eq. 8 right column, RoPE of q^R at position L_b - S + s), then the steps of transmla_decode_step (append,
 * absorb, split-KV decode, combine; with fewer than 48 new tokens the append's blocks run inside the layer's first
 * launch of linear maps, beside the queries), then the output projection W_O (Eq. 9, last line).  Every host-side
 * check of transmla_decode_step is made before anything is launched.  The linear maps are skinny
 * GEMMs with M = B*S that stream their weights once (mma.sync tiles; from 48 tokens on the large maps run as
 * TMA + tcgen05 tiles of 128 features with K cut into slices).  Needs D, H*dv (and r_q) multiples of 256; other rules
 * as for transmla_decode_step.  `scratch` is device memory of transmla_layer_scratch_bytes bytes, 256-byte
 * aligned. */
transmla_status_t transmla_layer_decode_step(const transmla_params_t* params /* host */,
                                             const transmla_layer_weights_t* weights /* host struct of device ptrs */,
                                             const void* x, const int32_t* page_table, const int32_t* seqlens,
                                             void* cache, void* workspace, size_t workspace_bytes, void* scratch,
                                             size_t scratch_bytes, void* y, int32_t* dev_status, void* stream);

/* Bytes of device staging transmla_decode_step_host needs for `params`. */
size_t transmla_step_staging_bytes(const transmla_params_t* params /* host */);

/* One whole decode step driven from host buffers: starts the copy of this step's inputs to the device
 * (x, q_nope, q_pe, page_table, seqlens), validates the tables on the host meanwhile (a bad table ends the
 * call before anything that uses the copies is launched), runs transmla_decode_step,
 * copies `out` (and `lse` if not NULL) back and waits for `stream`.  Weights and the cache stay
 * resident on the device.  When the host arrays are pinned (page-locked) the transfers are done by one
 * kernel each way that reads or writes the pinned memory directly; otherwise by one cudaMemcpyAsync per
 * array.  Uses host heap memory for the validation and, once per calling thread, 64 bytes of pinned host
 * memory for the status word; allocates no device memory.  Returns the first error, or
 * TRANSMLA_OK; `*h_dev_status` (host, may be NULL) receives the device status word.
 *   h_x [B,S,D], h_q_nope [B,S,H,dn], h_q_pe [B,S,H,dR], h_page_table, h_seqlens : host
 *   w_dkv_kr, w_uk, w_uv, cache, staging, workspace                              : device
 *   h_out [B,S,H,dv] bf16, h_lse [B,S,H] fp32 or NULL                            : host */
transmla_status_t transmla_decode_step_host(const transmla_params_t* params, const void* h_x,
                                            const void* h_q_nope, const void* h_q_pe,
                                            const int32_t* h_page_table, const int32_t* h_seqlens,
                                            const void* w_dkv_kr, const void* w_uk, const void* w_uv,
                                            void* cache, void* staging, size_t staging_bytes,
                                            void* workspace, size_t workspace_bytes, void* h_out,
                                            float* h_lse, int32_t* h_dev_status, void* stream);

/* Decode + combine without a caller workspace.  (The paper has no counterpart: this entry point
 * exists only for the sake of how the library is deployed.)
 *
 * Who needs it: callers that are not in a position to allocate device memory for the workspace -
 * an engine whose whole memory budget was handed out at start-up, code running inside another
 * runtime's callback or capture region where an allocation would stall the device, or a host
 * process whose device allocator belongs to a framework this library must not call into.
 *
 * What it does: exactly transmla_mla_decode followed by transmla_mla_combine, same arguments, same
 * results, but the workspace is a fixed array of transmla_static_workspace_capacity() bytes (16 MiB)
 * that is part of the library image; every GPU on which the library is loaded carries that array
 * until the process ends.  The call allocates and frees nothing on the device.
 *
 * Limits and rules:
 *   - transmla_workspace_layout(params).total_bytes must not exceed the capacity, otherwise the call
 *     returns TRANSMLA_ERR_WORKSPACE and launches nothing.  The size grows with
 *     (num_partitions + B - 1) * S * H * r * 4 bytes; pass a smaller params->num_partitions to fit.
 *   - The first call on each device looks up the array's device address (with that device current)
 *     and remembers it; make that first call outside any stream capture.  Device ordinals 0..63 are
 *     served; on a device beyond that the call returns TRANSMLA_ERR_CUDA.
 *   - All calls on a device share the one array and it keeps whatever the previous call left there.
 *     A step never reads a region it has not itself written first, so no clearing is needed, but two
 *     calls whose kernels can overlap on the GPU (different streams, no ordering) race on it: issue
 *     them on one stream or order them with events.
 *   q_nope, q_pe, w_uk, w_uv, cache, page_table, seqlens, out, lse_out, dev_status: device, as in
 *   transmla_mla_decode / transmla_mla_combine. */
size_t transmla_static_workspace_capacity(void);
transmla_status_t transmla_mla_attention_static(const transmla_params_t* params /* host */, const void* q_nope,
                                                const void* q_pe, const void* w_uk, const void* w_uv,
                                                const void* cache, const int32_t* page_table,
                                                const int32_t* seqlens, void* out, float* lse_out,
                                                int32_t* dev_status, void* stream);

/* Diagnostic: demonstrates the bounded waits of the kernels (no counterpart in the paper).  Launches one
 * block that waits, through the same helper the split-KV kernel uses, on a barrier that is never
 * satisfied.  After the limit (about 0.2 s) the wait gives up, TRANSMLA_DEV_TIMEOUT is set in *dev_status
 * (device int32, required), a second wait returns immediately and the kernel ends; the context stays
 * usable.  cycles_out (device int64[2], may be NULL) receives the SM cycles spent in the two waits. */
transmla_status_t transmla_selftest_bounded_wait(int32_t* dev_status, long long* cycles_out, void* stream);

/* FP8 latent cache (the paper's abstract names FP8 quantisation as combinable with the method and gives no detail; the
 * stored format is this library's own).  Only r = 512, dR = 64.  A token's row is TRANSMLA_FP8_ROW_BYTES = 656 bytes:
 *     bytes   0..511   e4m3 codes (OCP 8-bit float: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, largest
 *                      finite value 448, no infinities) of c_t / scale_t, nearest with ties to even
 *     bytes 512..639   k^R_t / scale_t as 64 bf16 values
 *     bytes 640..643   scale_t = max_i |c_t[i]| / 448 as fp32 (1.0 for an all-zero row); bytes 644..655 unused
 * and the cache is [num_pages, P, 656] bytes, 128-byte aligned.  What the attention sees is the dequantised row
 * scale_t * code, scale_t * (k^R_t / scale_t); results are Eq. 9 on those values.  |c| must stay below 65504 (the
 * products run on fp16 copies of scale_t * code).
 *
 * transmla_latent_append_fp8: transmla_latent_append into such a cache.  `scratch` is device memory of at least
 * B * S * (r + dR) * 4 bytes, 16-byte aligned (the rows in fp32 between the projection and the quantisation: a row's
 * scale needs all of its values).  Two launches.
 * transmla_mla_decode_fp8: transmla_mla_decode over such a cache; same workspace, and transmla_mla_combine finishes
 * the step exactly as for a bf16 cache.  The scores run as native e4m3 products on the stored codes, with every
 * absorbed query row split into two e4m3 terms (about the precision of its bf16 value). */
transmla_status_t transmla_latent_append_fp8(const transmla_params_t* params /* host */, const void* x,
                                             const void* w_dkv_kr, const int32_t* positions, const int32_t* page_table,
                                             void* cache_fp8, void* scratch, size_t scratch_bytes, int32_t* dev_status,
                                             void* stream);
transmla_status_t transmla_mla_decode_fp8(const transmla_params_t* params /* host */, const void* q_nope, const void* q_pe,
                                          const void* w_uk, const void* cache_fp8, const int32_t* page_table,
                                          const int32_t* seqlens, void* workspace, size_t workspace_bytes,
                                          int32_t* dev_status, void* stream);

/* Prefill in the MHA form (Sec. 3.3: the compute-bound paradigm; Eq. 8 and Eq. 9 left).  For a chunk of S = q_len
 * query positions per sequence - the last S of the L_b cached tokens, position s sees tokens [0, L_b - S + s] - the
 * keys and values are decompressed once, k^C_{j,h} = W_UK_h c_j and v_{j,h} = W_UV_h c_j (Eq. 8), and ordinary causal
 * attention runs per head on  z = q_nope . k^C + q_pe . k^R  (Eq. 9 left).  Same result as transmla_mla_decode +
 * transmla_mla_combine for the same arguments; it costs 2 * r * (dn + dv) FLOPs per token and head once, instead of
 * the absorbed form's wider products for every query row, and pays from a few hundred query positions per sequence
 * on.  Only r = 512, dR = 64, dn = dv = 128 (TRANSMLA_ERR_SHAPE otherwise); q_len up to 2^20 (the limit
 * S*H <= 1024 of the decode calls does not apply); num_partitions is ignored.
 *   scratch: device, 128-byte aligned, at least transmla_prefill_scratch_bytes(params) bytes =
 *     num_pages * P * H * (dn + dv) * 2: the decompressed store, row page*P + slot = [H][k^C (dn) | v (dv)] bf16,
 *     written for every page that the page table names for tokens < L_b (rows of tokens >= L_b as zeros).
 *   transmla_prefill_decompress fills it (one launch), transmla_prefill_attention reads it (one launch; `cache` is
 *     read again for k^R), transmla_mla_prefill does both.  A store filled once serves any number of chunks over
 *     the same cached tokens.
 *   q_nope [B,S,H,dn], q_pe [B,S,H,dR] (rotated), w_uk [H,dn,r], w_uv [H,dv,r], cache, page_table, seqlens,
 *   out [B,S,H,dv] bf16, lse [B,S,H] fp32 (may be NULL), dev_status: device, as in transmla_mla_decode.
 * Errors as for the decode calls; bad page indices and lengths are reported through *dev_status. */
size_t transmla_prefill_scratch_bytes(const transmla_params_t* params /* host */);
transmla_status_t transmla_prefill_decompress(const transmla_params_t* params /* host */, const void* cache,
                                              const int32_t* page_table, const int32_t* seqlens, const void* w_uk,
                                              const void* w_uv, void* scratch, size_t scratch_bytes, int32_t* dev_status,
                                              void* stream);
transmla_status_t transmla_prefill_attention(const transmla_params_t* params /* host */, const void* q_nope, const void* q_pe,
                                             const void* cache, const void* scratch, size_t scratch_bytes,
                                             const int32_t* page_table, const int32_t* seqlens, void* out, float* lse,
                                             int32_t* dev_status, void* stream);
transmla_status_t transmla_mla_prefill(const transmla_params_t* params /* host */, const void* q_nope, const void* q_pe,
                                       const void* w_uk, const void* w_uv, const void* cache, const int32_t* page_table,
                                       const int32_t* seqlens, void* scratch, size_t scratch_bytes, void* out, float* lse,
                                       int32_t* dev_status, void* stream);

/* Conversion of a GQA layer to MLA on calibration activations (Sec. 4.2, 4.3; App. B, C, D).  A one-off per model,
 * not part of the decode step.  Every matrix here is fp32, dense, row-major, device memory, 16-byte aligned; the
 * calls enqueue on `stream`, allocate nothing and report numerical trouble through TRANSMLA_DEV_NUMERIC in
 * *dev_status.  Index conventions: the merged key of Sec. 4.1 has g*d entries, entry (j, c) = j*d + c for original
 * head j and dimension c; RoPE pair l of a head is (2l, 2l+1) = (real, imaginary).  `fold` = M of App. C: group G
 * holds frequencies G*M .. G*M+M-1 and has g*M real and g*M imaginary entries, entry i = p*g + j for frequency
 * G*M + p and head j.
 *   transmla_conv_gemm: C[M,N] = alpha * op(A) op(B); op(A) = A [M,K] (ta = 0) or the transpose of A [K,M]
 *     (ta = 1), op(B) from B [K,N] (tb = 0) or B [N,K] (tb = 1); lda/ldb/ldc are row strides in elements.  Serves
 *     the calibration activations (K = X W^T), second moments (Z^T Z) and the low-rank rewrite of App. D.2
 *     (W_DKV' = R^T W_DKV, W_UKV' = W_UKV R).
 *   transmla_conv_rorope_covariance: App. B's sigma_x + sigma_y per frequency group from key activations
 *     K [n, g*d]: cov [d/2/fold, g*fold, g*fold].  scratch: transmla_conv_rorope_scratch_bytes(n, g, d, fold).
 *     g*fold <= 128.
 *   transmla_conv_sym_eig: eigenvalues (descending) and eigenvectors (columns of eigvecs [batch, m, m]) of `batch`
 *     symmetric matrices a [batch, m, m], m <= 128 (cyclic Jacobi).  App. B: U_l is eigvecs of cov[l].
 *   transmla_conv_rorope_apply: Eq. 18's rotation of the rows of X [g*d, C] (W^K, or merged queries/keys as
 *     columns) into Y: component q of group G goes to head q / fold, frequency G*fold + q % fold, the real and the
 *     imaginary rows with the same U_G [g*fold, g*fold] (U [d/2/fold, g*fold, g*fold]).  Y must not alias X.
 *   transmla_conv_alpha: Eq. 19, *alpha_out (device) = mean_t ||k_nope,t|| / mean_t ||v_t|| over the rows of
 *     k_nope [n, mk] and v [n, mv]; scratch: 2n floats.  Deterministic summation order.
 *   transmla_conv_balance_concat: Z [n, mk+mv] = [k_nope / alpha | v] (App. D.2 step 1), alpha read on the device.
 *   transmla_conv_top_subspace: App. D.2 step 2 for a second-moment matrix too large for Jacobi: an orthonormal
 *     basis Q [m, r] of the r leading eigenvectors' span of the symmetric positive semi-definite Cmat [m, m], by
 *     `iters` rounds of Q <- orth(Cmat Q) (Cholesky QR with the Gram matrix and its factor in fp64: one per round,
 *     two before the first round and one more after the last; r <= 1024).  Q holds the
 *     start basis on entry (full column rank, e.g. random numbers drawn by the caller).  Any orthonormal basis of
 *     the span gives the same converted layer (App. D.2: the latent may be re-based).  scratch: 256-byte aligned,
 *     transmla_conv_subspace_scratch_bytes(m, r). */
transmla_status_t transmla_conv_gemm(int ta, int tb, int M, int N, int K, float alpha, const float* A, int lda,
                                     const float* B, int ldb, float* C, int ldc, void* stream);
size_t transmla_conv_rorope_scratch_bytes(int n, int g, int d, int fold);
transmla_status_t transmla_conv_rorope_covariance(const float* K, int n, int g, int d, int fold, void* scratch,
                                                  size_t scratch_bytes, float* cov, void* stream);
transmla_status_t transmla_conv_sym_eig(float* a, int batch, int m, float* eigvals, float* eigvecs, int32_t* dev_status,
                                        void* stream);
transmla_status_t transmla_conv_rorope_apply(const float* X, int C, const float* U, int g, int d, int fold, float* Y,
                                             void* stream);
transmla_status_t transmla_conv_alpha(const float* k_nope, int n, int mk, const float* v, int mv, float* scratch,
                                      float* alpha_out, void* stream);
transmla_status_t transmla_conv_balance_concat(const float* k_nope, int n, int mk, const float* v, int mv,
                                               const float* alpha, float* Z, void* stream);
size_t transmla_conv_subspace_scratch_bytes(int m, int r);
transmla_status_t transmla_conv_top_subspace(const float* Cmat, int m, int r, int iters, float* Q, void* scratch,
                                             size_t scratch_bytes, int32_t* dev_status, void* stream);

/* Whether transmla_mla_decode with these `params` hands pages to CTAs at run time (1) or keeps to the page ranges of
 * the split plan (0); see transmla_params_t.num_partitions.  With run-time claims the default path is not
 * bit-stable from run to run (results agree to fp32 rounding); pass the partition count that
 * transmla_workspace_layout reports as an explicit num_partitions to get the planned, bit-stable path.  (No
 * counterpart in the paper: the split is this library's own.) */
int transmla_page_claims_at_run_time(const transmla_params_t* params /* host */);

/* Diagnostic: read-only streaming probe (no counterpart in the paper; it measures, it computes nothing).  Streams
 * exactly the pages that the split-KV kernel of transmla_mla_decode reads for `params` - same grid, same split
 * plan (taken from the workspace that a preceding transmla_mla_decode with the same `params` filled), same ring of
 * TMA page loads - and discards them.  Timed with events around it, it gives the floor that launch, ramp-up and
 * the memory system put under the split-KV kernel for this workload.  Only for r = 512, dR = 64
 * (TRANSMLA_ERR_SHAPE otherwise).  Writes nothing but *dev_status (bad page indices are reported as usual). */
transmla_status_t transmla_stream_probe(const transmla_params_t* params /* host */, const void* cache,
                                        const int32_t* page_table, const void* workspace, size_t workspace_bytes,
                                        int32_t* dev_status, void* stream);

/* Timing hook: the next transmla_mla_decode issued by the calling thread records `start_event`
 * immediately before and `stop_event` immediately after its split-KV kernel on that call's stream
 * (both cudaEvent_t passed as void*; NULL, NULL clears the hook).  The hook is consumed by that call. */
void transmla_profile_decode_kernel(void* start_event, void* stop_event);

/* Human-readable name of a status code (static storage). */
const char* transmla_status_string(transmla_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* TRANSMLA_H_ */
