// Internal launcher interface between the C-ABI layer (ctx.cu) and the kernels.
// Every launcher enqueues on `stream`, never synchronises, and returns the CUDA error of the launch.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace moe {

// Raises a kernel's dynamic shared-memory limit once per kernel, device and size, so that steady-state launches
// make no driver calls besides the launch itself (which also keeps them legal while a stream is being captured).
cudaError_t ensure_dynamic_smem_impl(const void* kern, size_t bytes);
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kern, size_t bytes) {
  return ensure_dynamic_smem_impl(reinterpret_cast<const void*>(kern), bytes);
}

// Programmatic dependent launch: the kernels of the library are launched with "programmatic stream serialization
// allowed" (the GEMMs for small problems only, see kGemmOverlapMaxRows), so their CTAs may become resident and run their prologue (barrier set-up, tensor-memory allocation,
// tensor-map prefetch) while the previous kernel of the stream is still draining; pdl_wait() then blocks until that
// kernel has completed and its writes are visible.  Rules: every thread calls pdl_wait() before its first access to
// global memory (reads AND writes: the predecessor may still be reading what this kernel overwrites), and
// pdl_launch_dependents() right after it, which lets the NEXT kernel start its own prologue as soon as SM resources
// free up.  A step of six dependent kernels sheds the launch latency and prologue of each of them this way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(bool allow_overlap, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = allow_overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
// The GEMM kernels take the overlap only for problems of up to this many rows: measured on a B200, a step of a
// few hundred microseconds gains 7 % from it (six launch latencies and prologues hidden), while steps of several
// milliseconds LOSE 1.5-5 % when their GEMM launches carry the attribute (the small kernels keep it at every size;
// re-measured in the sustained regime with the small-M kernel's early set-up: a limit of 32768 rows or none at all
// changes nothing on the weight-streaming workloads and costs 3-6 % on the tensor-bound one).
#ifndef MOE_GEMM_OVERLAP_MAX_ROWS
#define MOE_GEMM_OVERLAP_MAX_ROWS 8192
#endif
constexpr int64_t kGemmOverlapMaxRows = MOE_GEMM_OVERLAP_MAX_ROWS;
#endif

// Device status codes (same values as moe_status in the public header).
constexpr int kStOk = 0;
constexpr int kStTimeout = 6;
constexpr int kStBadIndex = 7;

// ---- a1 route ------------------------------------------------------------------------------
cudaError_t launch_route(const float* logits, const float* bias, int T, int E, int k, float scale, int32_t* idx,
                         float* w, cudaStream_t stream, int* n_launches);

// ---- a2-a4 layout --------------------------------------------------------------------------
// Slots per warp-owned chunk in the multi-CTA path, and the scratch it needs.
constexpr int kLayoutChunk = 256;
inline size_t layout_scratch_ints(int64_t n_slots, int E) {
  int64_t chunks = (n_slots + kLayoutChunk - 1) / kLayoutChunk;
  return (size_t)(chunks > 0 ? chunks : 1) * (size_t)E;
}
cudaError_t launch_layout(const int32_t* topk_idx, int64_t n_slots, int E, int32_t* counts, int32_t* offsets,
                          int32_t* perm, int32_t* inv_perm, int32_t* scratch, int* status, cudaStream_t stream,
                          int* n_launches);

// ---- a5 permute, a9 combine ----------------------------------------------------------------
// H counts 2-byte columns (a row of H E4M3 codes is H/2 of them).  row_val / row_val_perm (optional): one fp32
// value per source row is copied to each of its destination rows.
// wait_limit_ns: time limit of the kernels' bounded waits (0 = the default of 2 s).
cudaError_t launch_permute(const void* x, const int32_t* inv_perm, void* x_perm, int T, int k, int H, int* status,
                           cudaStream_t stream, int* n_launches, const float* row_val = nullptr,
                           float* row_val_perm = nullptr, unsigned long long wait_limit_ns = 0);
cudaError_t launch_combine(const void* y_perm, const void* y_shared, const int32_t* inv_perm, const float* topk_w,
                           void* out, int T, int k, int H, int* status, cudaStream_t stream, int* n_launches,
                           unsigned long long wait_limit_ns = 0);

// ---- a6-a8 grouped GEMM --------------------------------------------------------------------
// One grouped GEMM pass:  out[r, :] = epilogue( A[r, :] . W[e]^T )  for r in expert e's segment.
//   gated:     W[e] is [2*n_feat, K]; out[r,i] = silu(A.W[e,i]) * (A.W[e,n_feat+i]),  i < n_feat
//   not gated: W[e] is [n_feat, K];   out[r,c] = A.W[e,c]
// offsets == nullptr means a single group of `fixed_rows` rows (the shared expert).
struct GemmProblem {
  const void* A;           // bf16 [rows_cap, K]
  const void* W;           // bf16 [E, (gated?2:1)*n_feat, K]
  void* out;               // bf16 [rows_cap, n_feat]
  const int32_t* offsets;  // [E+1] device, or nullptr
  int32_t fixed_rows;      // rows when offsets == nullptr
  int64_t rows_cap;        // rows addressable in A / out (capacity of the buffers)
  int64_t rows_bound;      // upper bound on the rows actually routed this call (T*k or T)
  int32_t E;               // experts in W and offsets
  int32_t n_feat;
  int32_t K;
  bool gated;
  int32_t e_begin = 0;     // this launch covers experts [e_begin, e_end) only (a prefill segment);
  int32_t e_end = -1;      // e_end < 0 means E
  // Row gather (tensor-core large-M gated pass only): when gather_src is set, A is not read; row p of the
  // operand is gather_src[perm[p] / top_k, :] instead (gather_src is bf16 [T, K], perm is [rows_bound]).
  const void* gather_src = nullptr;
  const int32_t* perm = nullptr;
  int32_t top_k = 1;
  // FP8 variant (tensor-core path only): A and W hold E4M3 codes; the result is scaled by
  // row_scale[row] * w_scale[expert, weight row] (w_scale: [E, (gated?2:1)*n_feat]) before the epilogue's maths.
  bool fp8 = false;
  const float* row_scale = nullptr;
  const float* w_scale = nullptr;
  // Bounded waits of the tensor-core kernels: time limit in nanoseconds (0 = the default of 2 s), and the
  // failure-detection hook (the TMA producer issues nothing, so every consumer wait runs into the limit).
  unsigned long long wait_limit_ns = 0;
  bool debug_stall = false;
  // Small-M kernel: two words of device memory, {next tile, CTAs finished}, zero before the launch; the launch's CTAs
  // take their tiles from the first (an atomic counter over the size-ordered tile list) and the last CTA to finish
  // puts both back to zero.  Consecutive launches of a stream must use different pairs: with the launch overlap the
  // next kernel's CTAs take tiles while this one's are still finishing.
  int* tile_counters = nullptr;
  // Preemption at tile granularity (small-M kernel only; both null = off).  Before it takes a tile a CTA reads
  // *yield_req; when it is non-zero the CTA finishes the tiles it has taken, adds one to *stopped and exits, and the
  // tile counter is left where it is: launching the same problem again with the same tile_counters goes on with the
  // tiles not yet taken.
  const int* yield_req = nullptr;
  int* stopped = nullptr;
  // Every launch of a pass that may be stopped and launched again sets this (also a launch without yield_req that
  // finishes such a pass): all its tiles come from the counter, none is dealt statically.
  bool resumable = false;
  // Small-M kernel: `offsets` was final before the previous kernel of the stream started, so the kernel may read it
  // (and fetch weights) before it waits for that kernel; only the rows of A (and the FP8 row scales) wait.
  bool offsets_settled = false;
  // Upper bound on the rows of any one group (a token reaches an expert at most once, so T), or 0 if unknown.  With
  // at most 16, every non-empty group is one tile of the same cost and the small-M kernel skips ordering them.
  int32_t max_group_rows = 0;
};

// A dense group (the shared expert) that rides in the same launch as a grouped problem: its tiles are added
// to the tile list, so a pass that would fill only a few CTAs by itself shares the persistent grid.
struct GemmDenseGroup {
  const void* A;    // bf16 [rows, K]
  const void* W;    // bf16 [(gated?2:1)*n_feat, K]
  void* out;        // bf16 [rows, n_feat]
  int32_t rows;
  int32_t n_feat;
  int32_t K;
  const float* row_scale = nullptr;  // FP8 variant: [rows]
  const float* w_scale = nullptr;    // FP8 variant: [(gated?2:1)*n_feat]
};

// FP8 variant: per-row dynamic quantisation of bf16 rows [rows, n] -> E4M3 codes [rows, n] + scale [rows]
// (n a multiple of 8, at most 8192).
cudaError_t launch_quantize_rows(const void* x, int64_t rows, int n, void* q, float* scale, cudaStream_t stream,
                                 int* n_launches);

cudaError_t launch_gemm_validation(const GemmProblem& p, cudaStream_t stream, int* n_launches);

// Tensor-core path (tcgen05 + TMEM + TMA), large-M variant: 128 tokens fill the MMA M dimension.  `max_ctas`
// caps the persistent grid.  Returns cudaErrorNotSupported for shapes it does not handle.
// `dense` (optional) is computed in the same launch with the same `gated` epilogue.
cudaError_t launch_gemm_tc(const GemmProblem& p, const GemmDenseGroup* dense, int max_ctas, int* status,
                           cudaStream_t stream, int* n_launches);
// Weight-streaming variant (swap-AB with the MMA N following each expert's row count, up to 256 tokens per tile,
// operands in a byte ring): the variant for experts of up to a few hundred rows, where the step is bound by the
// bytes the SMs ingest.  Same contract as launch_gemm_tc; no row gather.
cudaError_t launch_gemm_stream(const GemmProblem& p, const GemmDenseGroup* dense, int max_ctas, int* status,
                               cudaStream_t stream, int* n_launches);
// One-time driver entry-point lookup for tensor-map encoding; returns false (with a reason) if unavailable.
bool gemm_tc_init(const char** why);

}  // namespace moe
