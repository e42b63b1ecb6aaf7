// Stages a2-a4: per-expert counts, exclusive scan, stable token-to-expert permutation.
//
// The permutation must be bit-exact and run-to-run identical, so no slot is claimed with a global
// atomic.  The flat slots are cut into warp-owned chunks; a warp walks its chunk 32 slots at a time
// and ranks equal experts inside a step with __match_any_sync, which keeps ascending slot order.
//   small N (decode, low latency): ONE CTA does count -> scan -> place in shared memory, one launch.
//   large N (prefill):             count per chunk -> per-expert scan over chunks (one CTA per 32
//                                  experts) -> scan over experts and place per chunk.
#include <mutex>

#include "kernels.h"

namespace moe {
namespace {

constexpr int kFusedWarps = 32;           // single-CTA path: 32 warps
constexpr int kFusedMaxSlotsPerWarp = 512;  // -> up to 16384 slots in one CTA
constexpr int kChunkWarpsPerBlock = 4;    // multi-CTA path: warps (= chunks) per CTA

__device__ __forceinline__ void flag_status(int* status, int code) {
  if (status != nullptr) atomicCAS(status, kStOk, code);
}

constexpr int kBatch = 8;  // steps of 32 slots whose index loads are issued together (latency hiding)

// Counts one chunk [f0, f1) into hist[0..E) (shared memory, zeroed by the caller).
__device__ __forceinline__ void count_chunk(const int32_t* __restrict__ topk_idx, int64_t f0, int64_t f1, int E,
                                            int* hist, int* status) {
  const int lane = threadIdx.x & 31;
  for (int64_t base = f0; base < f1; base += 32 * kBatch) {
    int ev[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int64_t f = base + 32 * u + lane;
      ev[u] = (f < f1) ? __ldg(topk_idx + f) : 0;
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      if (base + 32 * u + lane >= f1) continue;
      const int e = ev[u];
      if (e >= 0 && e < E) atomicAdd(&hist[e], 1);  // integer adds commute: the count is order-independent
      else flag_status(status, kStBadIndex);
    }
  }
}

// Places one chunk.  run[e] holds the destination of the chunk's next slot of expert e.
__device__ __forceinline__ void place_chunk(const int32_t* __restrict__ topk_idx, int64_t f0, int64_t f1, int E,
                                            int* run, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
  const int lane = threadIdx.x & 31;
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int64_t base0 = f0; base0 < f1; base0 += 32 * kBatch) {
    int ev[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int64_t f = base0 + 32 * u + lane;
      ev[u] = (f < f1) ? __ldg(topk_idx + f) : -1;
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int64_t base = base0 + 32 * u;
      if (base >= f1) break;  // uniform across the warp
      const int64_t f = base + lane;
      const int e = ev[u];
      const bool valid = (e >= 0 && e < E);
      const int keyv = valid ? e : (E + lane);  // invalid lanes never group with anyone
      const unsigned peers = __match_any_sync(0xffffffffu, keyv);
      int p = -1;
      if (valid) p = run[e] + __popc(peers & lt_mask);
      __syncwarp();
      if (valid && (peers & lt_mask) == 0u) run[e] += __popc(peers);  // the lowest lane of a group advances it
      __syncwarp();
      if (f < f1) {
        inv_perm[f] = p;
        if (valid) perm[p] = (int32_t)f;
      }
    }
  }
}

// Block-wide exclusive scan of counts[0..E) -> offsets[0..E]; E <= 1024, blockDim.x a multiple of 32 and >= E...
// handled in rounds of blockDim.x so that any E works.  `warp_sums` is 33 ints of shared scratch.
__device__ void block_exclusive_scan(const int* counts_sh, int E, int32_t* __restrict__ offsets_out, int* offsets_sh,
                                     int* warp_sums) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int carry = 0;
  for (int base = 0; base < E; base += blockDim.x) {
    const int e = base + threadIdx.x;
    const int v = (e < E) ? counts_sh[e] : 0;
    int incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += n;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int ws = (lane < nwarps) ? warp_sums[lane] : 0;
      int wincl = ws;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, wincl, off);
        if (lane >= off) wincl += n;
      }
      if (lane < nwarps) warp_sums[lane] = wincl - ws;  // exclusive prefix of the warp totals
      if (lane == 31) warp_sums[32] = wincl;            // total of this round
    }
    __syncthreads();
    const int excl = carry + warp_sums[warp] + incl - v;
    if (e < E) {
      offsets_sh[e] = excl;
      if (offsets_out != nullptr) offsets_out[e] = excl;
    }
    carry += warp_sums[32];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    offsets_sh[E] = carry;
    if (offsets_out != nullptr) offsets_out[E] = carry;
  }
  __syncthreads();
}

// ---- single-CTA path: count, scan and place in one launch -------------------------------------
// shared memory: hist[kFusedWarps][E] | offsets_sh[E+1] | counts_sh[E] | warp_sums[33]
__global__ void __launch_bounds__(kFusedWarps * 32)
layout_fused_kernel(const int32_t* __restrict__ topk_idx, int n_slots, int E, int slots_per_warp,
                    int32_t* __restrict__ counts, int32_t* __restrict__ offsets, int32_t* __restrict__ perm,
                    int32_t* __restrict__ inv_perm, int* status) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ int sh[];
  int* hist = sh;
  int* offsets_sh = hist + kFusedWarps * E;
  int* counts_sh = offsets_sh + (E + 1);
  int* warp_sums = counts_sh + E;
  const int warp = threadIdx.x >> 5;

  for (int i = threadIdx.x; i < kFusedWarps * E; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const int64_t f0 = min((int64_t)warp * slots_per_warp, (int64_t)n_slots);
  const int64_t f1 = min(f0 + slots_per_warp, (int64_t)n_slots);
  count_chunk(topk_idx, f0, f1, E, hist + warp * E, status);
  __syncthreads();
  // per expert: exclusive prefix over the warps' chunks, total into counts
  for (int e = threadIdx.x; e < E; e += blockDim.x) {
    int sum = 0;
    for (int wv = 0; wv < kFusedWarps; ++wv) {
      const int c = hist[wv * E + e];
      hist[wv * E + e] = sum;
      sum += c;
    }
    counts_sh[e] = sum;
    counts[e] = sum;
  }
  __syncthreads();
  block_exclusive_scan(counts_sh, E, offsets, offsets_sh, warp_sums);
  int* run = hist + warp * E;
  for (int e = threadIdx.x & 31; e < E; e += 32) run[e] += offsets_sh[e];
  __syncwarp();
  place_chunk(topk_idx, f0, f1, E, run, perm, inv_perm);
}

// ---- multi-CTA path ------------------------------------------------------------------------------
// (1) per-chunk histograms: chunk_counts[chunk][e]
__global__ void __launch_bounds__(kChunkWarpsPerBlock * 32)
layout_count_kernel(const int32_t* __restrict__ topk_idx, int64_t n_slots, int E, int n_chunks,
                    int32_t* __restrict__ chunk_counts, int* status) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ int sh[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x * kChunkWarpsPerBlock + warp;
  int* hist = sh + warp * E;
  for (int e = lane; e < E; e += 32) hist[e] = 0;
  __syncwarp();
  if (chunk >= n_chunks) return;
  const int64_t f0 = (int64_t)chunk * kLayoutChunk;
  const int64_t f1 = min(f0 + kLayoutChunk, n_slots);
  count_chunk(topk_idx, f0, f1, E, hist, status);
  __syncwarp();
  for (int e = lane; e < E; e += 32) chunk_counts[(size_t)chunk * E + e] = hist[e];
}

// (2) per expert an exclusive prefix over chunks (in place) and the total -> counts.  One CTA per 32 experts;
//     warp w owns the w-th of 32 contiguous runs of chunks, lane l the CTA's l-th expert, so a warp's loads are
//     one 128-byte line per chunk and go out in batches of kBatch before anything depends on them.  A run of
//     at most kBatch chunks (up to 65536 slots) is read once and kept in registers for the second walk.
__global__ void __launch_bounds__(1024)
layout_scan_kernel(int32_t* __restrict__ chunk_counts, int n_chunks, int E, int32_t* __restrict__ counts) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int partial[32][33];
  const int lane = threadIdx.x & 31, part = threadIdx.x >> 5;
  const int e = blockIdx.x * 32 + lane;
  const bool active = e < E;
  const int per = (n_chunks + 31) / 32;
  const int c0 = min(part * per, n_chunks), c1 = min(c0 + per, n_chunks);
  int first[kBatch];  // the run's first batch
#pragma unroll
  for (int u = 0; u < kBatch; ++u) first[u] = (active && c0 + u < c1) ? chunk_counts[(size_t)(c0 + u) * E + e] : 0;
  int sum = 0;
#pragma unroll
  for (int u = 0; u < kBatch; ++u) sum += first[u];
  if (active) {
    for (int cb = c0 + kBatch; cb < c1; cb += kBatch) {
      int v[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) v[u] = (cb + u < c1) ? chunk_counts[(size_t)(cb + u) * E + e] : 0;
#pragma unroll
      for (int u = 0; u < kBatch; ++u) sum += v[u];
    }
  }
  partial[part][lane] = sum;
  __syncthreads();
  if (!active) return;
  int run = 0;
  for (int q = 0; q < part; ++q) run += partial[q][lane];
  if (part == 31) counts[e] = run + sum;
#pragma unroll
  for (int u = 0; u < kBatch; ++u) {
    if (c0 + u < c1) chunk_counts[(size_t)(c0 + u) * E + e] = run;
    run += first[u];
  }
  for (int cb = c0 + kBatch; cb < c1; cb += kBatch) {
    int v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) v[u] = (cb + u < c1) ? chunk_counts[(size_t)(cb + u) * E + e] : 0;
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      if (cb + u < c1) chunk_counts[(size_t)(cb + u) * E + e] = run;
      run += v[u];
    }
  }
}

// (3) every CTA scans the counts over experts itself (CTA 0 also stores the result -> offsets) and places its
//     chunks at offsets[e] + (prefix of earlier chunks)[e]
//     shared memory: run[warps][E] | counts_sh[E] | offsets_sh[E+1] | warp_sums[33]
__global__ void __launch_bounds__(kChunkWarpsPerBlock * 32)
layout_place_kernel(const int32_t* __restrict__ topk_idx, int64_t n_slots, int E, int n_chunks,
                    const int32_t* __restrict__ chunk_prefix, const int32_t* __restrict__ counts,
                    int32_t* __restrict__ offsets, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ int sh[];
  int* counts_sh = sh + kChunkWarpsPerBlock * E;
  int* offsets_sh = counts_sh + E;
  int* warp_sums = offsets_sh + (E + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int e = threadIdx.x; e < E; e += blockDim.x) counts_sh[e] = counts[e];
  __syncthreads();
  block_exclusive_scan(counts_sh, E, blockIdx.x == 0 ? offsets : nullptr, offsets_sh, warp_sums);
  const int chunk = blockIdx.x * kChunkWarpsPerBlock + warp;
  if (chunk >= n_chunks) return;
  int* run = sh + warp * E;
  for (int e = lane; e < E; e += 32) run[e] = offsets_sh[e] + chunk_prefix[(size_t)chunk * E + e];
  __syncwarp();
  const int64_t f0 = (int64_t)chunk * kLayoutChunk;
  const int64_t f1 = min(f0 + kLayoutChunk, n_slots);
  place_chunk(topk_idx, f0, f1, E, run, perm, inv_perm);
}

__global__ void layout_empty_kernel(int E, int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  pdl_wait();
  pdl_launch_dependents();
  for (int e = threadIdx.x; e <= E; e += blockDim.x) {
    if (e < E) counts[e] = 0;
    offsets[e] = 0;
  }
}

}  // namespace

cudaError_t launch_layout(const int32_t* topk_idx, int64_t n_slots, int E, int32_t* counts, int32_t* offsets,
                          int32_t* perm, int32_t* inv_perm, int32_t* scratch, int* status, cudaStream_t stream,
                          int* n_launches) {
  cudaError_t err;
  if (n_slots <= 0) {
    err = launch_pdl(true, layout_empty_kernel, dim3(1), dim3(256), 0, stream, E, counts, offsets);
    if (err == cudaSuccess && n_launches) *n_launches += 1;
    return err;
  }
  const size_t fused_smem = ((size_t)kFusedWarps * E + (E + 1) + E + 33) * sizeof(int);
  if (n_slots <= (int64_t)kFusedWarps * kFusedMaxSlotsPerWarp && fused_smem <= 200 * 1024) {
    int spw = (int)((n_slots + kFusedWarps - 1) / kFusedWarps);
    spw = (spw + 31) / 32 * 32;
    if ((err = ensure_dynamic_smem(layout_fused_kernel, fused_smem)) != cudaSuccess) return err;
    err = launch_pdl(true, layout_fused_kernel, dim3(1), dim3(kFusedWarps * 32), fused_smem, stream, topk_idx, (int)n_slots, E, spw, counts, offsets,
                                                                     perm, inv_perm, status);
    if (err == cudaSuccess && n_launches) *n_launches += 1;
    return err;
  }
  const int n_chunks = (int)((n_slots + kLayoutChunk - 1) / kLayoutChunk);
  const int blocks = (n_chunks + kChunkWarpsPerBlock - 1) / kChunkWarpsPerBlock;
  const size_t chunk_smem = (size_t)kChunkWarpsPerBlock * E * sizeof(int);
  if ((err = launch_pdl(true, layout_count_kernel, dim3(blocks), dim3(kChunkWarpsPerBlock * 32), chunk_smem, stream, topk_idx, n_slots, E, n_chunks,
                                                                                scratch, status)) != cudaSuccess) return err;
  if ((err = launch_pdl(true, layout_scan_kernel, dim3((E + 31) / 32), dim3(1024), 0, stream, scratch, n_chunks, E, counts)) != cudaSuccess) return err;
  const size_t place_smem = chunk_smem + ((size_t)E + (E + 1) + 33) * sizeof(int);
  launch_pdl(true, layout_place_kernel, dim3(blocks), dim3(kChunkWarpsPerBlock * 32), place_smem, stream, topk_idx, n_slots, E, n_chunks,
                                                                                scratch, counts, offsets, perm,
                                                                                inv_perm);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  if (n_launches) *n_launches += 3;
  return cudaSuccess;
}

}  // namespace moe

// ------------------------------------------------------------------------------------------------
// Dispatch layout for callers that cannot allocate.
//
// Some hosts of this library are not allowed to obtain device memory at the point where they need a
// layout: code that lives inside another framework's memory pool and must not disturb it, or a runtime
// that has handed all device memory to its own allocator and has no cudaMalloc left to call.  They cannot give a context a workspace either.  For
// them the chunk histograms of the multi-CTA path live in this fixed array instead.  It is part of the
// loaded module, so every GPU that loads the library holds these 256 KiB until the process exits.
#include "../../include/moe_pd.h"

namespace {

constexpr int kStaticScratchInts = 64 * 1024;  // 256 KiB: up to ceil(N/256) * E = 65536 histogram cells
static __device__ __align__(256) int32_t g_static_layout_scratch[kStaticScratchInts];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
int32_t* g_static_scratch_addr[kMaxDevices] = {};  // device address of the array, per device ordinal

}  // namespace

extern "C" moe_status moe_dispatch_layout_static(const int32_t* topk_idx, int32_t T, int32_t top_k,
                                                 int32_t n_experts, int32_t* counts, int32_t* offsets,
                                                 int32_t* perm, int32_t* inv_perm, void* cuda_stream) {
  if (T < 0 || top_k < 1 || n_experts < 1 || n_experts > 1024) return MOE_ERR_INVALID_ARG;
  if (!counts || !offsets || (T > 0 && (!topk_idx || !perm || !inv_perm))) return MOE_ERR_INVALID_ARG;
  const int64_t n_slots = (int64_t)T * top_k;
  if (n_slots > ((int64_t)1 << 30)) return MOE_ERR_CAPACITY;
  if (moe::layout_scratch_ints(n_slots, n_experts) > (size_t)kStaticScratchInts) return MOE_ERR_CAPACITY;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOE_ERR_CUDA;
  int32_t* scratch = nullptr;
  {
    // Set-up, once per device, with that device current: in host code the array's name is only a
    // stand-in for the symbol, so ask the runtime for the address the kernels must be given.
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_layout_scratch) != cudaSuccess || p == nullptr) {
        (void)cudaGetLastError();
        return MOE_ERR_CUDA;
      }
      g_static_scratch_addr[dev] = static_cast<int32_t*>(p);
    }
    scratch = g_static_scratch_addr[dev];
  }
  // Nothing in the scratch has to start at zero: the count kernel writes every histogram cell that the
  // scan and place kernels read afterwards, so what the previous call left behind is never seen.
  cudaError_t e = moe::launch_layout(topk_idx, n_slots, n_experts, counts, offsets, perm, inv_perm, scratch,
                                     /*status=*/nullptr, static_cast<cudaStream_t>(cuda_stream), nullptr);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return MOE_ERR_CUDA;
  }
  return MOE_OK;
}
