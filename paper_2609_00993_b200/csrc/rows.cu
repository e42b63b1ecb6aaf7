// Stage a5 (routed row movement) and stage a9 (weighted combine).  Both are pure HBM streaming:
// every access is a 128-bit vector, a row is read once and written k times (permute) or k rows are
// gathered, summed in fp32 and written once (combine).
#include <cuda_bf16.h>

#include "kernels.h"

namespace moe {
namespace {

constexpr int kPermuteThreads = 256;
constexpr int kPermuteVecPerThread = 4;  // 16-byte vectors held in registers per pass
constexpr int kCombineThreads = 256;

// x_perm[inv_perm[t*k+j], :] = x[t, :]  for j < k.  One CTA walks tokens; a token's row is loaded once
// into registers and stored to its k destinations.
__global__ void __launch_bounds__(kPermuteThreads)
permute_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ inv_perm, uint4* __restrict__ x_perm,
                    int T, int k, int H8) {
  for (int t = blockIdx.x; t < T; t += gridDim.x) {
    const uint4* src = x + (size_t)t * H8;
    for (int v0 = 0; v0 < H8; v0 += kPermuteThreads * kPermuteVecPerThread) {
      uint4 val[kPermuteVecPerThread];
#pragma unroll
      for (int u = 0; u < kPermuteVecPerThread; ++u) {
        const int v = v0 + u * kPermuteThreads + threadIdx.x;
        if (v < H8) val[u] = __ldg(src + v);
      }
      for (int j = 0; j < k; ++j) {
        const int p = __ldg(inv_perm + (size_t)t * k + j);
        if (p < 0) continue;  // dropped slot (expert index was out of range)
        uint4* dst = x_perm + (size_t)p * H8;
#pragma unroll
        for (int u = 0; u < kPermuteVecPerThread; ++u) {
          const int v = v0 + u * kPermuteThreads + threadIdx.x;
          if (v < H8) dst[v] = val[u];
        }
      }
    }
  }
}

__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], const uint4& v, float w) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float2 f = __bfloat1622float2(h[q]);
    acc[2 * q] = fmaf(w, f.x, acc[2 * q]);
    acc[2 * q + 1] = fmaf(w, f.y, acc[2 * q + 1]);
  }
}

// out[t,:] = sum_j w[t,j] * y_perm[inv_perm[t*k+j],:] (+ y_shared[t,:]); ascending j, then the shared row.
// Persistent CTAs walk (token, 256-vector column block) items; a thread owns one 16-byte vector of the
// output row, keeps the k gathered loads in flight together, and fetches the next item's row indices and
// weights before it consumes the current rows, so the index -> row dependency is off the critical path.
// KU is the unroll width of the gather (k <= KU handled in one pass).
template <int KU>
__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const uint4* __restrict__ y_perm, const uint4* __restrict__ y_shared,
               const int32_t* __restrict__ inv_perm, const float* __restrict__ topk_w, uint4* __restrict__ out, int T,
               int k, int H8, int col_blocks) {
  const long long n_items = (long long)T * col_blocks;
  long long item = blockIdx.x;
  if (item >= n_items) return;
  int pj[KU];
  float wj[KU];
  auto load_meta = [&](long long it) {
    const int t = (int)(it / col_blocks);
#pragma unroll
    for (int u = 0; u < KU; ++u) {
      pj[u] = -1;
      wj[u] = 0.f;
      if (u < k) {
        pj[u] = __ldg(inv_perm + (size_t)t * k + u);
        wj[u] = __ldg(topk_w + (size_t)t * k + u);
      }
    }
  };
  load_meta(item);
  while (item < n_items) {
    const int t = (int)(item / col_blocks);
    const int v = (int)(item % col_blocks) * kCombineThreads + threadIdx.x;
    const bool in = v < H8;
    uint4 val[KU];
    float wc[KU];
#pragma unroll
    for (int u = 0; u < KU; ++u) {
      wc[u] = pj[u] >= 0 ? wj[u] : 0.f;
      val[u] = make_uint4(0u, 0u, 0u, 0u);
      if (in && pj[u] >= 0) val[u] = __ldg(y_perm + (size_t)pj[u] * H8 + v);
    }
    uint4 sh = make_uint4(0u, 0u, 0u, 0u);
    if (in && y_shared != nullptr) sh = __ldg(y_shared + (size_t)t * H8 + v);
    const long long next = item + gridDim.x;
    if (next < n_items) load_meta(next);  // issued while the rows above are still in flight
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < KU; ++u) fma_bf16x8(acc, val[u], wc[u]);
    // experts beyond KU (k > KU): plain second pass
    for (int j = KU; j < k; ++j) {
      const int pr = __ldg(inv_perm + (size_t)t * k + j);
      if (in && pr >= 0) fma_bf16x8(acc, __ldg(y_perm + (size_t)pr * H8 + v), __ldg(topk_w + (size_t)t * k + j));
    }
    if (y_shared != nullptr) fma_bf16x8(acc, sh, 1.0f);
    if (in) {
      uint4 o;
      __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int q = 0; q < 4; ++q) oh[q] = __floats2bfloat162_rn(acc[2 * q], acc[2 * q + 1]);
      out[(size_t)t * H8 + v] = o;
    }
    item = next;
  }
}

}  // namespace

cudaError_t launch_permute(const void* x, const int32_t* inv_perm, void* x_perm, int T, int k, int H,
                           cudaStream_t stream, int* n_launches) {
  if (T <= 0) return cudaSuccess;
  const int H8 = H / 8;
  const int blocks = T < 148 * 8 ? T : 148 * 8;
  permute_rows_kernel<<<blocks, kPermuteThreads, 0, stream>>>(static_cast<const uint4*>(x), inv_perm,
                                                              static_cast<uint4*>(x_perm), T, k, H8);
  cudaError_t err = cudaGetLastError();
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

cudaError_t launch_combine(const void* y_perm, const void* y_shared, const int32_t* inv_perm, const float* topk_w,
                           void* out, int T, int k, int H, cudaStream_t stream, int* n_launches) {
  if (T <= 0) return cudaSuccess;
  const int H8 = H / 8;
  const int col_blocks = (H8 + kCombineThreads - 1) / kCombineThreads;
  const long long n_items = (long long)T * col_blocks;
  const uint4* yp = static_cast<const uint4*>(y_perm);
  const uint4* ys = static_cast<const uint4*>(y_shared);
  uint4* o = static_cast<uint4*>(out);
  auto launch = [&](auto kern) {
    int dev = 0, sms = 148, per_sm = 2;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kCombineThreads, 0);
    const long long cap = (long long)sms * (per_sm > 0 ? per_sm : 1);  // one resident wave of persistent CTAs
    const int grid = (int)(n_items < cap ? n_items : cap);
    kern<<<grid, kCombineThreads, 0, stream>>>(yp, ys, inv_perm, topk_w, o, T, k, H8, col_blocks);
  };
  if (k > 4) launch(combine_kernel<8>);
  else if (k > 2) launch(combine_kernel<4>);
  else launch(combine_kernel<2>);
  cudaError_t err = cudaGetLastError();
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

}  // namespace moe
