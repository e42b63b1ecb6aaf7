// FP8 precision variant: per-row dynamic quantisation of bf16 activation rows to E4M3.
//
//   amax  = max(max_i |v_i|, 2^-100)       scale = amax / 448,  inv = 448 / amax
//   code_i = e4m3(v_i * inv)               round to nearest even, saturating at +-448
//
// The codes are integers decided by floating point, so every operation that decides them is spelled out in
// IEEE fp32 (__fdiv_rn once per row, __fmul_rn per element, cvt.rn.satfinite) and nothing is contracted or
// approximated.
// One warp (rows of up to 2048 elements) or one CTA of 128 threads (up to 8192) per row; the row stays in
// registers between the two passes, so it is read once: 2 n bytes in, n + 4 bytes out per row.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "kernels.h"

namespace moe {
namespace {

constexpr int kQuantThreads = 128;
constexpr int kQuantMaxVecs = 8;  // 16-byte vectors (8 bf16) per thread

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
  return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, __NV_E4M3);  // lo in bits 0-7
}

// ROW_WARPS = 4: one CTA per row (rows of up to 8192 elements).  ROW_WARPS = 1: one warp per row, four rows per
// CTA and no CTA-wide barrier (rows of up to 2048 elements).
template <int ROW_WARPS>
__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_kernel(const uint4* __restrict__ x, long long rows, int n_vec, uint2* __restrict__ q,
                     float* __restrict__ scale) {
  __shared__ uint32_t warp_max[kQuantThreads / 32];
  pdl_wait();
  pdl_launch_dependents();
  constexpr int kRowThreads = 32 * ROW_WARPS;
  const int tid = ROW_WARPS == 1 ? (int)(threadIdx.x & 31) : (int)threadIdx.x;
  const long long row = ROW_WARPS == 1 ? (long long)blockIdx.x * (kQuantThreads / 32) + (threadIdx.x >> 5)
                                       : (long long)blockIdx.x;
  if (ROW_WARPS == 1 && row >= rows) return;  // whole warps leave; there is no barrier on this path
  const uint4* xr = x + row * n_vec;
  uint4 v[kQuantMaxVecs];
  uint32_t m = 0;  // largest |bf16| as a bit pattern: for finite values the integer order is the value order
#pragma unroll
  for (int j = 0; j < kQuantMaxVecs; ++j) {
    const int i = tid + j * kRowThreads;
    v[j] = i < n_vec ? xr[i] : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      m = max(m, w[c] & 0x7fffu);
      m = max(m, (w[c] >> 16) & 0x7fffu);
    }
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if (ROW_WARPS > 1) {
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    m = max(max(warp_max[0], warp_max[1]), max(warp_max[2], warp_max[3]));
  }
  const float amax = fmaxf(bf16_bits_to_f32(m), 0x1p-100f);
  const float inv = __fdiv_rn(448.f, amax);
  if (tid == 0) scale[row] = __fdiv_rn(amax, 448.f);
  uint2* qr = q + row * n_vec;
#pragma unroll
  for (int j = 0; j < kQuantMaxVecs; ++j) {
    const int i = tid + j * kRowThreads;
    if (i >= n_vec) continue;
    const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
    uint32_t pair[4];
#pragma unroll
    for (int c = 0; c < 4; ++c)
      pair[c] = e4m3x2(__fmul_rn(bf16_bits_to_f32(w[c] & 0xffffu), inv), __fmul_rn(bf16_bits_to_f32(w[c] >> 16), inv));
    qr[i] = make_uint2(pair[0] | (pair[1] << 16), pair[2] | (pair[3] << 16));
  }
}

}  // namespace

cudaError_t launch_quantize_rows(const void* x, int64_t rows, int n, void* q, float* scale, cudaStream_t stream,
                                 int* n_launches) {
  if (rows <= 0) return cudaSuccess;
  if (n <= 0 || n % 8 != 0 || n > 8 * kQuantThreads * kQuantMaxVecs || rows > 0x7fffffffLL) return cudaErrorNotSupported;
  const int n_vec = n / 8;
  cudaError_t err;
  if (n_vec <= 32 * kQuantMaxVecs) {
    const long long blocks = (rows + kQuantThreads / 32 - 1) / (kQuantThreads / 32);
    err = launch_pdl(true, quantize_rows_kernel<1>, dim3((unsigned)blocks), dim3(kQuantThreads), 0, stream,
                     static_cast<const uint4*>(x), (long long)rows, n_vec, static_cast<uint2*>(q), scale);
  } else {
    err = launch_pdl(true, quantize_rows_kernel<4>, dim3((unsigned)rows), dim3(kQuantThreads), 0, stream,
                     static_cast<const uint4*>(x), (long long)rows, n_vec, static_cast<uint2*>(q), scale);
  }
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

}  // namespace moe
