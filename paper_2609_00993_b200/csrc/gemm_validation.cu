// Validation grouped GEMM on the CUDA cores: slow, short, and easy to check by eye.  It exists so that
// the whole layer can be compared with the CPU oracle independently of the tensor-core kernels, and
// to localise a fault to them.  Same contract as the tensor-core path (see GemmProblem).
#include <cuda_bf16.h>

#include "kernels.h"

namespace moe {
namespace {

constexpr int kTile = 64;   // rows and features per CTA
constexpr int kStepK = 16;  // contraction elements staged per step

// grid = (ceil(n_feat / 64), upper bound on sum_e ceil(rows_e / 64)); 256 threads, 4x4 outputs each.
template <bool GATED>
__global__ void __launch_bounds__(256)
gemm_validation_kernel(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ W,
                       __nv_bfloat16* __restrict__ out, const int32_t* __restrict__ offsets, int fixed_rows, int E,
                       int n_feat, int K) {
  __shared__ float As[kStepK][kTile + 1];
  __shared__ float Wg[kStepK][kTile + 1];
  __shared__ float Wu[GATED ? kStepK : 1][kTile + 1];
  __shared__ int s_e, s_row0, s_rows;
  pdl_wait();
  pdl_launch_dependents();

  if (threadIdx.x == 0) {  // which expert and which 64-row tile of it does blockIdx.y name?
    int tile = blockIdx.y, e = 0, found = -1, r0 = 0, nr = 0;
    for (; e < E; ++e) {
      const int beg = offsets ? offsets[e] : 0;
      const int cnt = offsets ? offsets[e + 1] - beg : fixed_rows;
      const int tiles = (cnt + kTile - 1) / kTile;
      if (tile < tiles) {
        found = e; r0 = beg + tile * kTile; nr = min(kTile, cnt - tile * kTile);
        break;
      }
      tile -= tiles;
    }
    s_e = found; s_row0 = r0; s_rows = nr;
  }
  __syncthreads();
  if (s_e < 0) return;
  const int e = s_e, row0 = s_row0, rows = s_rows;
  const int f0 = blockIdx.x * kTile;
  const size_t w_rows = (size_t)(GATED ? 2 : 1) * n_feat;
  const __nv_bfloat16* We = W + (size_t)e * w_rows * K;

  const int tr = (threadIdx.x / 16) * 4, tc = (threadIdx.x % 16) * 4;
  float accg[4][4] = {}, accu[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += kStepK) {
    for (int i = threadIdx.x; i < kTile * kStepK; i += 256) {
      const int r = i / kStepK, kk = i % kStepK;
      const bool kin = (k0 + kk) < K;
      As[kk][r] = (r < rows && kin) ? __bfloat162float(A[(size_t)(row0 + r) * K + k0 + kk]) : 0.f;
      const int f = f0 + r;
      Wg[kk][r] = (f < n_feat && kin) ? __bfloat162float(We[(size_t)f * K + k0 + kk]) : 0.f;
      if (GATED) Wu[kk][r] = (f < n_feat && kin) ? __bfloat162float(We[(size_t)(n_feat + f) * K + k0 + kk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kStepK; ++kk) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float a = As[kk][tr + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          accg[i][j] = fmaf(a, Wg[kk][tc + j], accg[i][j]);
          if (GATED) accu[i][j] = fmaf(a, Wu[kk][tc + j], accu[i][j]);
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = tr + i, f = f0 + tc + j;
      if (r < rows && f < n_feat) {
        float v = accg[i][j];
        if (GATED) v = v / (1.f + expf(-v)) * accu[i][j];
        out[(size_t)(row0 + r) * n_feat + f] = __float2bfloat16_rn(v);
      }
    }
  }
}

}  // namespace

cudaError_t launch_gemm_validation(const GemmProblem& p, cudaStream_t stream, int* n_launches) {
  if (p.rows_bound <= 0) return cudaSuccess;
  const int64_t groups = p.offsets ? p.E : 1;
  int64_t row_tiles = p.rows_bound / kTile + (groups < p.rows_bound ? groups : p.rows_bound);
  if (row_tiles > 65535) return cudaErrorNotSupported;
  dim3 grid((p.n_feat + kTile - 1) / kTile, (unsigned)row_tiles);
  const auto* A = static_cast<const __nv_bfloat16*>(p.A);
  const auto* W = static_cast<const __nv_bfloat16*>(p.W);
  auto* out = static_cast<__nv_bfloat16*>(p.out);
  const int e_begin = p.offsets ? p.e_begin : 0;
  const int e_end = (p.offsets && p.e_end >= 0) ? p.e_end : (int)groups;
  const int E = e_end - e_begin;  // experts of this launch
  const int32_t* offs = p.offsets ? p.offsets + e_begin : nullptr;
  W += (size_t)e_begin * (size_t)(p.gated ? 2 : 1) * p.n_feat * p.K;
  if (p.gated) (void)launch_pdl(true, gemm_validation_kernel<true>, grid, dim3(256), 0, stream, A, W, out, offs, p.fixed_rows, E, p.n_feat, p.K);
  else (void)launch_pdl(true, gemm_validation_kernel<false>, grid, dim3(256), 0, stream, A, W, out, offs, p.fixed_rows, E, p.n_feat, p.K);
  cudaError_t err = cudaGetLastError();
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

}  // namespace moe
