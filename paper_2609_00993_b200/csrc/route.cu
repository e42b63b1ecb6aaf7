// Stage a1: top-k routing over given router logits.  One warp per token; each lane keeps
// ceil(E/32) selection keys in registers (128-bit loads when E is a multiple of 128), and k rounds of
// a shuffle arg-max on (key descending, expert index ascending) pick the experts.  The routed weights
// are a max-subtracted softmax over the k selected unbiased logits.
#include "kernels.h"

namespace moe {
namespace {

constexpr int kWarpsPerBlock = 8;

// Does candidate (v1, e1) come before (v0, e0) in the selection order?
__device__ __forceinline__ bool comes_before(float v1, int e1, float v0, int e0) {
  return (v1 > v0) || (v1 == v0 && e1 < e0);
}

// VPT: keys per lane (power of two >= ceil(E/32)).  VEC: lanes own runs of 4 consecutive experts.
template <int VPT, bool VEC>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
route_kernel(const float* __restrict__ logits, const float* __restrict__ bias, int T, int E, int k, float scale,
             int32_t* __restrict__ idx, float* __restrict__ w) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (t >= T) return;
  const float* row = logits + (size_t)t * E;

  // expert owned by this lane's i-th register; increasing in i so that "first wins" keeps the lower index
  auto expert_of = [&](int i) -> int { return VEC ? 128 * (i >> 2) + 4 * lane + (i & 3) : 32 * i + lane; };

  float key[VPT];
  if constexpr (VEC) {
#pragma unroll
    for (int q = 0; q < VPT / 4; ++q) {
      const int e0 = 128 * q + 4 * lane;
      if (e0 < E) {
        float4 v = *reinterpret_cast<const float4*>(row + e0);
        if (bias != nullptr) {
          float4 b = *reinterpret_cast<const float4*>(bias + e0);
          v.x = __fadd_rn(v.x, b.x); v.y = __fadd_rn(v.y, b.y); v.z = __fadd_rn(v.z, b.z); v.w = __fadd_rn(v.w, b.w);
        }
        key[4 * q + 0] = v.x; key[4 * q + 1] = v.y; key[4 * q + 2] = v.z; key[4 * q + 3] = v.w;
      } else {
        key[4 * q + 0] = key[4 * q + 1] = key[4 * q + 2] = key[4 * q + 3] = 0.f;
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int e = 32 * i + lane;
      float v = 0.f;
      if (e < E) {
        v = row[e];
        if (bias != nullptr) v = __fadd_rn(v, bias[e]);
      }
      key[i] = v;
    }
  }

  unsigned taken = 0u;  // bit i: this lane's i-th key is already selected
  int my_e = 0;         // lane j (< k) ends up holding the j-th selected expert
  for (int j = 0; j < k; ++j) {
    float bv = 0.f;
    int be = 0x7fffffff;
    bool has = false;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
      const int e = expert_of(i);
      const bool avail = (e < E) && !((taken >> i) & 1u);
      if (avail && (!has || key[i] > bv)) {
        bv = key[i]; be = e; has = true;
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
      const int oe = __shfl_xor_sync(0xffffffffu, be, off);
      const bool oh = __shfl_xor_sync(0xffffffffu, (int)has, off) != 0;
      if (oh && (!has || comes_before(ov, oe, bv, be))) {
        bv = ov; be = oe; has = true;
      }
    }
    be = __shfl_sync(0xffffffffu, be, 0);  // one answer for the warp even if the order was not total (NaN)
    const int owner = VEC ? ((be & 127) >> 2) : (be & 31);
    const int slot = VEC ? (4 * (be >> 7) + (be & 3)) : (be >> 5);
    if (lane == owner) taken |= (1u << slot);
    if (lane == j) my_e = be;
  }

  const bool active = lane < k;
  const float l = active ? row[my_e] : -INFINITY;
  float m = l;
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  const float p = active ? expf(l - m) : 0.f;
  float s = 0.f;
  for (int j = 0; j < k; ++j) s += __shfl_sync(0xffffffffu, p, j);  // summed in j order
  if (active) {
    idx[(size_t)t * k + lane] = my_e;
    w[(size_t)t * k + lane] = scale * p / s;
  }
}

template <int VPT>
cudaError_t launch_vpt(bool vec, const float* logits, const float* bias, int T, int E, int k, float scale,
                       int32_t* idx, float* w, cudaStream_t stream) {
  const int blocks = (T + kWarpsPerBlock - 1) / kWarpsPerBlock;
  if constexpr (VPT >= 4) {
    if (vec) {
      route_kernel<VPT, true><<<blocks, kWarpsPerBlock * 32, 0, stream>>>(logits, bias, T, E, k, scale, idx, w);
      return cudaGetLastError();
    }
  }
  route_kernel<VPT, false><<<blocks, kWarpsPerBlock * 32, 0, stream>>>(logits, bias, T, E, k, scale, idx, w);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_route(const float* logits, const float* bias, int T, int E, int k, float scale, int32_t* idx,
                         float* w, cudaStream_t stream, int* n_launches) {
  if (T <= 0) return cudaSuccess;
  const int per_lane = (E + 31) / 32;
  const bool vec = (E % 128 == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15u) == 0) &&
                   (bias == nullptr || (reinterpret_cast<uintptr_t>(bias) & 15u) == 0);
  cudaError_t err;
  if (per_lane <= 1) err = launch_vpt<1>(false, logits, bias, T, E, k, scale, idx, w, stream);
  else if (per_lane <= 2) err = launch_vpt<2>(false, logits, bias, T, E, k, scale, idx, w, stream);
  else if (per_lane <= 4) err = launch_vpt<4>(vec, logits, bias, T, E, k, scale, idx, w, stream);
  else if (per_lane <= 8) err = launch_vpt<8>(vec, logits, bias, T, E, k, scale, idx, w, stream);
  else if (per_lane <= 16) err = launch_vpt<16>(vec, logits, bias, T, E, k, scale, idx, w, stream);
  else err = launch_vpt<32>(vec, logits, bias, T, E, k, scale, idx, w, stream);
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

}  // namespace moe
