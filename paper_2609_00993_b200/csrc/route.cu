// Stage a1: top-k routing over given router logits.  One warp per token; each lane keeps
// ceil(E/32) selection keys in registers (128-bit loads when E is a multiple of 128) as order-preserving integer
// images.  Selection: k warp maxima over the lanes' own maxima give a threshold that at least k keys reach; the few
// keys that reach it are compacted into a per-warp list and each is ranked exactly against the others (key
// descending, expert index ascending).  Only when ties put more than 32 keys at the threshold do k rounds of a
// warp arg-max over all keys run instead (redux.sync: a max over the key images, then a min over the expert
// indices that hold it).  The routed weights are a max-subtracted softmax over the k selected
// unbiased logits, summed in selection order.
#include "kernels.h"

namespace moe {
namespace {

constexpr int kWarpsPerBlock = 8;

// Monotone map from a finite float to an unsigned integer (larger float <=> larger integer), so that the
// warp arg-max can use the integer redux instructions.  -0.0 has been folded into +0.0 before the call,
// which keeps the IEEE tie between the two zeros.
__device__ __forceinline__ unsigned ordered_bits(float v) {
  const unsigned u = __float_as_uint(v);
  return u ^ ((unsigned)((int)u >> 31) | 0x80000000u);  // negative: all bits flipped; else the sign bit set
}

// VPT: keys per lane (power of two >= ceil(E/32)).  VEC: lanes own runs of 4 consecutive experts.
template <int VPT, bool VEC>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
route_kernel(const float* __restrict__ logits, const float* __restrict__ bias, int T, int E, int k, float scale,
             int32_t* __restrict__ idx, float* __restrict__ w) {
  pdl_wait();
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (t >= T) return;
  const float* row = logits + (size_t)t * E;

  // expert owned by this lane's i-th register; increasing in i so that "first wins" keeps the lower index
  auto expert_of = [&](int i) -> int { return VEC ? 128 * (i >> 2) + 4 * lane + (i & 3) : 32 * i + lane; };

  unsigned key[VPT];  // ordered_bits(logit + bias)
  if constexpr (VEC) {
#pragma unroll
    for (int q = 0; q < VPT / 4; ++q) {
      const int e0 = 128 * q + 4 * lane;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (e0 < E) {
        v = *reinterpret_cast<const float4*>(row + e0);
        if (bias != nullptr) {
          const float4 b = *reinterpret_cast<const float4*>(bias + e0);
          v.x = __fadd_rn(v.x, b.x); v.y = __fadd_rn(v.y, b.y); v.z = __fadd_rn(v.z, b.z); v.w = __fadd_rn(v.w, b.w);
        }
      }
      key[4 * q + 0] = ordered_bits(v.x + 0.0f); key[4 * q + 1] = ordered_bits(v.y + 0.0f);
      key[4 * q + 2] = ordered_bits(v.z + 0.0f); key[4 * q + 3] = ordered_bits(v.w + 0.0f);
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
      key[i] = ordered_bits(v + 0.0f);
    }
  }

  // ---- selection.  Fast path: the k-th largest of the 32 lane maxima is a threshold that at least k keys reach
  // (the maxima of k different lanes); the keys that reach it -- typically k to 2k of them -- are the only
  // candidates, and each is ranked exactly against the others (key descending, expert index ascending).  When
  // ties put more than 32 keys at or above the threshold the k-round warp arg-max below takes over.
  int my_e = 0;  // lane j (< k) ends up holding the j-th selected expert
  __shared__ unsigned long long s_cand[kWarpsPerBlock][32];
  __shared__ int s_sel[kWarpsPerBlock][32];
  const int wib = threadIdx.x >> 5;
  unsigned lmax = 0u;  // 0 is below the image of every float
#pragma unroll
  for (int i = 0; i < VPT; ++i)
    if (expert_of(i) < E) lmax = max(lmax, key[i]);
  unsigned tau = 0u, cur = lmax;
  for (int j = 0; j < k; ++j) {
    tau = __reduce_max_sync(0xffffffffu, cur);
    const unsigned holders = __ballot_sync(0xffffffffu, cur == tau);
    if (lane == __ffs(holders) - 1) cur = 0u;  // remove one holder per round
  }
  // One pass compacts the candidates into the warp's list (any order) as (key image << 32 | ~expert index) -- a
  // larger entry comes earlier in (key descending, expert index ascending) -- and counts them; places beyond the
  // list's 32 are not written.
  unsigned lt_mask;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(lt_mask));
  int n_cand = 0;
#pragma unroll
  for (int i = 0; i < VPT; ++i) {
    const bool c = expert_of(i) < E && key[i] >= tau;
    const unsigned b = __ballot_sync(0xffffffffu, c);
    const int pos = n_cand + __popc(b & lt_mask);
    if (c && pos < 32) s_cand[wib][pos] = ((unsigned long long)key[i] << 32) | (unsigned)(0x7fffffff - expert_of(i));
    n_cand += __popc(b);
  }
  if (n_cand <= 32) {
    // rank each candidate against all
    __syncwarp();
    if (lane < n_cand) {
      const unsigned long long pc = s_cand[wib][lane];
      int rank = 0;
      for (int q = 0; q < n_cand; ++q) rank += s_cand[wib][q] > pc ? 1 : 0;
      if (rank < k) s_sel[wib][rank] = 0x7fffffff - (int)(unsigned)(pc & 0xffffffffull);
    }
    __syncwarp();
    if (lane < k) my_e = s_sel[wib][lane];
  } else {
    unsigned taken = 0u;  // bit i: this lane's i-th key is already selected
    for (int j = 0; j < k; ++j) {
      unsigned bv = 0u;
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
      // warp arg-max on (key descending, expert index ascending): largest key, then the lowest index holding it
      const unsigned top = __reduce_max_sync(0xffffffffu, has ? bv : 0u);
      const int win = (int)__reduce_min_sync(0xffffffffu, (unsigned)((has && bv == top) ? be : 0x7fffffff));
      const int owner = VEC ? ((win & 127) >> 2) : (win & 31);
      const int slot = VEC ? (4 * (win >> 7) + (win & 3)) : (win >> 5);
      if (lane == owner) taken |= (1u << slot);
      if (lane == j) my_e = win;
    }
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
      return launch_pdl(true, route_kernel<VPT, true>, dim3(blocks), dim3(kWarpsPerBlock * 32), 0, stream, logits, bias, T, E, k,
                        scale, idx, w);
    }
  }
  return launch_pdl(true, route_kernel<VPT, false>, dim3(blocks), dim3(kWarpsPerBlock * 32), 0, stream, logits, bias, T, E, k, scale,
                    idx, w);
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
