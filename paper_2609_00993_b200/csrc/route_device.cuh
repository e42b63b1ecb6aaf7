// Stage a1 for one token by one warp: shared by the routing kernel and by the decode path's fused
// routing + layout kernel.  (Included by route.cu and layout.cu.)
#pragma once
#include <cstdint>

namespace moe {

// Monotone map from a finite float to an unsigned integer (larger float <=> larger integer), so that the
// warp arg-max can use the integer redux instructions.  -0.0 has been folded into +0.0 before the call,
// which keeps the IEEE tie between the two zeros.
__device__ __forceinline__ unsigned ordered_bits(float v) {
  const unsigned u = __float_as_uint(v);
  return u ^ ((unsigned)((int)u >> 31) | 0x80000000u);  // negative: all bits flipped; else the sign bit set
}

// Routes one token: `row` = its E logits, `bias` = the selection bias or nullptr; writes the k selected experts (in
// selection order) and their weights.  s_cand (32 entries of 8 bytes) and s_sel (32 ints) are this warp's scratch in
// shared memory.  VPT: keys per lane (power of two >= ceil(E/32)).  VEC: lanes own runs of 4 consecutive experts
// (E a multiple of 128, 16-byte aligned rows).  All 32 lanes of the warp call it together.
template <int VPT, bool VEC>
__device__ __forceinline__ void route_one_token(const float* __restrict__ row, const float* __restrict__ bias, int E,
                                                int k, float scale, int32_t* __restrict__ idx_out,
                                                float* __restrict__ w_out, unsigned long long* s_cand, int* s_sel,
                                                int lane) {
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
    if (c && pos < 32) s_cand[pos] = ((unsigned long long)key[i] << 32) | (unsigned)(0x7fffffff - expert_of(i));
    n_cand += __popc(b);
  }
  if (n_cand <= 32) {
    // rank each candidate against all
    __syncwarp();
    if (lane < n_cand) {
      const unsigned long long pc = s_cand[lane];
      int rank = 0;
      for (int q = 0; q < n_cand; ++q) rank += s_cand[q] > pc ? 1 : 0;
      if (rank < k) s_sel[rank] = 0x7fffffff - (int)(unsigned)(pc & 0xffffffffull);
    }
    __syncwarp();
    if (lane < k) my_e = s_sel[lane];
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
    idx_out[lane] = my_e;
    w_out[lane] = scale * p / s;
  }
}

}  // namespace moe
