// Stage a5 (routed row movement) and stage a9 (weighted combine).  Both are pure HBM streaming, so both move
// rows with bulk asynchronous copies (cp.async.bulk) through shared-memory slots: a copy of several KB is one
// instruction, completion is tracked by mbarriers (loads) and bulk groups (stores), and many tens of KB per SM
// stay in flight without costing registers or issue slots.
//   permute  one warp per CTA walks (token, row chunk) items: the chunk is loaded once into a slot and stored
//            from there to its k destination rows.
//   combine  a producer warp gathers the k (+ shared) row chunks of an item into a slot, four consumer warps
//            sum them in fp32 in ascending expert order, round once to bf16 and store.  Deterministic.
// Every mbarrier wait is bounded; on expiry the kernel records a timeout in the status word and stops.
#include <cuda_bf16.h>

#include <map>
#include <mutex>
#include <tuple>

#include "kernels.h"

namespace moe {
namespace {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s: far beyond any legitimate wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait: gives up after limit_ns of wall time (global timer, read every 256 polls).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (uint32_t i = 0;; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (i >= 256u) {
      if ((i & 255u) == 0u) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (t0 == 0) t0 = now;
        else if (now - t0 > limit_ns) return false;
      }
      __nanosleep(64);
    }
  }
}
// global -> shared, `bytes` a multiple of 16, both addresses 16-byte aligned; completes on the mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// shared -> global, tracked by the issuing thread's bulk groups
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void flag_timeout(int* status) {
  if (status != nullptr) atomicCAS(status, kStOk, kStTimeout);
}
// After a wait has run out: copies this CTA issued may still be landing in its shared memory, so give them
// time before the CTA exits and the memory is handed to the next one.
__device__ __forceinline__ void linger_after_timeout() {
  for (int i = 0; i < 64; ++i) __nanosleep(1000);
}

// ------------------------------------------------------------------------------------------- a5 permute
constexpr int kPermuteSlots = 4;
constexpr int kPermuteChunkCols = 4096;  // bf16 columns per item: at most 8 KB per slot

// x_perm[inv_perm[t*k+j], c0:c1] = x[t, c0:c1] for j < k.  One warp per CTA; lane j stores destination j.
// Optionally one fp32 value per row travels with it: row_val_perm[inv_perm[t*k+j]] = row_val[t].
// dynamic shared memory: kPermuteSlots slots of slot_bytes | full[kPermuteSlots]
__global__ void __launch_bounds__(32)
permute_rows_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ inv_perm,
                    __nv_bfloat16* __restrict__ x_perm, int T, int k, int H, int col_blocks, int slot_bytes,
                    const float* __restrict__ row_val, float* __restrict__ row_val_perm, int* status,
                    unsigned long long wait_limit_ns) {
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t slots = smem_u32(smem);
  const uint32_t bar_full = slots + (uint32_t)(kPermuteSlots * slot_bytes);
  const int lane = threadIdx.x;
  const long long n_items = (long long)T * col_blocks;
  if (lane == 0) {
    for (int s = 0; s < kPermuteSlots; ++s) mbar_init(bar_full + 8u * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();
  pdl_wait();  // the barriers are set up; nothing of the previous kernel's results has been touched yet
  pdl_launch_dependents();

  auto item_of = [&](long long n) { return (long long)blockIdx.x + n * gridDim.x; };
  auto issue_load = [&](long long n) {  // lane 0 only
    const long long it = item_of(n);
    if (it >= n_items) return;
    const int t = (int)(it / col_blocks), c0 = (int)(it % col_blocks) * kPermuteChunkCols;
    const uint32_t bytes = (uint32_t)(min(kPermuteChunkCols, H - c0) * 2);
    const uint32_t s = (uint32_t)(n % kPermuteSlots);
    mbar_expect_tx(bar_full + 8u * s, bytes);
    bulk_load(slots + s * (uint32_t)slot_bytes, x + (size_t)t * H + c0, bytes, bar_full + 8u * s);
  };

  if (lane == 0)
    for (int n = 0; n < kPermuteSlots; ++n) issue_load(n);
  bool ok = true;
  for (long long n = 0; item_of(n) < n_items; ++n) {
    const long long it = item_of(n);
    const int t = (int)(it / col_blocks), c0 = (int)(it % col_blocks) * kPermuteChunkCols;
    const uint32_t bytes = (uint32_t)(min(kPermuteChunkCols, H - c0) * 2);
    const uint32_t s = (uint32_t)(n % kPermuteSlots), ph = (uint32_t)((n / kPermuteSlots) & 1);
    int dst_row = -1;
    if (lane < k) dst_row = __ldg(inv_perm + (size_t)t * k + lane);  // in flight while the row chunk arrives
    ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8u * s, ph, wait_limit_ns));
    if (!ok) break;
    if (dst_row >= 0) bulk_store(x_perm + (size_t)dst_row * H + c0, slots + s * (uint32_t)slot_bytes, bytes);
    bulk_commit();
    if (row_val != nullptr && c0 == 0 && dst_row >= 0) row_val_perm[dst_row] = __ldg(row_val + t);
    // the slot used one item ago may be refilled once every lane's stores from it have read shared memory
    bulk_wait_read<1>();
    __syncwarp();
    if (lane == 0 && n >= 1) issue_load(n - 1 + kPermuteSlots);
  }
  bulk_wait_read<0>();
  if (!ok) {
    if (lane == 0) flag_timeout(status);
    linger_after_timeout();
  }
}

// ------------------------------------------------------------------------------------------- a9 combine
constexpr int kCombineChunkCols = 1024;  // bf16 columns per item: 2 KB per gathered row chunk
constexpr int kCombineConsumers = 128;   // one 16-byte vector (8 columns) per consumer thread
constexpr int kCombineThreads = kCombineConsumers + 32;
constexpr int kCombineMaxStages = 4;

// acc += w * v for eight bf16 values; a bf16 widens to fp32 by a 16-bit shift (low half) or a mask (high half)
__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], const uint4& v, float w) {
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    acc[2 * q] = fmaf(w, __uint_as_float(u[q] << 16), acc[2 * q]);
    acc[2 * q + 1] = fmaf(w, __uint_as_float(u[q] & 0xffff0000u), acc[2 * q + 1]);
  }
}

// out[t, c0:c1] = sum_j w[t,j] * y_perm[inv_perm[t*k+j], c0:c1] (+ y_shared[t, c0:c1]); ascending j, then shared.
// dynamic shared memory, per stage: (k+1) row chunks of chunk_bytes | k weights | valid mask; then barriers.
// Producer lane j gathers row j; lane 0 also fetches the shared row.  KT > 0 fixes k at compile time (the sum
// over experts is then fully unrolled); KT = 0 takes k at run time.
template <int KT>
__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const __nv_bfloat16* __restrict__ y_perm, const __nv_bfloat16* __restrict__ y_shared,
               const int32_t* __restrict__ inv_perm, const float* __restrict__ topk_w, __nv_bfloat16* __restrict__ out,
               int T, int k, int H, int col_blocks, int chunk_bytes, int stage_bytes, int n_stages, int* status,
               unsigned long long wait_limit_ns) {
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t base = smem_u32(smem);
  const uint32_t bar_full = base + (uint32_t)(n_stages * stage_bytes);
  const uint32_t bar_empty = bar_full + 8u * n_stages;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int meta_off = (k + 1) * chunk_bytes;  // weights (k floats), then the valid mask
  const long long n_items = (long long)T * col_blocks;
  const bool shared = y_shared != nullptr;
  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, kCombineConsumers / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  pdl_wait();
  pdl_launch_dependents();

  if (warp == kCombineConsumers / 32) {
    // ============================================================ producer warp: lane j gathers row j
    bool ok = true;
    long long n = 0;
    for (long long it = blockIdx.x; it < n_items; it += gridDim.x, ++n) {
      const int t = (int)(it / col_blocks), c0 = (int)(it % col_blocks) * kCombineChunkCols;
      const uint32_t bytes = (uint32_t)(min(kCombineChunkCols, H - c0) * 2);
      const uint32_t s = (uint32_t)(n % n_stages), ph = (uint32_t)((n / n_stages) & 1);
      int row = -1;
      float wv = 0.f;
      if (lane < k) {
        row = __ldg(inv_perm + (size_t)t * k + lane);
        wv = __ldg(topk_w + (size_t)t * k + lane);
      }
      ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8u * s, ph ^ 1u, wait_limit_ns));
      if (!ok) break;
      uint8_t* st = smem + (size_t)s * stage_bytes;
      const unsigned valid = __ballot_sync(0xffffffffu, row >= 0);
      if (lane < k) reinterpret_cast<float*>(st + meta_off)[lane] = wv;
      if (lane == 0) *reinterpret_cast<unsigned*>(st + meta_off + 4 * k) = valid;
      __syncwarp();
      const uint32_t full = bar_full + 8u * s;
      if (lane == 0) mbar_expect_tx(full, (uint32_t)(__popc(valid) + (shared ? 1 : 0)) * bytes);
      __syncwarp();
      const uint32_t dst = base + s * (uint32_t)stage_bytes;
      if (row >= 0) bulk_load(dst + (uint32_t)(lane * chunk_bytes), y_perm + (size_t)row * H + c0, bytes, full);
      if (shared && lane == 0) bulk_load(dst + (uint32_t)(k * chunk_bytes), y_shared + (size_t)t * H + c0, bytes, full);
    }
    if (!ok) {
      if (lane == 0) flag_timeout(status);
      linger_after_timeout();
    }
  } else {
    // ============================================================ consumer warps: one 16-byte vector each
    bool ok = true;
    long long n = 0;
    const int v = threadIdx.x;
    for (long long it = blockIdx.x; it < n_items; it += gridDim.x, ++n) {
      const int t = (int)(it / col_blocks), c0 = (int)(it % col_blocks) * kCombineChunkCols;
      const int cols = min(kCombineChunkCols, H - c0);
      const uint32_t s = (uint32_t)(n % n_stages), ph = (uint32_t)((n / n_stages) & 1);
      ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8u * s, ph, wait_limit_ns));
      if (!ok) break;
      const uint8_t* st = smem + (size_t)s * stage_bytes;
      const float* wts = reinterpret_cast<const float*>(st + meta_off);
      const unsigned valid = *reinterpret_cast<const unsigned*>(st + meta_off + 4 * k);
      if (v * 8 < cols) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const uint8_t* mine = st + v * 16;
        if (KT > 0 && valid == (1u << KT) - 1u) {  // the usual case: every slot routed, k known at compile time
#pragma unroll
          for (int j = 0; j < KT; ++j)
            fma_bf16x8(acc, *reinterpret_cast<const uint4*>(mine + (size_t)j * chunk_bytes), wts[j]);
        } else {
          for (int j = 0; j < k; ++j)
            if ((valid >> j) & 1u)
              fma_bf16x8(acc, *reinterpret_cast<const uint4*>(mine + (size_t)j * chunk_bytes), wts[j]);
        }
        if (shared) fma_bf16x8(acc, *reinterpret_cast<const uint4*>(mine + (size_t)k * chunk_bytes), 1.0f);
        uint4 o;
        __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int q = 0; q < 4; ++q) oh[q] = __floats2bfloat162_rn(acc[2 * q], acc[2 * q + 1]);
        *reinterpret_cast<uint4*>(out + (size_t)t * H + c0 + v * 8) = o;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8u * s);
    }
    if (!ok) {
      if (lane == 0) flag_timeout(status);
      linger_after_timeout();
    }
  }
}

// CTAs of `kern` that fit on the device at once (one resident wave for a persistent grid); looked up once per
// kernel, device and shared-memory size, so that steady-state launches make no driver call besides the launch.
int resident_ctas(const void* kern, int threads, size_t smem) {
  static std::mutex mu;
  static std::map<std::tuple<const void*, int, size_t>, int> known;
  int dev = 0;
  cudaGetDevice(&dev);
  std::lock_guard<std::mutex> lock(mu);
  int& v = known[std::make_tuple(kern, dev, smem)];
  if (v == 0) {
    int sms = 148, per_sm = 1;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem);
    v = sms * (per_sm > 0 ? per_sm : 1);
  }
  return v;
}

}  // namespace

cudaError_t launch_permute(const void* x, const int32_t* inv_perm, void* x_perm, int T, int k, int H, int* status,
                           cudaStream_t stream, int* n_launches, const float* row_val, float* row_val_perm,
                           unsigned long long wait_limit_ns) {
  if (T <= 0) return cudaSuccess;
  if (k > 32) return cudaErrorNotSupported;  // one storing lane per destination
  const int col_blocks = (H + kPermuteChunkCols - 1) / kPermuteChunkCols;
  const int slot_bytes = (H < kPermuteChunkCols ? H : kPermuteChunkCols) * 2;
  const size_t smem = (size_t)kPermuteSlots * slot_bytes + 8 * kPermuteSlots;
  cudaError_t err = ensure_dynamic_smem(permute_rows_kernel, smem);
  if (err != cudaSuccess) return err;
  const long long n_items = (long long)T * col_blocks;
  const long long cap = resident_ctas(reinterpret_cast<const void*>(permute_rows_kernel), 32, smem);
  const int grid = (int)(n_items < cap ? n_items : cap);
  err = launch_pdl(true, permute_rows_kernel, dim3(grid), dim3(32), smem, stream, static_cast<const __nv_bfloat16*>(x), inv_perm,
                   static_cast<__nv_bfloat16*>(x_perm), T, k, H, col_blocks, slot_bytes, row_val, row_val_perm, status,
                   wait_limit_ns ? wait_limit_ns : kWaitLimitNs);
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

cudaError_t launch_combine(const void* y_perm, const void* y_shared, const int32_t* inv_perm, const float* topk_w,
                           void* out, int T, int k, int H, int* status, cudaStream_t stream, int* n_launches,
                           unsigned long long wait_limit_ns) {
  if (T <= 0) return cudaSuccess;
  if (k > 32) return cudaErrorNotSupported;  // one gathering lane per row
  const int col_blocks = (H + kCombineChunkCols - 1) / kCombineChunkCols;
  const int chunk_bytes = (H < kCombineChunkCols ? H : kCombineChunkCols) * 2;
  const int stage_bytes = ((k + 1) * chunk_bytes + 4 * k + 4 + 127) / 128 * 128;
  int stages = (64 * 1024) / stage_bytes;  // about 64 KB of slots per CTA, three CTAs per SM
  if (stages > kCombineMaxStages) stages = kCombineMaxStages;
  if (stages < 2) stages = 2;
  const size_t smem = (size_t)stages * stage_bytes + 16 * stages;
  auto launch = [&](auto kern) -> cudaError_t {
    cudaError_t e = ensure_dynamic_smem(kern, smem);
    if (e != cudaSuccess) return e;
    const long long n_items = (long long)T * col_blocks;
    const long long cap = resident_ctas(reinterpret_cast<const void*>(kern), kCombineThreads, smem);
    const int grid = (int)(n_items < cap ? n_items : cap);
    return launch_pdl(true, kern, dim3(grid), dim3(kCombineThreads), smem, stream, static_cast<const __nv_bfloat16*>(y_perm),
                      static_cast<const __nv_bfloat16*>(y_shared), inv_perm, topk_w, static_cast<__nv_bfloat16*>(out), T, k,
                      H, col_blocks, chunk_bytes, stage_bytes, stages, status,
                      wait_limit_ns ? wait_limit_ns : kWaitLimitNs);
  };
  cudaError_t err = k == 8 ? launch(combine_kernel<8>) : k == 4 ? launch(combine_kernel<4>)
                  : k == 2 ? launch(combine_kernel<2>) : launch(combine_kernel<0>);
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

}  // namespace moe
