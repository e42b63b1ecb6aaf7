// Stages a6-a8, weight-streaming variant of the grouped expert GEMM (sm_100a): swap-AB on the 5th-generation
// tensor cores.  128 weight rows fill the MMA M dimension, the expert's tokens sit in N, and N follows the expert:
//
//   tile       (expert, token chunk, feature tile).  An expert's rows are cut into ceil(rows / 256) equal chunks
//              (rounded up to 16), so an expert of up to 256 rows is ONE tile per feature tile and its weights
//              enter an SM once; the MMA N is the chunk's row count rounded up to 16 (16..256).
//   operands   a k-block (64 K-elements = 128-byte rows, 128-byte swizzle) is two 128-row weight boxes (32 KB,
//              gated: gate rows + the matching up rows; one TMA copy through a 4-D map) and exactly N token rows
//              (one TMA copy through the map whose box has N rows: 16 maps, one per multiple of 16).  What bounds
//              this regime is the bytes an SM ingests, so nothing is fetched that is not multiplied.
//   ring       k-blocks live in a byte ring of 2 KB slots with FIFO allocation (a k-block takes 16 slots for its
//              weights and N/16 for its token rows, two pieces that need not be adjacent), so a tile of few
//              tokens keeps more k-blocks in flight than a tile of many; up to 8 k-blocks in flight, each with
//              a full/empty mbarrier pair.  Producer and MMA issuer derive the same slot positions from the
//              same tile sequence.
//   TMEM       512 columns = two halves.  A tile of N <= 128 takes one half (its two accumulators side by side)
//              and alternates halves, so its epilogue overlaps the next tile's MMAs; a tile of N > 128 takes both.
//   epilogue   lane = weight row (output feature), column = token: tcgen05.ld -> (scale) -> SwiGLU -> bf16;
//              neighbouring lanes exchange values so that every store writes a feature pair.  The gated epilogue
//              hands the accumulator back before its exchanges and stores.
//   schedule   the tile list is ordered by expert size, largest first.  Its first waves are dealt statically (CTAs
//              in step share weights and rows through L2), the last two waves' worth of tiles -- the smallest -- are
//              handed out by an atomic counter to whichever CTA is free; the producer publishes the tiles it takes
//              in a four-entry queue that the MMA issuer and the epilogue warps follow.
//   set-up     with the launch overlap, the tile list is built and weight boxes are requested before the kernel
//              waits for the previous kernel of the stream; only the token rows and the stores wait for it.
//
// Warp roles (320 threads): warps 0-7 epilogue (two per TMEM lane group), warp 8 TMA producer, warp 9 MMA issuer
// and TMEM owner.
// Every mbarrier wait is bounded: on expiry the kernel records a timeout in the status word, raises a CTA-wide
// abort flag, lets copies in flight land, frees its TMEM and returns.
// The same kernel serves E4M3 operands (kind::f8f6f4, 128 K-elements per k-block, accumulator scaled by the
// row's and the weight row's scale in the epilogue).
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>

#include "kernels.h"
#include "tc_common.cuh"

namespace moe {
namespace {

using namespace tc;

#ifndef MOE_STREAM_ISSUERS
#define MOE_STREAM_ISSUERS 1
#endif
#ifndef MOE_STREAM_EPI_WARPS
#define MOE_STREAM_EPI_WARPS 8
#endif
// MMA-issuing threads: one for both weight boxes (1) or one per box (2).  Two were measured and are no faster:
// what the issuer waits for is the tensor pipe, which in turn waits for shared-memory bandwidth.
constexpr int kIssuers = MOE_STREAM_ISSUERS;
// Epilogue warps: 4 (each owns 32 TMEM lanes = 32 weight rows) or 8 (two warps per lane group, one taking the
// even and one the odd 16-token chunks), which halves the time a tile of more than 128 tokens keeps the MMA
// issuer waiting for its single accumulator.
constexpr int kEpilogueWarps = MOE_STREAM_EPI_WARPS;
constexpr int kProducerWarp = kEpilogueWarps;
constexpr int kMmaWarp = kEpilogueWarps + 1;  // issuer of box 0 and TMEM owner; the next warp issues box 1 when kIssuers == 2
constexpr int kThreads = 32 * (kEpilogueWarps + 1 + kIssuers);
constexpr int kSortMaxExperts = 512;  // the tile list is ordered by expert size up to this many experts
constexpr int kSlotBytes = 2048;                        // ring granularity: 16 token rows of one k-block
constexpr int kWSlots = 2 * kWBoxBytes / kSlotBytes;    // 16 slots: the two weight boxes
constexpr int kMaxTileRows = 256;                       // largest MMA N
constexpr int kNB = 8;                                  // k-blocks in flight at most (barrier pairs)
constexpr int kXMaps = 16;                              // token-row boxes of 16 (b + 1) rows
constexpr uint32_t kTmemCols = 512;
constexpr int kQ = 4;                                   // entries of the CTA's tile queue
#ifndef MOE_STREAM_DYN_WAVES
#define MOE_STREAM_DYN_WAVES 2
#endif
constexpr int kDynWaves = MOE_STREAM_DYN_WAVES;         // waves' worth of tiles, at the list's end, handed out dynamically

struct StreamParams {
  const int32_t* offsets;  // [E+1] (already advanced to the first expert of the launch) or nullptr
  int32_t fixed_rows;
  int32_t E;               // experts covered by this launch
  int32_t e_base;          // index of the launch's first expert in the weight tensor
  int32_t n_feat;          // output features (I for the gated pass, H for the down pass)
  int32_t K;
  __nv_bfloat16* out;      // [rows, n_feat]
  int32_t ring_slots;
  int* status;
  int32_t inject_producer_stall;  // failure-detection test hook: the TMA producer issues nothing
  unsigned long long wait_limit_ns;
  // optional dense group (shared expert) computed by the same launch; rows2 == 0: none
  int32_t rows2;
  int32_t n_feat2;
  int32_t K2;
  __nv_bfloat16* out2;
  // FP8 variant: the accumulator is scaled by row_scale[row] * w_scale[weight row]
  const float* row_scale;
  const float* row_scale2;
  const float* w_scale;
  const float* w_scale2;
  // The launch's tile counter and the count of CTAs that have finished (two words in device memory, zero before the
  // first launch that uses them; the last CTA to finish puts them back to zero).
  int* tile_ctr;
  int* done_ctr;
  int32_t all_dynamic;  // every tile comes from the counter (a pass that may be launched again to go on)
  // preemption at tile granularity (both null: off)
  const int* yield_req;
  int* stopped;
  // The expert offsets were final before the PREVIOUS kernel of the stream started (and the weights always are):
  // the tile list is built and weight boxes are fetched before this kernel waits for that previous kernel, which
  // only the token rows (and the FP8 row scales) depend on.
  int32_t early_setup;
  int32_t sort_tiles;  // 0: every group has at most one tile of the smallest size, so their order does not matter
};

#ifdef MOE_STREAM_PROF
// Debug build only: per-CTA role timings of the last launches (8 words per CTA, accumulated).
__device__ unsigned long long g_stream_prof[8 * 256];
__device__ unsigned long long g_stream_ts[8 * 256];  // global-timer stamps of the last launch, 8 per CTA
#define PROF_T0() const long long prof_t0 = clock64()
#define PROF_ADD(var) var += clock64() - prof_t0
#define PROF_STAMP(slot) g_stream_ts[8 * blockIdx.x + (slot)] = global_ns()
#else
#define PROF_T0()
#define PROF_ADD(var)
#define PROF_STAMP(slot)
#endif

struct StreamMaps {
  CUtensorMap x[kXMaps], x2[kXMaps];  // token rows, boxes of 16, 32, ..., 256 rows (x2: the dense group's)
};

struct STile {
  int e, row0, rows, ft;
  bool dense;
};

// An expert's (or the dense group's) rows in ceil(cnt / 256) chunks of equal size, rounded up to 16.
__device__ __forceinline__ void chunking(int cnt, int& tiles, int& chunk) {
  tiles = (cnt + kMaxTileRows - 1) / kMaxTileRows;
  chunk = tiles > 0 ? (((cnt + tiles - 1) / tiles) + 15) & ~15 : 0;
}

// tile -> (expert, first row, valid rows, feature tile).  The dense group's tiles come first (chunk major),
// then the experts' in the order `order` (largest first): prefix[i] = chunks of the experts at positions < i.
__device__ __forceinline__ STile decode_tile(int tile, int dense_tiles, int n_ft2, int rows2, int n_ft, int E,
                                             const int* prefix, const int* order, const int* beg, const int* cnts) {
  STile t;
  int tiles, chunk;
  if (tile < dense_tiles) {
    const int rt = tile / n_ft2;
    chunking(rows2, tiles, chunk);
    t.e = 0;
    t.ft = tile - rt * n_ft2;
    t.row0 = rt * chunk;
    t.rows = min(chunk, rows2 - t.row0);
    t.dense = true;
    return t;
  }
  tile -= dense_tiles;
  const int rt = tile / n_ft;
  int lo = 0, hi = E;  // largest position in [0,E) with prefix[position] <= rt
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= rt) lo = mid; else hi = mid;
  }
  const int e = order[lo], cnt = cnts[e];
  chunking(cnt, tiles, chunk);
  const int mt = rt - prefix[lo];
  t.e = e;
  t.ft = tile - rt * n_ft;
  t.row0 = beg[e] + mt * chunk;
  t.rows = min(chunk, cnt - mt * chunk);
  t.dense = false;
  return t;
}

template <bool GATED, bool FP8>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_stream_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_w2,
                           const __grid_constant__ StreamMaps xmaps, const __grid_constant__ StreamParams p) {
  constexpr int kbk = FP8 ? 2 * kBlockK : kBlockK;  // K elements per k-block
  extern __shared__ uint8_t smem_raw[];
  // carve: ring (ring_slots x 2 KB) | full[kNB] empty[kNB] tfull[2] tempty[2] tqfull[kQ] tqempty[kQ] | tmem slot
  //        | abort | stopped | sizes[kNB] | tq[kQ] | prefix[E+1] | order[E] | beg[E] | cnts[E]
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
  uint8_t* base = smem_raw + (base_addr - raw_addr);
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)p.ring_slots * kSlotBytes);
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8u * kNB;
  const uint32_t bar_tfull = bar_empty + 8u * kNB;
  const uint32_t bar_tempty = bar_tfull + 16u;
  const uint32_t bar_tqfull = bar_tempty + 16u;         // the tile queue: an entry has been published
  const uint32_t bar_tqempty = bar_tqfull + 8u * kQ;    // ... and read by the issuer and every epilogue warp
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kNB + 4 + 2 * kQ);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* stopped_here = reinterpret_cast<volatile int*>(tmem_slot + 2);  // the producer stopped on request
  int* sizes = reinterpret_cast<int*>(tmem_slot + 3);  // slots held by the k-blocks in flight (producer only)
  volatile int* tq = reinterpret_cast<volatile int*>(sizes + kNB);  // tile queue entries (-1: no more tiles)
  int* prefix = sizes + kNB + kQ;
  int* order = prefix + (p.E + 1);
  int* beg = order + p.E;
  int* cnts = beg + p.E;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  [[maybe_unused]] const int unit = (int)blockIdx.x;
  if (threadIdx.x == 0) PROF_STAMP(0);
  constexpr int kFeatPerTile = GATED ? 128 : 256;
  const int n_ft = (p.n_feat + kFeatPerTile - 1) / kFeatPerTile;
  const int num_kb1 = (p.K + kbk - 1) / kbk, num_kb2 = (p.K2 + kbk - 1) / kbk;
  const int n_ft2 = (p.n_feat2 + kFeatPerTile - 1) / kFeatPerTile;
  const int dense_tiles = p.rows2 > 0 ? ((p.rows2 + kMaxTileRows - 1) / kMaxTileRows) * n_ft2 : 0;
  const unsigned long long limit = p.wait_limit_ns;

  // ---- set-up: barriers and TMEM (before the previous kernel of the stream is known to be complete), then the
  // tile list (experts ordered by size, largest first)
  if (threadIdx.x == 32 * kProducerWarp) {
    for (int s = 0; s < kNB; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, kIssuers);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, kIssuers);
      mbar_init(bar_tempty + 8u * a, kEpilogueWarps);
    }
    for (int q = 0; q < kQ; ++q) {
      mbar_init(bar_tqfull + 8u * q, 1);
      mbar_init(bar_tqempty + 8u * q, kIssuers + kEpilogueWarps);
    }
    *abort_flag = 0;
    *stopped_here = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kMmaWarp) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  // With early set-up only the threads that touch what the previous kernel wrote wait for it: the producer before
  // its first token-row copy, the epilogue warps before their first store.  Dependents are released only by
  // threads that have waited, so a later kernel never starts before the kernel two places back has completed.
  if (!p.early_setup) {
    pdl_wait();
    pdl_launch_dependents();
  }
  if (threadIdx.x == 0) PROF_STAMP(1);
  for (int e = threadIdx.x; e < p.E; e += kThreads) {
    const int b = p.offsets ? p.offsets[e] : 0;
    int c = p.offsets ? p.offsets[e + 1] - b : p.fixed_rows;
    if (c < 0) c = 0;
    beg[e] = b;
    cnts[e] = c;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < p.E; e += kThreads) {
    int rank = e;  // more than kSortMaxExperts experts: the natural order
    if (p.sort_tiles && p.E <= kSortMaxExperts) {
      const int c = cnts[e];
      rank = 0;
      for (int j = 0; j < p.E; ++j) {
        const int cj = cnts[j];
        rank += (cj > c || (cj == c && j < e)) ? 1 : 0;
      }
    }
    order[rank] = e;
  }
  __syncthreads();
  if (warp == 0) {
    int carry = 0;
    for (int b = 0; b < p.E; b += 32) {
      const int i = b + lane;
      const int cnt = i < p.E ? cnts[order[i]] : 0;
      const int tiles = (cnt + kMaxTileRows - 1) / kMaxTileRows;
      int incl = tiles;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += n;
      }
      if (i < p.E) prefix[i] = carry + incl - tiles;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) prefix[p.E] = carry;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) PROF_STAMP(2);
  const int total_tiles = dense_tiles + prefix[p.E] * n_ft;
  const uint32_t R = (uint32_t)p.ring_slots;

  if (warp == kProducerWarp) {
    // ================================================================= TMA producer (one lane)
    if (lane == 0 && !p.inject_producer_stall) {
      uint32_t head = 0, free_slots = R, kb_idx = 0, oldest = 0;
      bool ok = true;
      // Early set-up: until this thread has waited for the previous kernel, token-row copies are put off (their
      // ring space is allocated and their bytes announced) while the weight boxes of up to kNB k-blocks go out.
      bool dep_waited = !p.early_setup;
      int n_def = 0;
      uint32_t def_dst[kNB], def_full[kNB];
      int def_k0[kNB], def_row0[kNB];
      const CUtensorMap* def_map[kNB];
      auto dep_wait_and_flush = [&]() {
        pdl_wait();
        pdl_launch_dependents();
        dep_waited = true;
        for (int i = 0; i < n_def; ++i) tma_load_2d(def_dst[i], def_map[i], def_full[i], def_k0[i], def_row0[i]);
        n_def = 0;
      };
      [[maybe_unused]] long long prof_wait_empty = 0, prof_tiles = 0;
      [[maybe_unused]] const long long prof_start = clock64();
      int yield_seen = 0;
      if (p.yield_req != nullptr)
        asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(yield_seen) : "l"(p.yield_req) : "memory");
      // Tiles are handed out by a counter in device memory, in the list's order (largest experts first): a CTA
      // that finishes early takes the next tile, whichever CTA would have had it.  The producer publishes every tile
      // it takes -- and finally -1 -- in a small queue that the issuer and the epilogue warps follow.
      uint32_t tcount = 0;
      auto publish = [&](int tile) -> bool {
        const uint32_t q = tcount % kQ, par = ((tcount / kQ) & 1u) ^ 1u;
        // the epilogue warps free an entry only after the tile before it, which needs its token rows: the copies
        // put off by the early set-up go out before this thread blocks
        if (!dep_waited && !mbar_try_wait(bar_tqempty + 8u * q, par)) dep_wait_and_flush();
        if (!mbar_wait(bar_tqempty + 8u * q, par, abort_flag, limit)) return false;
        tq[q] = tile;
        mbar_arrive(bar_tqfull + 8u * q);
        ++tcount;
        return true;
      };
      // The counter is read a few k-blocks before the current tile's last copy, so that the atomic's round trip hides
      // behind those copies -- and no earlier, so that a CTA does not hold a second tile while another CTA has none.
      // A stop on request therefore takes effect after the tile that had already been taken.
      // The first waves are dealt statically (wave w: tile w * grid + the CTA's index, alternately forwards and
      // backwards): CTAs that run in step start the tiles that share an expert's weights or rows together, and the
      // second reader finds them in L2.  The last kDynWaves waves' worth of tiles -- the smallest ones, the list being
      // ordered by size -- go to whichever CTA is free, which evens out what the static part left uneven.  A pass that
      // can be stopped on request is dynamic throughout: its next launch only needs the counter to go on.
      const int grid = (int)gridDim.x;
      // (At least the first wave is static, which also spares every CTA a contended atomic at the start.)
      const int w_static = p.all_dynamic ? 0 : max(1, total_tiles / grid - kDynWaves);
      int sw = 0;
      auto next_tile = [&]() -> int {
        if (sw < w_static) {
          const int w = sw++;
          return w * grid + ((w & 1) ? grid - 1 - (int)blockIdx.x : (int)blockIdx.x);
        }
        return w_static * grid + atomicAdd(p.tile_ctr, 1);
      };
      int taken = next_tile();
      for (;;) {
        const int tile = taken < total_tiles ? taken : -1;
        if (!publish(tile)) {
          ok = false;
          break;
        }
        if (tile < 0) break;
        bool stop_after = false;
        const STile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, order, beg, cnts);
        const uint32_t n = (uint32_t)((t.rows + 15) & ~15);
        const int w_row0 = t.ft * kFeatPerTile;
        const CUtensorMap* mw = t.dense ? &map_w2 : &map_w;
        const CUtensorMap* mx = (t.dense ? xmaps.x2 : xmaps.x) + ((n >> 4) - 1u);  // the box of exactly n rows
        const int w_e = t.dense ? 0 : p.e_base + t.e;
        const int num_kb = t.dense ? num_kb2 : num_kb1;
        const int fetch_kb = num_kb > 4 ? num_kb - 4 : 0;
        for (int kb = 0, k0 = 0; kb < num_kb && ok; ++kb, k0 += kbk) {
          if (kb == fetch_kb) {
            if (p.yield_req != nullptr) {
              // the request word was read a tile ago, so looking at it here does not stall the pipeline; the read for
              // the next tile goes out now
              stop_after = yield_seen != 0;
              asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(yield_seen) : "l"(p.yield_req) : "memory");
            }
            if (!stop_after) taken = next_tile();
          }
          // The ring is allocated per operand: the weight boxes and the token rows of a k-block are two contiguous
          // pieces that need not be adjacent, so the weights of the next k-block go out as soon as 16 slots are
          // free.  A piece never wraps: it skips what is left at the ring's end.
          const uint32_t nx = n >> 4;
          const bool wrap_w = head + (uint32_t)kWSlots > R;
          const uint32_t pad_w = wrap_w ? R - head : 0u;
          const uint32_t head_w = wrap_w ? 0u : head;
          const bool wrap_x = head_w + (uint32_t)kWSlots + nx > R;
          const uint32_t pad_x = wrap_x ? R - (head_w + (uint32_t)kWSlots) : 0u;
          const uint32_t head_x = wrap_x ? 0u : head_w + (uint32_t)kWSlots;
          auto reclaim = [&](uint32_t need, bool count_limit) {
            // nothing is consumed before the token rows are in: wait for the previous kernel before blocking
            if (!dep_waited && (free_slots < need || (count_limit && kb_idx - oldest >= (uint32_t)kNB)))
              dep_wait_and_flush();
            while (free_slots < need || (count_limit && kb_idx - oldest >= (uint32_t)kNB)) {
              PROF_T0();
              const bool got = mbar_wait(bar_empty + 8u * (oldest % kNB), (oldest / kNB) & 1u, abort_flag, limit);
              PROF_ADD(prof_wait_empty);
              if (!got) return false;
              free_slots += (uint32_t)sizes[oldest % kNB];
              ++oldest;
            }
            return true;
          };
          if (!reclaim((uint32_t)kWSlots + pad_w, true)) { ok = false; break; }
          free_slots -= (uint32_t)kWSlots + pad_w;
          const uint32_t full = bar_full + 8u * (kb_idx % kNB);
          mbar_expect_tx(full, 2u * kWBoxBytes + n * 128u);
          // one copy per operand: both weight boxes (gated: the map's third dimension steps from the gate rows
          // to the up rows; down pass: 256 consecutive rows), then the n token rows
          const uint32_t st_w = base_addr + head_w * (uint32_t)kSlotBytes;
          if (GATED) tma_load_4d(st_w, mw, full, k0, w_row0, 0, w_e);
          else tma_load_3d(st_w, mw, full, k0, w_row0, w_e);
          if (!reclaim(nx + pad_x, false)) { ok = false; break; }
          free_slots -= nx + pad_x;
          sizes[kb_idx % kNB] = (int)((uint32_t)kWSlots + pad_w + nx + pad_x);
          if (dep_waited) {
            tma_load_2d(base_addr + head_x * (uint32_t)kSlotBytes, mx, full, k0, t.row0);
          } else {
            def_dst[n_def] = base_addr + head_x * (uint32_t)kSlotBytes;
            def_full[n_def] = full;
            def_map[n_def] = mx;
            def_k0[n_def] = k0;
            def_row0[n_def] = t.row0;
            ++n_def;
          }
          head = head_x + nx;
          ++kb_idx;
        }
        if (stop_after && ok) {
          *stopped_here = 1;  // no further tile is taken: the other roles finish the published ones and leave
          if (!publish(-1)) ok = false;
          break;
        }
      }
      if (!dep_waited) dep_wait_and_flush();
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(p.status, kStOk, kStTimeout);
      }
#ifdef MOE_STREAM_PROF
      atomicAdd(&g_stream_prof[8 * unit + 0], (unsigned long long)(clock64() - prof_start));
      atomicAdd(&g_stream_prof[8 * unit + 1], (unsigned long long)prof_wait_empty);
#endif
    }
  } else if (warp >= kMmaWarp) {
    // ================================================================= MMA issuer(s) (one lane each)
    // With two issuers, warp 5 multiplies weight box 0 into accumulator a and warp 6 box 1 into accumulator b;
    // both wait on the same barriers, and every barrier they signal counts one arrival from each.
    const bool do_a = kIssuers == 1 || warp == kMmaWarp, do_b = kIssuers == 1 || warp != kMmaWarp;
    if (lane == 0) {
      uint32_t head = 0, kb_idx = 0, use0 = 0, use1 = 0, next_half = 0;
      bool ok = true;
      [[maybe_unused]] long long prof_wait_full = 0, prof_wait_acc = 0, prof_tiles = 0;
      [[maybe_unused]] const long long prof_start = clock64();
      const uint32_t desc_hi = (uint32_t)(umma_smem_desc(0) >> 32);
      const uint32_t lo_base = (uint32_t)umma_smem_desc(base_addr);  // slot 0
      constexpr uint32_t lo_slot = (uint32_t)kSlotBytes >> 4, lo_box = (uint32_t)kWBoxBytes >> 4;
      uint32_t tcount = 0;
      for (;;) {
        const uint32_t q = tcount % kQ;
        if (!mbar_wait(bar_tqfull + 8u * q, (tcount / kQ) & 1u, abort_flag, limit)) {
          ok = false;
          break;
        }
        const int tile = tq[q];
        mbar_arrive(bar_tqempty + 8u * q);
        ++tcount;
        if (tile < 0) break;
        const STile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, order, beg, cnts);
        const uint32_t n = (uint32_t)((t.rows + 15) & ~15);
        const bool big = n > 128u;
        uint32_t d_a, d_b;
        PROF_T0();
        if (big) {
          if (!mbar_wait(bar_tempty, (use0 & 1u) ^ 1u, abort_flag, limit) ||
              !mbar_wait(bar_tempty + 8u, (use1 & 1u) ^ 1u, abort_flag, limit)) { ok = false; break; }
          d_a = tmem_base;
          d_b = tmem_base + 256u;
        } else {
          const uint32_t h = next_half;
          next_half ^= 1u;
          if (!mbar_wait(bar_tempty + 8u * h, ((h ? use1 : use0) & 1u) ^ 1u, abort_flag, limit)) { ok = false; break; }
          d_a = tmem_base + 256u * h;
          d_b = d_a + 128u;
          if (h) ++use1; else ++use0;
        }
        PROF_ADD(prof_wait_acc);
#ifdef MOE_STREAM_PROF
        ++prof_tiles;
#endif
        tc_fence_after();
        const uint32_t idesc = FP8 ? umma_idesc_e4m3(128, n) : umma_idesc(128, n);
        const int num_kb = t.dense ? num_kb2 : num_kb1;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (head + (uint32_t)kWSlots > R) head = 0;  // the producer's allocation, step for step
          const uint32_t pos_w = head;
          head += (uint32_t)kWSlots;
          if (head + (n >> 4) > R) head = 0;
          const uint32_t pos_x = head;
          head += n >> 4;
          {
            PROF_T0();
            const bool got = mbar_wait(bar_full + 8u * (kb_idx % kNB), (kb_idx / kNB) & 1u, abort_flag, limit);
            PROF_ADD(prof_wait_full);
            if (!got) { ok = false; break; }
          }
          if (kb_idx == 0) PROF_STAMP(3);
          tc_fence_after();
          const uint32_t lo_w0 = lo_base + pos_w * lo_slot, lo_w1 = lo_w0 + lo_box, lo_x = lo_base + pos_x * lo_slot;
#pragma unroll
          for (int kk = 0; kk < kBlockK / kUmmaK; ++kk) {
            const uint32_t adv = (uint32_t)((kk * kUmmaK * 2) >> 4);  // +32 bytes per MMA, in 16-byte units
            const uint32_t acc = (kb | kk) != 0 ? 1u : 0u;
            if (FP8) {
              if (do_a) umma_e4m3_lo(d_a, lo_w0 + adv, lo_x + adv, desc_hi, idesc, acc);
              if (do_b) umma_e4m3_lo(d_b, lo_w1 + adv, lo_x + adv, desc_hi, idesc, acc);
            } else {
              if (do_a) umma_bf16_lo(d_a, lo_w0 + adv, lo_x + adv, desc_hi, idesc, acc);
              if (do_b) umma_bf16_lo(d_b, lo_w1 + adv, lo_x + adv, desc_hi, idesc, acc);
            }
          }
          umma_commit(bar_empty + 8u * (kb_idx % kNB));  // the k-block's slots are free once these MMAs have read them
          ++kb_idx;
        }
        if (!ok) break;
        if (big) {
          umma_commit(bar_tfull);
          umma_commit(bar_tfull + 8u);
          ++use0;
          ++use1;
        } else {
          umma_commit(bar_tfull + 8u * (next_half ^ 1u));
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(p.status, kStOk, kStTimeout);
      }
      PROF_STAMP(4);
#ifdef MOE_STREAM_PROF
      if (warp == kMmaWarp)
      atomicAdd(&g_stream_prof[8 * unit + 2], (unsigned long long)(clock64() - prof_start));
      if (warp == kMmaWarp) {
      atomicAdd(&g_stream_prof[8 * unit + 3], (unsigned long long)prof_wait_full);
      atomicAdd(&g_stream_prof[8 * unit + 4], (unsigned long long)prof_wait_acc);
      atomicAdd(&g_stream_prof[8 * unit + 5], (unsigned long long)prof_tiles);
      atomicAdd(&g_stream_prof[8 * unit + 6], (unsigned long long)kb_idx);
      }
#endif
    }
  } else {
    // ================================================================= epilogue (warps 0-7)
    // lane = weight row (output feature) of each box, TMEM column = token
    if (p.early_setup) {
      pdl_wait();
      pdl_launch_dependents();
    }
    uint32_t use0 = 0, use1 = 0, next_half = 0;
    bool ok = true;
    const int lg = warp & 3;                         // TMEM lane group of this warp: lanes 32 lg .. 32 lg + 31
    const int c_first = kEpilogueWarps == 8 ? 16 * (warp >> 2) : 0, c_step = kEpilogueWarps == 8 ? 32 : 16;
    const uint32_t lane_base = ((uint32_t)(lg * 32)) << 16;
    const int fl = lg * 32 + lane;
    const bool even = (lane & 1) == 0;
    uint32_t tcount = 0;
    for (;;) {
      const uint32_t q = tcount % kQ;
      if (!mbar_wait(bar_tqfull + 8u * q, (tcount / kQ) & 1u, abort_flag, limit)) {
        ok = false;
        break;
      }
      const int tile = tq[q];
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tqempty + 8u * q);
      ++tcount;
      if (tile < 0) break;
      const STile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, order, beg, cnts);
      const uint32_t n = (uint32_t)((t.rows + 15) & ~15);
      const bool big = n > 128u;
      uint32_t h = 0, d_a, d_b;
      if (big) {
        if (!mbar_wait(bar_tfull, use0 & 1u, abort_flag, limit) ||
            !mbar_wait(bar_tfull + 8u, use1 & 1u, abort_flag, limit)) { ok = false; break; }
        ++use0;
        ++use1;
        d_a = tmem_base;
        d_b = tmem_base + 256u;
      } else {
        h = next_half;
        next_half ^= 1u;
        if (!mbar_wait(bar_tfull + 8u * h, (h ? use1 : use0) & 1u, abort_flag, limit)) { ok = false; break; }
        if (h) ++use1; else ++use0;
        d_a = tmem_base + 256u * h;
        d_b = d_a + 128u;
      }
      tc_fence_after();
      d_a += lane_base;
      d_b += lane_base;
      __nv_bfloat16* const out = t.dense ? p.out2 : p.out;
      const int n_feat = t.dense ? p.n_feat2 : p.n_feat;
      const int f_a = t.ft * kFeatPerTile + fl;  // box 0 feature
      const int f_b = f_a + kWBoxRows;           // box 1 feature (down pass only)
      float ws_a = 1.f, ws_b = 1.f;              // FP8: scales of this lane's two weight rows
      const float* rsp = nullptr;
      if (FP8) {
        rsp = (t.dense ? p.row_scale2 : p.row_scale) + t.row0;
        const float* const wsp =
            t.dense ? p.w_scale2 : p.w_scale + (size_t)(p.e_base + t.e) * (GATED ? 2 : 1) * n_feat;
        if (f_a < n_feat) ws_a = wsp[f_a];
        if (GATED ? f_a < n_feat : f_b < n_feat) ws_b = wsp[GATED ? n_feat + f_a : f_b];
      }
      // Feature pairs: an even lane keeps the even tokens of a 16-token chunk and receives its odd neighbour's
      // values for them (features f, f+1 of one token are one 4-byte store); the odd lane does the same for
      // the odd tokens.  n_feat is a multiple of 8, so a pair is inside the row or outside it as a whole.
      const int f_pair = (GATED ? f_a : 0) & ~1;
      auto release_acc = [&]() {  // hand the accumulator half (or both) back to the MMA issuer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (big) {
            mbar_arrive(bar_tempty);
            mbar_arrive(bar_tempty + 8u);
          } else {
            mbar_arrive(bar_tempty + 8u * h);
          }
        }
      };
      if (GATED && kEpilogueWarps == 8) {
        // Two phases, so that the accumulator goes back to the MMA issuer as early as possible (a tile of more than
        // 128 tokens holds all of TMEM, and the issuer waits for it): first every chunk is loaded (the next chunk's
        // loads in flight meanwhile), put through SwiGLU and packed to bf16 in registers -- a warp has at most 8
        // chunks of 16 tokens; then the accumulator is released; only then come the lane exchanges and the stores.
        uint32_t pk[8][8];  // pk[m][i]: this lane's feature for tokens c + 2i (low half) and c + 2i + 1 (high half)
        uint32_t na[16], nb[16];
        if (c_first < t.rows) {
          tmem_ld16(d_a + (uint32_t)c_first, na);
          tmem_ld16(d_b + (uint32_t)c_first, nb);
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          const int c = c_first + m * c_step;
          if (c < t.rows) {
            float g[16], u[16];
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              g[i] = __uint_as_float(na[i]);
              u[i] = __uint_as_float(nb[i]);
            }
            if (c + c_step < t.rows) {
              tmem_ld16(d_a + (uint32_t)(c + c_step), na);
              tmem_ld16(d_b + (uint32_t)(c + c_step), nb);
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              if (FP8) {
                const float rs = (c + i < t.rows) ? __ldg(rsp + c + i) : 0.f;
                g[i] *= rs * ws_a;
                u[i] *= rs * ws_b;
              }
              g[i] = silu_mul(g[i], u[i]);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) pk[m][i] = pack_bf16(g[2 * i], g[2 * i + 1]);
          }
        }
        release_acc();
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          const int c = c_first + m * c_step;
          if (c < t.rows) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t mine = pk[m][i];
              const uint32_t nbr = __shfl_xor_sync(0xffffffffu, mine, 1);
              // even lane (even feature f): token c+2i, features (f, f+1) = (own low, neighbour's low);
              // odd lane: token c+2i+1, features (f-1, f) = (neighbour's high, own high)
              const uint32_t pa = even ? __byte_perm(mine, nbr, 0x5410) : __byte_perm(nbr, mine, 0x7632);
              const int tok = c + 2 * i + (even ? 0 : 1);
              if (tok < t.rows && f_pair < n_feat)
                *reinterpret_cast<uint32_t*>(out + (size_t)(t.row0 + tok) * n_feat + f_pair) = pa;
            }
          }
        }
        continue;
      }
      // the loads of the next 16-token chunk are in flight while this one is converted and stored
      uint32_t na[16], nb[16];
      if (c_first < t.rows) {
        tmem_ld16(d_a + (uint32_t)c_first, na);
        tmem_ld16(d_b + (uint32_t)c_first, nb);
      }
      for (int c = c_first; c < t.rows; c += c_step) {
        uint32_t ra[16], rb[16];
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          ra[i] = na[i];
          rb[i] = nb[i];
        }
        if (c + c_step < t.rows) {
          tmem_ld16(d_a + (uint32_t)(c + c_step), na);
          tmem_ld16(d_b + (uint32_t)(c + c_step), nb);
        }
        float va[16], vb[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float a = __uint_as_float(ra[i]), b = __uint_as_float(rb[i]);
          if (FP8) {
            const float rs = (c + i < t.rows) ? __ldg(rsp + c + i) : 0.f;
            a *= rs * ws_a;
            b *= rs * ws_b;
          }
          va[i] = GATED ? silu_mul(a, b) : a;
          vb[i] = b;
        }
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          // values of token c+i (even lanes keep) and c+i+1 (odd lanes keep)
          const float keep_a = even ? va[i] : va[i + 1], send_a = even ? va[i + 1] : va[i];
          const float recv_a = __shfl_xor_sync(0xffffffffu, send_a, 1);
          const int tok = c + i + (even ? 0 : 1);
          const uint32_t pa = even ? pack_bf16(keep_a, recv_a) : pack_bf16(recv_a, keep_a);
          if (GATED) {
            if (tok < t.rows && f_pair < n_feat)
              *reinterpret_cast<uint32_t*>(out + (size_t)(t.row0 + tok) * n_feat + f_pair) = pa;
          } else {
            const float keep_b = even ? vb[i] : vb[i + 1], send_b = even ? vb[i + 1] : vb[i];
            const float recv_b = __shfl_xor_sync(0xffffffffu, send_b, 1);
            const uint32_t pb = even ? pack_bf16(keep_b, recv_b) : pack_bf16(recv_b, keep_b);
            const int fa2 = f_a & ~1, fb2 = f_b & ~1;
            if (tok < t.rows) {
              __nv_bfloat16* orow = out + (size_t)(t.row0 + tok) * n_feat;
              if (fa2 < n_feat) *reinterpret_cast<uint32_t*>(orow + fa2) = pa;
              if (fb2 < n_feat) *reinterpret_cast<uint32_t*>(orow + fb2) = pb;
            }
          }
        }
      }
      release_acc();
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(p.status, kStOk, kStTimeout);
    }
  }

  // ---- teardown
  if (threadIdx.x == 0) PROF_STAMP(5);
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) PROF_STAMP(6);
  if (threadIdx.x == 0) {
    // The last CTA to get here puts the counters back for the next launch that uses them.  After a stop on request
    // the tile counter stays: the next launch of the pass goes on where this one stopped taking tiles.
    if (*stopped_here) atomicAdd(p.stopped, 1);
    __threadfence();
    if (atomicAdd(p.done_ctr, 1) == (int)gridDim.x - 1) {
      const bool any_stopped = p.stopped != nullptr && *reinterpret_cast<volatile int*>(p.stopped) != 0;
      *p.done_ctr = 0;
      if (!any_stopped) *p.tile_ctr = 0;
    }
  }
  if (*abort_flag) {
    // give copies still in flight time to land in this CTA's shared memory before it is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <typename Kernel>
cudaError_t launch_variant(Kernel kern, const CUtensorMap& mw, const CUtensorMap& mw2, const StreamMaps& xm,
                           const StreamParams& prm, int grid, size_t smem, cudaStream_t stream, bool overlap) {
  cudaError_t err = ensure_dynamic_smem(kern, smem);
  if (err != cudaSuccess) return err;
  return launch_pdl(overlap, kern, dim3(grid), dim3(kThreads), smem, stream, mw, mw2, xm, prm);
}

}  // namespace

cudaError_t launch_gemm_stream(const GemmProblem& p, const GemmDenseGroup* dense, int max_ctas, int* status,
                               cudaStream_t stream, int* n_launches) {
  if (dense != nullptr && dense->rows <= 0) dense = nullptr;
  if (p.rows_bound <= 0 && dense == nullptr) return cudaSuccess;
  if (p.rows_bound <= 0) return cudaErrorInvalidValue;  // a dense group never comes without its routed pass
  if (dense != nullptr && (dense->K % 8 != 0 || dense->n_feat % 8 != 0)) return cudaErrorNotSupported;
  if (!encoder_ready()) return cudaErrorNotSupported;
  if (p.K % 8 != 0 || p.n_feat % 8 != 0 || p.E < 1 || p.E > 1024) return cudaErrorNotSupported;
  if (p.gather_src != nullptr) return cudaErrorNotSupported;
  if (p.rows_bound > 0x7fffffffLL / 2) return cudaErrorNotSupported;
  const bool fp8 = p.fp8;
  if (fp8 && (p.row_scale == nullptr || p.w_scale == nullptr || p.K % 16 != 0 || p.n_feat % 64 != 0 ||
              (dense != nullptr && (dense->row_scale == nullptr || dense->w_scale == nullptr || dense->K % 16 != 0 ||
                                    dense->n_feat % 64 != 0))))
    return cudaErrorNotSupported;
  const uint64_t esz = fp8 ? 1 : 2;                                // bytes per operand element
  const uint32_t box_k = (uint32_t)(fp8 ? 2 * kBlockK : kBlockK);  // 128 bytes of K per k-block row
  const int groups = p.offsets ? p.E : 1;
  const int e_begin = p.offsets ? p.e_begin : 0;
  const int e_end = (p.offsets && p.e_end >= 0) ? p.e_end : groups;
  if (e_begin < 0 || e_end > groups || e_begin >= e_end) return cudaErrorInvalidValue;

  CUtensorMap mw, mw2;
  StreamMaps xm;
  // Weights: one box holds both 128-row weight boxes of a k-block.  Gated pass: [groups][2][n_feat][K] with a box
  // of 128 rows x 2 (gate rows and the matching up rows); down pass: [groups][n_feat][K] with a box of 256 rows.
  auto encode_w = [&](CUtensorMap* m, const void* W, uint64_t K, uint64_t n_feat, uint64_t n_groups) {
    if (p.gated) {
      const uint64_t dims[4] = {K, n_feat, 2, n_groups};
      const uint64_t str[3] = {K * esz, n_feat * K * esz, 2 * n_feat * K * esz};
      const uint32_t box[4] = {box_k, (uint32_t)kWBoxRows, 2u, 1u};
      return encode_map(m, W, 4, dims, str, box, fp8);
    }
    const uint64_t dims[3] = {K, n_feat, n_groups};
    const uint64_t str[2] = {K * esz, n_feat * K * esz};
    const uint32_t box[3] = {box_k, 2u * kWBoxRows, 1u};
    return encode_map(m, W, 3, dims, str, box, fp8);
  };
  auto encode_x = [&](CUtensorMap* maps, const void* A, uint64_t K, uint64_t rows) {
    for (int b = 0; b < kXMaps; ++b) {
      const uint64_t dims[2] = {K, rows};
      const uint64_t str[1] = {K * esz};
      const uint32_t box[2] = {box_k, 16u * (uint32_t)(b + 1)};
      if (!encode_map(&maps[b], A, 2, dims, str, box, fp8)) return false;
    }
    return true;
  };
  if (!encode_w(&mw, p.W, (uint64_t)p.K, (uint64_t)p.n_feat, (uint64_t)groups)) return cudaErrorInvalidValue;
  if (!encode_x(xm.x, p.A, (uint64_t)p.K, (uint64_t)p.rows_bound)) return cudaErrorInvalidValue;
  mw2 = mw;
  for (int b = 0; b < kXMaps; ++b) xm.x2[b] = xm.x[b];
  if (dense != nullptr) {
    if (!encode_w(&mw2, dense->W, (uint64_t)dense->K, (uint64_t)dense->n_feat, 1)) return cudaErrorInvalidValue;
    if (!encode_x(xm.x2, dense->A, (uint64_t)dense->K, (uint64_t)dense->rows)) return cudaErrorInvalidValue;
  }

  StreamParams prm;
  prm.offsets = p.offsets ? p.offsets + e_begin : nullptr;
  prm.fixed_rows = p.fixed_rows;
  prm.E = e_end - e_begin;
  prm.e_base = e_begin;
  prm.n_feat = p.n_feat;
  prm.K = p.K;
  prm.out = static_cast<__nv_bfloat16*>(p.out);
  prm.status = status;
  prm.inject_producer_stall = p.debug_stall ? 1 : 0;
  prm.wait_limit_ns = p.wait_limit_ns ? p.wait_limit_ns : kWaitLimitNs;
  prm.rows2 = dense ? dense->rows : 0;
  prm.n_feat2 = dense ? dense->n_feat : 8;
  prm.K2 = dense ? dense->K : 8;
  prm.out2 = dense ? static_cast<__nv_bfloat16*>(dense->out) : nullptr;
  prm.row_scale = p.row_scale;
  prm.w_scale = p.w_scale;
  prm.row_scale2 = dense ? dense->row_scale : nullptr;
  prm.w_scale2 = dense ? dense->w_scale : nullptr;
  if (p.tile_counters == nullptr) return cudaErrorInvalidValue;
  prm.tile_ctr = p.tile_counters;
  prm.done_ctr = p.tile_counters + 1;
  prm.all_dynamic = p.resumable ? 1 : 0;
  const bool preemptible = p.yield_req != nullptr && p.stopped != nullptr;
  prm.sort_tiles = (p.max_group_rows > 0 && p.max_group_rows <= 16) ? 0 : 1;
  prm.early_setup = (p.offsets_settled && !preemptible) ? 1 : 0;
  prm.yield_req = preemptible ? p.yield_req : nullptr;
  prm.stopped = preemptible ? p.stopped : nullptr;

  const size_t tail = (2 * kNB + 4 + 2 * kQ) * sizeof(uint64_t) + 3 * sizeof(uint32_t) + (kNB + kQ) * sizeof(int) +
                      4 * (size_t)(prm.E + 1) * sizeof(int);
  const int slots = (int)((kSmemBudget - 1024 - (int)tail) / kSlotBytes);
  if (slots < 2 * (kWSlots + kMaxTileRows / 16)) return cudaErrorNotSupported;
  prm.ring_slots = slots;
#ifdef MOE_STREAM_PROF
  if (const char* rs = getenv("MOE_STREAM_RING_SLOTS")) {  // debug build only: a smaller ring, to see what in-flight bytes buy
    const int v = atoi(rs);
    if (v >= 2 * (kWSlots + kMaxTileRows / 16) && v < slots) prm.ring_slots = v;
  }
#endif
  const size_t smem = 1024 + (size_t)slots * kSlotBytes + tail;

  const int feat_per_tile = p.gated ? 128 : 256;
  const int64_t n_ft = (p.n_feat + feat_per_tile - 1) / feat_per_tile;
  const int64_t row_tiles = p.rows_bound / kMaxTileRows + (prm.E < p.rows_bound ? prm.E : p.rows_bound);
  int64_t tiles = row_tiles * n_ft;
  if (dense != nullptr)
    tiles += (int64_t)((dense->rows + kMaxTileRows - 1) / kMaxTileRows) * ((dense->n_feat + feat_per_tile - 1) / feat_per_tile);
  int grid = (int)(tiles < (int64_t)max_ctas ? tiles : (int64_t)max_ctas);
  if (grid < 1) grid = 1;
  const bool overlap = p.rows_bound <= kGemmOverlapMaxRows;
  cudaError_t err;
  if (fp8)
    err = p.gated ? launch_variant(grouped_gemm_stream_kernel<true, true>, mw, mw2, xm, prm, grid, smem, stream, overlap)
                  : launch_variant(grouped_gemm_stream_kernel<false, true>, mw, mw2, xm, prm, grid, smem, stream, overlap);
  else
    err = p.gated ? launch_variant(grouped_gemm_stream_kernel<true, false>, mw, mw2, xm, prm, grid, smem, stream, overlap)
                  : launch_variant(grouped_gemm_stream_kernel<false, false>, mw, mw2, xm, prm, grid, smem, stream, overlap);
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

#ifdef MOE_STREAM_PROF
}  // namespace moe
extern "C" int moe_debug_stream_ts(unsigned long long* host) {
  return (int)cudaMemcpyFromSymbol(host, moe::g_stream_ts, sizeof(unsigned long long) * 8 * 256);
}
extern "C" int moe_debug_stream_prof(unsigned long long* host, int clear) {
  cudaError_t e = cudaMemcpyFromSymbol(host, moe::g_stream_prof, sizeof(unsigned long long) * 8 * 256);
  if (e == cudaSuccess && clear) {
    static unsigned long long zeros[8 * 256] = {};
    e = cudaMemcpyToSymbol(moe::g_stream_prof, zeros, sizeof zeros);
  }
  return (int)e;
}
namespace moe {
#endif

}  // namespace moe
