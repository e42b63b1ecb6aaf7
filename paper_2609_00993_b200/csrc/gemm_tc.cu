// Stages a6-a8: grouped expert GEMM on the 5th-generation tensor cores (sm_100a).
//
//   operands   bf16, K-major, staged in shared memory by TMA (128-byte swizzle), 64 K-elements per stage
//   math       tcgen05.mma (kind::f16, M=128) issued by one thread, fp32 accumulators in TMEM
//   epilogue   tcgen05.ld -> registers -> (SwiGLU) -> bf16 -> a per-warp swizzled staging tile in shared
//              memory -> tiled bulk stores (TMA) of 32-row x 64-feature boxes; the accumulator stage is handed
//              back as soon as it has been read, so the next tile's MMAs overlap the stores (two TMEM
//              accumulator stages)
//   schedule   persistent CTAs walk the tile list (expert, row tile, feature tile); the list is derived
//              on the device from the expert offsets, so no host synchronisation is needed
//
// This file is the large-M variant: tokens fill the MMA M dimension (128 rows); a stage's weight tile is 256 rows
// (gated: 128 gate rows + the matching 128 up rows), one N=256 MMA per 16 K-elements.  It is the variant for
// experts of many hundreds of rows, where the pass is bound by the tensor cores; the swap-AB variant for experts
// of few rows (weight streaming) is gemm_stream.cu.
// The kernel also exists for E4M3 operands (the FP8 precision variant): the same pipeline with 128 K-elements
// per stage row, tcgen05.mma.kind::f8f6f4 (32 K-elements per instruction) and an epilogue that multiplies the
// accumulator by the row's and the weight row's scale before SwiGLU / the bf16 store.
// An expert's row tile may run past the end of its segment: TMA needs no alignment on the row coordinate, so
// segments are NOT padded; rows that belong to the next expert are computed and simply not stored.  A last tile
// of at most 96 rows fetches only a 32-, 64- or 96-row box of token rows (whatever else lies in the stage is
// multiplied and dropped).
//
// Warp roles (192 threads): warps 0-3 epilogue (TMEM lanes 32w..32w+31), warp 4 TMA producer, warp 5 MMA
// issuer and TMEM owner.  The optional row-gather instantiation adds warps 6-9, which fetch the routed
// experts' token rows straight from the unpermuted activations with 16-byte asynchronous copies (the
// permutation is applied on the fly, so the separate row-permute pass is skipped).  Every mbarrier wait is bounded: on expiry the kernel records a timeout in the
// status word, raises a CTA-wide abort flag, lets copies in flight land, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>
#include <map>
#include <mutex>

#include "kernels.h"
#include "tc_common.cuh"

namespace moe {
namespace {

using namespace tc;

constexpr int kThreads = 192;
constexpr int kEpilogueWarps = 4;
constexpr int kProducerWarp = 4;
constexpr int kMmaWarp = 5;
constexpr int kGatherWarp0 = 6;      // row-gather variant: warps 6..9 fill the X tile themselves
constexpr int kGatherThreads = 128;
constexpr int kThreadsGather = kThreads + kGatherThreads;
constexpr int kMaxStages = 8;
constexpr int kEpiStagingBytes = kEpilogueWarps * 32 * 128;  // per-warp 32 x 128-byte staging tiles

struct TcParams {
  const int32_t* offsets;  // [E+1] (already advanced to the first expert of the launch) or nullptr
  int32_t fixed_rows;
  int32_t E;               // experts covered by this launch
  int32_t e_base;          // index of the launch's first expert in the weight tensor
  int32_t n_feat;          // output features (I for the gated pass, H for the down pass)
  int32_t K;
  __nv_bfloat16* out;      // [rows, n_feat]
  int32_t row_tile;        // tokens per tile: 128
  int32_t n_stages;
  int32_t x_tile_bytes;    // row_tile * 128
  int* status;
  int32_t inject_producer_stall;  // failure-detection test hook: the TMA producer issues nothing
  unsigned long long wait_limit_ns;
  // row-gather variant: row p of the grouped operand is gather_src[perm[p] / top_k, :] (gather_src2[p, :] for
  // the dense group); no permuted copy of the rows exists
  const __nv_bfloat16* gather_src;
  const __nv_bfloat16* gather_src2;
  const int32_t* perm;
  int32_t top_k;
  // optional dense group (shared expert) computed by the same launch; rows2 == 0: none
  int32_t rows2;
  int32_t n_feat2;
  int32_t K2;
  __nv_bfloat16* out2;
  // FP8 variant: operands are E4M3 codes; the accumulator is scaled by row_scale[row] * w_scale[weight row]
  // (w_scale: [experts, weight rows of one expert]; *2: the dense group's)
  const float* row_scale;
  const float* row_scale2;
  const float* w_scale;
  const float* w_scale2;
};


// Output tensor maps (large-M epilogue): [rows, n_feat] bf16 with boxes of 64 features x 32 rows, 128-byte swizzle
struct OutMaps {
  CUtensorMap o, o2;
  // large-M: the token rows again with 32-, 64- and 96-row boxes, for an expert's last tile when it holds no
  // more rows than that (the other rows of the X tile are never stored, so nothing needs to be fetched for them)
  CUtensorMap xs[3], xs2[3];
};
struct Tile {
  int e, row0, rows, ft;
  bool dense;  // a tile of the dense group
};

// tile -> (expert, first row, valid rows, feature tile).  The dense group's tiles come first (row tile major),
// then the experts': prefix[e] = row tiles of experts < e.
__device__ __forceinline__ Tile decode_tile(int tile, int dense_tiles, int n_ft2, int rows2, int n_ft, int E,
                                            const int* prefix, const int* seg, int row_tile) {
  Tile t;
  if (tile < dense_tiles) {
    const int rt = tile / n_ft2;
    t.e = 0;
    t.ft = tile - rt * n_ft2;
    t.row0 = rt * row_tile;
    t.rows = min(row_tile, rows2 - t.row0);
    t.dense = true;
    return t;
  }
  tile -= dense_tiles;
  const int rt = tile / n_ft;
  int lo = 0, hi = E;  // largest e in [0,E) with prefix[e] <= rt
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= rt) lo = mid; else hi = mid;
  }
  t.e = lo;
  t.ft = tile - rt * n_ft;
  const int mt = rt - prefix[lo];
  t.row0 = seg[lo] + mt * row_tile;
  t.rows = min(row_tile, seg[lo + 1] - t.row0);
  t.dense = false;
  return t;
}

// ------------------------------------------------------------------------------------- the kernel
// GATHER (large-M, gated pass only): the token rows are not read from a permuted copy.  Four extra warps copy
// each row's 128-byte slice for the current k-block from its source row (perm[p] / top_k) into the X tile with
// 16-byte cp.async, in the same 128-byte-swizzled layout TMA would produce; the stage's barrier counts one
// arrival per gather thread, delivered when that thread's copies have landed.  TMA then carries the weights only.
// FP8: both operands are E4M3 codes, a pipeline stage holds 128 K-elements (still 128 bytes per row), and the
// epilogue multiplies the accumulator by the row's and the weight row's scale.
template <bool GATED, bool GATHER, bool FP8>
__global__ void __launch_bounds__(GATHER ? kThreadsGather : kThreads, 1)
grouped_gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_x2, const __grid_constant__ CUtensorMap map_w2,
                       const __grid_constant__ OutMaps omaps, const __grid_constant__ TcParams p) {
  static_assert(!(GATHER && FP8), "the row gather exists for bf16 operands only");
  constexpr int kbk = FP8 ? 2 * kBlockK : kBlockK;  // K elements per stage
  extern __shared__ uint8_t smem_raw[];
  // carve: [stages] | epilogue staging (large-M) | barriers | tmem slot | abort | prefix[E+1] | seg[E+1]
  //   stage: W box0 | W box1 | X tile
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
  uint8_t* base = smem_raw + (base_addr - raw_addr);
  const int stage_bytes = 2 * kWBoxBytes + p.x_tile_bytes;
  uint8_t* epi_smem = base + (size_t)p.n_stages * stage_bytes;  // kEpilogueWarps x 4 KB, large-M only
  uint8_t* after = epi_smem + kEpiStagingBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(after);  // full[S], empty[S], tmem_full[2], tmem_empty[2]
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8u * p.n_stages;
  const uint32_t bar_tfull = bar_empty + 8u * p.n_stages;
  const uint32_t bar_tempty = bar_tfull + 16u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* prefix = reinterpret_cast<int*>(tmem_slot + 2);
  int* seg = prefix + (p.E + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = (int)blockIdx.x, n_units = (int)gridDim.x;
  const int tile_rows = p.row_tile;  // token rows per tile of the list
  constexpr int kFeatPerTile = GATED ? 128 : 256;
  const int n_ft = (p.n_feat + kFeatPerTile - 1) / kFeatPerTile;
  const int num_kb1 = (p.K + kbk - 1) / kbk, num_kb2 = (p.K2 + kbk - 1) / kbk;
  const int n_ft2 = (p.n_feat2 + kFeatPerTile - 1) / kFeatPerTile;
  const int dense_tiles = p.rows2 > 0 ? ((p.rows2 + p.row_tile - 1) / p.row_tile) * n_ft2 : 0;
  constexpr uint32_t acc_cols = 256u;  // TMEM columns per accumulator stage
  constexpr uint32_t tmem_cols = 2u * acc_cols;

  // ---- set-up: barriers, TMEM (both before the previous kernel of the stream is known to be complete), tile list
  if (threadIdx.x == 32) {
    for (int s = 0; s < p.n_stages; ++s) {
      mbar_init(bar_full + 8u * s, GATHER ? 1 + kGatherThreads : 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, kEpilogueWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kMmaWarp) tmem_alloc(smem_u32(tmem_slot), tmem_cols);
  pdl_wait();
  pdl_launch_dependents();
  if (warp == 0) {
    int carry = 0;
    for (int b = 0; b < p.E; b += 32) {
      const int e = b + lane;
      int beg = 0, cnt = 0;
      if (e < p.E) {
        beg = p.offsets ? p.offsets[e] : 0;
        cnt = p.offsets ? p.offsets[e + 1] - beg : p.fixed_rows;
        if (cnt < 0) cnt = 0;
        seg[e] = beg;
        if (e == p.E - 1) seg[p.E] = beg + cnt;
      }
      const int tiles = (cnt + tile_rows - 1) / tile_rows;
      int incl = tiles;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += n;
      }
      if (e < p.E) prefix[e] = carry + incl - tiles;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) prefix[p.E] = carry;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total_tiles = dense_tiles + prefix[p.E] * n_ft;

  if (warp == kProducerWarp) {
    // ================================================================= TMA producer (one lane)
    if (lane == 0 && !p.inject_producer_stall) {
      RingCursor ring;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
        const Tile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, seg, tile_rows);
        const int w_row0 = t.ft * kFeatPerTile;
        const int w_row1 = GATED ? (t.dense ? p.n_feat2 : p.n_feat) + t.ft * kFeatPerTile : w_row0 + kWBoxRows;
        const CUtensorMap* mw = t.dense ? &map_w2 : &map_w;
        const CUtensorMap* mx = t.dense ? &map_x2 : &map_x;
        const int w_e = t.dense ? 0 : p.e_base + t.e;
        const int num_kb = t.dense ? num_kb2 : num_kb1;
        const uint32_t x_rows = (uint32_t)((t.rows + 31) & ~31);  // rows worth fetching, in steps of 32
        const bool short_x = !GATHER && x_rows < 128u;
        const CUtensorMap* mxs = (t.dense ? omaps.xs2 : omaps.xs) + (short_x ? x_rows / 32u - 1u : 0u);
        for (int kb = 0, k0 = 0; kb < num_kb; ++kb, k0 += kbk) {
          if (!mbar_wait(bar_empty + 8u * ring.stage, ring.phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
          const uint32_t full = bar_full + 8u * ring.stage;
          const uint32_t st = base_addr + ring.stage * (uint32_t)stage_bytes;
          mbar_expect_tx(full, GATHER ? 2u * kWBoxBytes : (short_x ? 2u * kWBoxBytes + x_rows * 128u : (uint32_t)stage_bytes));
          tma_load_3d(st, mw, full, k0, w_row0, w_e);
          tma_load_3d(st + kWBoxBytes, mw, full, k0, w_row1, w_e);
          if (!GATHER) tma_load_2d(st + 2 * kWBoxBytes, short_x ? mxs : mx, full, k0, t.row0);
          ring.advance((uint32_t)p.n_stages);
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(p.status, kStOk, kStTimeout);
      }
    }
  } else if (warp == kMmaWarp) {
    // ================================================================= MMA issuer (one lane)
    if (lane == 0) {
      uint32_t tile_iter = 0;
      RingCursor ring;
      bool ok = true;
      // descriptor words: only the 14-bit start-address field of the low word changes between MMAs
      const uint32_t desc_hi = (uint32_t)(umma_smem_desc(0) >> 32);
      const uint32_t lo_base = (uint32_t)umma_smem_desc(base_addr);  // stage 0, weight box 0
      const uint32_t lo_stage = (uint32_t)stage_bytes >> 4, lo_box = (uint32_t)kWBoxBytes >> 4;
      for (int tile = unit; tile < total_tiles && ok; tile += n_units, ++tile_iter) {
        const Tile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, seg, tile_rows);
        const uint32_t as = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
        if (!mbar_wait(bar_tempty + 8u * as, aph ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d0 = tmem_base + as * acc_cols;
        const uint32_t idesc = FP8 ? umma_idesc_e4m3(128, 256) : umma_idesc(128, 256);
        const int num_kb = t.dense ? num_kb2 : num_kb1;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(bar_full + 8u * ring.stage, ring.phase, abort_flag, p.wait_limit_ns)) { ok = false; break; }
          if (GATHER) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // X rows came by cp.async
          tc_fence_after();
          const uint32_t lo_w0 = lo_base + ring.stage * lo_stage;  // weight box 0; box 1 and the X tile follow
#pragma unroll
          for (int kk = 0; kk < kBlockK / kUmmaK; ++kk) {
            const uint32_t adv = (uint32_t)((kk * kUmmaK * 2) >> 4);  // +32 bytes per MMA (16 bf16 or 32 E4M3), in 16-byte units
            const uint32_t acc = (kb | kk) != 0 ? 1u : 0u;
            auto mma = [&](uint32_t d, uint32_t a_lo, uint32_t b_lo) {
              if (FP8) umma_e4m3_lo(d, a_lo, b_lo, desc_hi, idesc, acc);
              else umma_bf16_lo(d, a_lo, b_lo, desc_hi, idesc, acc);
            };
            // the two weight boxes are contiguous: one N = 256 operand
            mma(d0, lo_w0 + 2 * lo_box + adv, lo_w0 + adv);
          }
          umma_commit(bar_empty + 8u * ring.stage);  // the stage is free once these MMAs have read it
          ring.advance((uint32_t)p.n_stages);
        }
        if (ok) umma_commit(bar_tfull + 8u * as);  // accumulator complete
      }
      if (!ok) {
        *abort_flag = 1;
        atomicCAS(p.status, kStOk, kStTimeout);
      }
    }
  } else if (GATHER && warp >= kGatherWarp0) {
    // ================================================================= row gather (warps 6-9)
    // thread g owns the 16-byte piece (g & 7) of rows (g >> 3) + 16 i, i < 8, of every stage
    const int g = (int)threadIdx.x - kGatherWarp0 * 32;
    const int piece = g & 7, rbase = g >> 3;
    const uint32_t dst_off = (uint32_t)(rbase * 128 + ((piece ^ (rbase & 7)) << 4));  // 128-byte swizzle
    RingCursor ring;
    bool ok = true;
    // The source row of each of this thread's 8 rows (flat slot = perm[row]; source row = slot / top_k; the
    // dense group's rows are their own source) is fetched one tile ahead, so that the dependent perm load is
    // not on the path of a tile's first copies.  -1: the row lies past the tile's end.
    int slot_next[8];
    auto fetch_slots = [&](int tile, int (&slot)[8]) {
      if (tile >= total_tiles) return;
      const Tile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, seg, tile_rows);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int r = rbase + 16 * i;
        slot[i] = -1;
        if (r < t.rows) slot[i] = t.dense ? (t.row0 + r) * p.top_k : __ldg(p.perm + t.row0 + r);
      }
    };
    fetch_slots(unit, slot_next);
    for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
      const Tile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, seg, tile_rows);
      const __nv_bfloat16* src = t.dense ? p.gather_src2 : p.gather_src;
      const int Kt = t.dense ? p.K2 : p.K;
      const __nv_bfloat16* row_ptr[8];  // nullptr: the row is left as it is; its result is never stored
#pragma unroll
      for (int i = 0; i < 8; ++i)
        row_ptr[i] = slot_next[i] < 0 ? nullptr : src + (size_t)(slot_next[i] / p.top_k) * Kt + piece * 8;
      fetch_slots(tile + n_units, slot_next);
      const int num_kb = t.dense ? num_kb2 : num_kb1;
      for (int kb = 0, k0 = 0; kb < num_kb; ++kb, k0 += kBlockK) {
        if (!mbar_wait(bar_empty + 8u * ring.stage, ring.phase ^ 1u, abort_flag, p.wait_limit_ns)) { ok = false; break; }
        const uint32_t xs = base_addr + ring.stage * (uint32_t)stage_bytes + 2 * kWBoxBytes + dst_off;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (row_ptr[i] != nullptr) cp_async_16(xs + (uint32_t)(i * 16 * 128), row_ptr[i] + k0);
        // one arrival on the stage's barrier, delivered by the hardware when this thread's copies have landed
        cp_async_arrive_on(bar_full + 8u * ring.stage);
        ring.advance((uint32_t)p.n_stages);
      }
    }
    if (!ok) {
      *abort_flag = 1;
      atomicCAS(p.status, kStOk, kStTimeout);
    }
  } else {
    // ================================================================= epilogue (warps 0-3)
    uint32_t tile_iter = 0;
    bool ok = true;
    const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
    for (int tile = unit; tile < total_tiles && ok; tile += n_units, ++tile_iter) {
      const Tile t = decode_tile(tile, dense_tiles, n_ft2, p.rows2, n_ft, p.E, prefix, seg, tile_rows);
      const uint32_t as = tile_iter & 1u, aph = (tile_iter >> 1) & 1u;
      auto release_acc = [&]() {  // hand the accumulator stage back to the MMA issuer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8u * as);
      };
      if (!mbar_wait(bar_tfull + 8u * as, aph, abort_flag, p.wait_limit_ns)) { ok = false; break; }
      tc_fence_after();
      const uint32_t d0 = tmem_base + as * acc_cols + lane_base;
      __nv_bfloat16* const out = t.dense ? p.out2 : p.out;
      const int n_feat = t.dense ? p.n_feat2 : p.n_feat;
      // FP8: scales of this tile's rows and of its expert's weight rows (gate rows first, then up rows)
      const float* const rsp = FP8 ? (t.dense ? p.row_scale2 : p.row_scale) + t.row0 : nullptr;
      const float* const wsp =
          FP8 ? (t.dense ? p.w_scale2 : p.w_scale + (size_t)(p.e_base + t.e) * (GATED ? 2 : 1) * n_feat) : nullptr;
      bool released = false;  // has this warp already handed the accumulator stage back?
      {
        // lane = token row, column = output feature.  Two 32-column chunks (128 bytes of a row) at a time go
        // through a per-warp staging tile in shared memory whose 16-byte pieces are XOR-swizzled by row: that
        // is conflict-free both ways and it is TMA's 128-byte swizzle, so a warp whose 32 rows are all valid
        // sends the 4 KB box with one tiled bulk store.  A ragged warp (the expert's last rows) stores by hand,
        // every store instruction writing four whole 128-byte lines.
        constexpr int kPairs = kFeatPerTile / 64;
        uint8_t* stage_tile = epi_smem + warp * 4096;  // 32 rows x 128 bytes
        const int rows_here = t.rows - warp * 32;       // rows of this warp's 32 that are valid (may be <= 0)
        const float rs = (FP8 && lane < rows_here) ? rsp[warp * 32 + lane] : 0.f;  // FP8: this lane's row scale
        for (int pc = 0; pc < kPairs; ++pc) {
          const int f0 = t.ft * kFeatPerTile + pc * 64;
          if (f0 >= n_feat) break;  // uniform across the CTA
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t ra[32], packed[16];
            tmem_ld32(d0 + (uint32_t)(pc * 64 + h * 32), ra);
            // FP8: the 32 columns' weight-row scales (the same for every lane: broadcast loads); a chunk that
            // reaches past n_feat reads no scales and is not stored either
            const bool scaled = FP8 && f0 + h * 32 + 32 <= n_feat;
            if (GATED) {
              uint32_t rb[32];
              tmem_ld32(d0 + (uint32_t)(128 + pc * 64 + h * 32), rb);
              tmem_ld_wait();
              if (FP8) {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                  const float4 sg = scaled ? __ldg(reinterpret_cast<const float4*>(wsp + f0 + h * 32) + q)
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                  const float4 su = scaled ? __ldg(reinterpret_cast<const float4*>(wsp + n_feat + f0 + h * 32) + q)
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                  ra[4 * q + 0] = __float_as_uint(__uint_as_float(ra[4 * q + 0]) * (rs * sg.x));
                  ra[4 * q + 1] = __float_as_uint(__uint_as_float(ra[4 * q + 1]) * (rs * sg.y));
                  ra[4 * q + 2] = __float_as_uint(__uint_as_float(ra[4 * q + 2]) * (rs * sg.z));
                  ra[4 * q + 3] = __float_as_uint(__uint_as_float(ra[4 * q + 3]) * (rs * sg.w));
                  rb[4 * q + 0] = __float_as_uint(__uint_as_float(rb[4 * q + 0]) * (rs * su.x));
                  rb[4 * q + 1] = __float_as_uint(__uint_as_float(rb[4 * q + 1]) * (rs * su.y));
                  rb[4 * q + 2] = __float_as_uint(__uint_as_float(rb[4 * q + 2]) * (rs * su.z));
                  rb[4 * q + 3] = __float_as_uint(__uint_as_float(rb[4 * q + 3]) * (rs * su.w));
                }
              }
#pragma unroll
              for (int i = 0; i < 16; ++i)
                packed[i] = pack_bf16(silu_mul(__uint_as_float(ra[2 * i]), __uint_as_float(rb[2 * i])),
                                      silu_mul(__uint_as_float(ra[2 * i + 1]), __uint_as_float(rb[2 * i + 1])));
            } else {
              tmem_ld_wait();
              if (FP8) {
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                  const float4 sw = scaled ? __ldg(reinterpret_cast<const float4*>(wsp + f0 + h * 32) + q)
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                  ra[4 * q + 0] = __float_as_uint(__uint_as_float(ra[4 * q + 0]) * (rs * sw.x));
                  ra[4 * q + 1] = __float_as_uint(__uint_as_float(ra[4 * q + 1]) * (rs * sw.y));
                  ra[4 * q + 2] = __float_as_uint(__uint_as_float(ra[4 * q + 2]) * (rs * sw.z));
                  ra[4 * q + 3] = __float_as_uint(__uint_as_float(ra[4 * q + 3]) * (rs * sw.w));
                }
              }
#pragma unroll
              for (int i = 0; i < 16; ++i) packed[i] = pack_bf16(__uint_as_float(ra[2 * i]), __uint_as_float(ra[2 * i + 1]));
            }
            if (h == 1 && (pc == kPairs - 1 || f0 + 64 >= n_feat)) {
              release_acc();  // the accumulator has been read completely: hand it back before the stores go out
              released = true;
            }
            if (h == 0) {  // the previous tiled store (lane 0's) has read the staging tile
              if (lane == 0) bulk_wait_read_all();
              __syncwarp();
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
              *reinterpret_cast<uint4*>(stage_tile + lane * 128 + (((h * 4 + j) ^ (lane & 7)) << 4)) =
                  make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
          }
          if (rows_here >= 32 && f0 + 64 <= n_feat) {
            // a full 32-row x 64-feature box: one tiled bulk store (the staging layout is the 128-byte swizzle)
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(t.dense ? &omaps.o2 : &omaps.o, smem_u32(stage_tile), f0, t.row0 + warp * 32);
              bulk_commit();
            }
            continue;
          }
          __syncwarp();
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int rr = it * 4 + (lane >> 3), piece = lane & 7;
            const uint4 v = *reinterpret_cast<const uint4*>(stage_tile + rr * 128 + ((piece ^ (rr & 7)) << 4));
            if (rr < rows_here && f0 + piece * 8 < n_feat)
              *reinterpret_cast<uint4*>(out + (size_t)(t.row0 + warp * 32 + rr) * n_feat + f0 + piece * 8) = v;
          }
          __syncwarp();
        }
      }
      if (!released) release_acc();
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicCAS(p.status, kStOk, kStTimeout);
    }
    if (lane == 0) bulk_wait_all();  // the tiled stores are complete before the staging tiles are given up
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies still in flight time to land in this CTA's shared memory before it is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

// --------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
const char* g_init_error = nullptr;

template <typename Kernel>
cudaError_t launch_variant(Kernel kern, int threads, const CUtensorMap& mx, const CUtensorMap& mw,
                           const CUtensorMap& mx2, const CUtensorMap& mw2, const OutMaps& om, const TcParams& prm,
                           int grid, size_t smem, cudaStream_t stream, bool overlap) {
  cudaError_t err = ensure_dynamic_smem(kern, smem);
  if (err != cudaSuccess) return err;
  return launch_pdl(overlap, kern, dim3(grid), dim3(threads), smem, stream, mx, mw, mx2, mw2, om, prm);
}

}  // namespace

namespace tc {
// Encoded maps are pure functions of their arguments, so they are memoised process-wide: steady-state launches
// (same buffers, same shapes) then make no driver call besides the launch itself.
bool encode_map(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                const uint32_t* box, bool bytes) {
  if (rank < 2 || rank > 4) return false;
  struct Key {
    const void* base;
    uint64_t dims[4], strides[3];
    uint32_t box[4];
    int rank, bytes;
    bool operator<(const Key& o) const { return memcmp(this, &o, sizeof(Key)) < 0; }
  };
  Key key;
  memset(&key, 0, sizeof key);
  key.base = base;
  key.rank = rank;
  key.bytes = bytes ? 1 : 0;
  for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides_bytes[i];
  static std::mutex mu;
  static std::map<Key, CUtensorMap> cache;
  std::lock_guard<std::mutex> lock(mu);
  auto it = cache.find(key);
  if (it != cache.end()) {
    *map = it->second;
    return true;
  }
  cuuint64_t gdim[4];
  cuuint64_t gstr[3];
  cuuint32_t bdim[4];
  cuuint32_t estr[4] = {1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bdim[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  CUresult r = g_encode(map, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr,
                        bdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() >= 4096) cache.clear();
  cache.emplace(key, *map);
  return true;
}

bool encoder_ready() { return g_encode != nullptr || gemm_tc_init(nullptr); }
}  // namespace tc

bool gemm_tc_init(const char** why) {
  if (g_encode != nullptr) return true;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (err != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess) {
    g_init_error = "cuTensorMapEncodeTiled is not available from the installed driver";
    if (why) *why = g_init_error;
    (void)cudaGetLastError();
    return false;
  }
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return true;
}

cudaError_t launch_gemm_tc(const GemmProblem& p, const GemmDenseGroup* dense, int max_ctas, int* status,
                           cudaStream_t stream, int* n_launches) {
  constexpr int row_tile = 128;
  if (dense != nullptr && dense->rows <= 0) dense = nullptr;
  if (p.rows_bound <= 0 && dense == nullptr) return cudaSuccess;
  if (p.rows_bound <= 0) return cudaErrorInvalidValue;  // a dense group never comes without its routed pass
  if (dense != nullptr && (dense->K % 8 != 0 || dense->n_feat % 8 != 0)) return cudaErrorNotSupported;
  if (g_encode == nullptr && !gemm_tc_init(nullptr)) return cudaErrorNotSupported;
  if (p.K % 8 != 0 || p.n_feat % 8 != 0 || p.E < 1 || p.E > 1024) return cudaErrorNotSupported;
  const bool gather = p.gather_src != nullptr;
  if (gather && (!p.gated || p.perm == nullptr || p.top_k < 1 || p.K % kBlockK != 0 ||
                 (dense != nullptr && dense->K % kBlockK != 0)))
    return cudaErrorNotSupported;
  if (p.rows_bound > 0x7fffffffLL / 2) return cudaErrorNotSupported;

  const bool fp8 = p.fp8;
  if (fp8 && (gather || p.row_scale == nullptr || p.w_scale == nullptr || p.K % 16 != 0 || p.n_feat % 64 != 0 ||
              (dense != nullptr && (dense->row_scale == nullptr || dense->w_scale == nullptr || dense->K % 16 != 0 ||
                                    dense->n_feat % 64 != 0))))
    return cudaErrorNotSupported;
  const uint64_t esz = fp8 ? 1 : 2;                                    // bytes per operand element
  const uint32_t box_k = (uint32_t)(fp8 ? 2 * kBlockK : kBlockK);      // 128 bytes of K per stage row
  const int groups = p.offsets ? p.E : 1;
  const uint64_t w_rows = (uint64_t)(p.gated ? 2 : 1) * (uint64_t)p.n_feat;
  CUtensorMap mx, mw;
  {
    const uint64_t src_rows = gather ? (uint64_t)((p.rows_bound + p.top_k - 1) / p.top_k) : (uint64_t)p.rows_bound;
    const uint64_t dims[2] = {(uint64_t)p.K, src_rows};
    const uint64_t str[1] = {(uint64_t)p.K * esz};
    const uint32_t box[2] = {box_k, (uint32_t)row_tile};
    // with the row gather no tensor map of the token rows is used; encode the source so that the map is valid
    if (!encode_map(&mx, gather ? p.gather_src : p.A, 2, dims, str, box, fp8)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[3] = {(uint64_t)p.K, w_rows, (uint64_t)groups};
    const uint64_t str[2] = {(uint64_t)p.K * esz, w_rows * (uint64_t)p.K * esz};
    const uint32_t box[3] = {box_k, (uint32_t)kWBoxRows, 1u};
    if (!encode_map(&mw, p.W, 3, dims, str, box, fp8)) return cudaErrorInvalidValue;
  }

  const int e_begin = p.offsets ? p.e_begin : 0;
  const int e_end = (p.offsets && p.e_end >= 0) ? p.e_end : groups;
  if (e_begin < 0 || e_end > groups || e_begin >= e_end) return cudaErrorInvalidValue;
  CUtensorMap mx2 = mx, mw2 = mw;
  if (dense != nullptr) {
    const uint64_t w2_rows = (uint64_t)(p.gated ? 2 : 1) * (uint64_t)dense->n_feat;
    const uint64_t dx[2] = {(uint64_t)dense->K, (uint64_t)dense->rows};
    const uint64_t sx[1] = {(uint64_t)dense->K * esz};
    const uint32_t bx[2] = {box_k, (uint32_t)row_tile};
    if (!encode_map(&mx2, dense->A, 2, dx, sx, bx, fp8)) return cudaErrorInvalidValue;
    const uint64_t dw[3] = {(uint64_t)dense->K, w2_rows, 1};
    const uint64_t sw[2] = {(uint64_t)dense->K * esz, w2_rows * (uint64_t)dense->K * esz};
    const uint32_t bw[3] = {box_k, (uint32_t)kWBoxRows, 1u};
    if (!encode_map(&mw2, dense->W, 3, dw, sw, bw, fp8)) return cudaErrorInvalidValue;
  }
  OutMaps om;
  {
    const uint64_t d[2] = {(uint64_t)p.n_feat, (uint64_t)p.rows_cap};
    const uint64_t st[1] = {(uint64_t)p.n_feat * 2};
    const uint32_t bx[2] = {(uint32_t)(p.n_feat < 64 ? p.n_feat : 64), 32u};
    if (!encode_map(&om.o, p.out, 2, d, st, bx)) return cudaErrorInvalidValue;
    om.o2 = om.o;
    if (dense != nullptr) {
      const uint64_t d2[2] = {(uint64_t)dense->n_feat, (uint64_t)dense->rows};
      const uint64_t st2[1] = {(uint64_t)dense->n_feat * 2};
      const uint32_t bx2[2] = {(uint32_t)(dense->n_feat < 64 ? dense->n_feat : 64), 32u};
      if (!encode_map(&om.o2, dense->out, 2, d2, st2, bx2)) return cudaErrorInvalidValue;
    }
  }
  for (int m = 0; m < 3; ++m) {
    om.xs[m] = mx;
    om.xs2[m] = mx2;
  }
  if (!gather) {
    for (int m = 0; m < 3; ++m) {
      const uint64_t dims[2] = {(uint64_t)p.K, (uint64_t)p.rows_bound};
      const uint64_t str[1] = {(uint64_t)p.K * esz};
      const uint32_t box[2] = {box_k, (uint32_t)(32 * (m + 1))};
      if (!encode_map(&om.xs[m], p.A, 2, dims, str, box, fp8)) return cudaErrorInvalidValue;
      om.xs2[m] = om.xs[m];
      if (dense != nullptr) {
        const uint64_t dx[2] = {(uint64_t)dense->K, (uint64_t)dense->rows};
        const uint64_t sx[1] = {(uint64_t)dense->K * esz};
        if (!encode_map(&om.xs2[m], dense->A, 2, dx, sx, box, fp8)) return cudaErrorInvalidValue;
      }
    }
  }
  TcParams prm;
  prm.gather_src = static_cast<const __nv_bfloat16*>(p.gather_src);
  prm.gather_src2 = dense ? static_cast<const __nv_bfloat16*>(dense->A) : nullptr;
  prm.perm = p.perm ? p.perm + 0 : nullptr;
  prm.top_k = p.top_k;
  prm.rows2 = dense ? dense->rows : 0;
  prm.n_feat2 = dense ? dense->n_feat : 8;
  prm.K2 = dense ? dense->K : 8;
  prm.out2 = dense ? static_cast<__nv_bfloat16*>(dense->out) : nullptr;
  prm.row_scale = p.row_scale;
  prm.w_scale = p.w_scale;
  prm.row_scale2 = dense ? dense->row_scale : nullptr;
  prm.w_scale2 = dense ? dense->w_scale : nullptr;
  prm.offsets = p.offsets ? p.offsets + e_begin : nullptr;
  prm.fixed_rows = p.fixed_rows;
  prm.E = e_end - e_begin;
  prm.e_base = e_begin;
  prm.n_feat = p.n_feat;
  prm.K = p.K;
  prm.out = static_cast<__nv_bfloat16*>(p.out);
  prm.row_tile = row_tile;
  prm.x_tile_bytes = row_tile * kBlockK * 2;
  prm.status = status;
  prm.inject_producer_stall = p.debug_stall ? 1 : 0;
  prm.wait_limit_ns = p.wait_limit_ns ? p.wait_limit_ns : kWaitLimitNs;
  const int stage_bytes = 2 * kWBoxBytes + prm.x_tile_bytes;
  const size_t tail = kEpiStagingBytes + (2 * kMaxStages + 4) * sizeof(uint64_t) +
                      2 * sizeof(uint32_t) + 2 * (size_t)(prm.E + 1) * sizeof(int);
  int stages = (int)((kSmemBudget - 1024 - (int)tail) / stage_bytes);
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return cudaErrorNotSupported;
  prm.n_stages = stages;
  const size_t smem = 1024 + (size_t)stages * stage_bytes + tail;

  const int feat_per_tile = p.gated ? 128 : 256;
  const int64_t n_ft = (p.n_feat + feat_per_tile - 1) / feat_per_tile;
  const int64_t row_tiles = p.rows_bound / row_tile + (prm.E < p.rows_bound ? prm.E : p.rows_bound);
  int64_t tiles = row_tiles * n_ft;
  if (dense != nullptr)
    tiles += (int64_t)((dense->rows + row_tile - 1) / row_tile) * ((dense->n_feat + feat_per_tile - 1) / feat_per_tile);

  int grid = (int)(tiles < (int64_t)max_ctas ? tiles : (int64_t)max_ctas);
  if (grid < 1) grid = 1;
  const bool overlap = p.rows_bound <= kGemmOverlapMaxRows;
  cudaError_t err;
  if (gather)
    err = launch_variant(grouped_gemm_tc_kernel<true, true, false>, kThreadsGather, mx, mw, mx2, mw2, om, prm, grid, smem, stream, overlap);
  else if (fp8)
    err = p.gated ? launch_variant(grouped_gemm_tc_kernel<true, false, true>, kThreads, mx, mw, mx2, mw2, om, prm, grid, smem, stream, overlap)
                  : launch_variant(grouped_gemm_tc_kernel<false, false, true>, kThreads, mx, mw, mx2, mw2, om, prm, grid, smem, stream, overlap);
  else
    err = p.gated ? launch_variant(grouped_gemm_tc_kernel<true, false, false>, kThreads, mx, mw, mx2, mw2, om, prm, grid, smem, stream, overlap)
                  : launch_variant(grouped_gemm_tc_kernel<false, false, false>, kThreads, mx, mw, mx2, mw2, om, prm, grid, smem, stream, overlap);
  if (err == cudaSuccess && n_launches) *n_launches += 1;
  return err;
}

}  // namespace moe
