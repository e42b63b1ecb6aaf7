// C ABI (include/moe_pd.h): phase contexts, workspace carving, host-side validation, call ordering.
// All compute is in the kernels behind kernels.h; this file only validates, carves and enqueues.
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>
#include <new>
#include <vector>

#include "../../include/moe_pd.h"
#include "kernels.h"

namespace {

// ST_NOTIFIED: the first half of a split dispatch has been enqueued (counts, scan, permutation) and the routed
// data movement is pending; ST_LAYOUT_ONLY: a layout without rows (moe_dispatch_layout with x == NULL).
enum StepState { ST_IDLE = 0, ST_ROUTED = 1, ST_LAID_OUT = 2, ST_LAYOUT_ONLY = 3, ST_FFN_DONE = 4, ST_NOTIFIED = 5 };

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// One buffer set: everything the kernels of one step write.
struct BufferSet {
  char* x_perm;      // bf16 [N,H]
  char* act;         // bf16 [N,I]
  char* y_perm;      // bf16 [N,H]
  char* act_shared;  // bf16 [T,Is]
  char* y_shared;    // bf16 [T,H]
  int32_t* counts;   // [E]
  int32_t* offsets;  // [E+1]
  int32_t* perm;     // [N]
  int32_t* inv_perm; // [N]
  int32_t* topk_idx; // [N]   (host-input path)
  float* topk_w;     // [N]
  float* logits;     // [T,E] staging (host-input path)
  char* x_stage;     // bf16 [T,H]
  char* out_stage;   // bf16 [T,H]
  int32_t* scan;     // layout scratch
  // FP8 variant only: quantised activations and their per-row scales
  char* xq;          // e4m3 [N,H]
  float* sx;         // [N]
  char* aq;          // e4m3 [N,I]
  float* sa;         // [N]
  char* xq_tok;      // e4m3 [T,H]: x quantised in token order (the shared expert's GEMM1 input)
  float* sx_tok;     // [T]
  char* aq_shared;   // e4m3 [T,Is]
  float* sa_shared;  // [T]
};

struct Layout {
  size_t set_bytes;    // bytes of one buffer set
  size_t total_bytes;  // status block + all sets
  int n_sets;
};

// Status block at the start of the workspace: word 0 the device status, word 1 the count of CTAs that stopped on a
// yield request in the last preemptible launch, word 2 the yield request itself (device memory: every CTA polls it
// before each tile, which a word in host memory would not survive -- 148 SMs reading it over PCIe serialise), and
// from byte 64 on four pairs {next tile, CTAs finished} that the small-M GEMM launches use in rotation.
constexpr size_t kStatusBlock = 8192;
constexpr size_t kTileCounterOffset = 64;
constexpr int kTileCounterPairs = 4;

// Walks the carve of one buffer set; with base == nullptr it only measures.
size_t carve_set(const moe_config& c, char* base, BufferSet* out) {
  const size_t T = (size_t)c.max_tokens, N = T * (size_t)c.top_k, H = (size_t)c.hidden, I = (size_t)c.inter;
  const size_t E = (size_t)c.n_experts, Is = c.n_shared ? (size_t)c.shared_inter : 0;
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    char* p = base ? base + off : nullptr;
    off += align_up(bytes ? bytes : 1, 256);
    return p;
  };
  const size_t f8 = c.weight_format == MOE_WEIGHTS_FP8_E4M3 ? 1 : 0;
  BufferSet b;
  b.x_perm = take(f8 ? 0 : N * H * 2);  // an FP8 context moves quantised rows (xq) instead
  b.act = take(N * I * 2);
  b.y_perm = take(N * H * 2);
  b.act_shared = take(T * Is * 2);
  b.y_shared = take(c.n_shared ? T * H * 2 : 0);
  b.counts = reinterpret_cast<int32_t*>(take(E * 4));
  b.offsets = reinterpret_cast<int32_t*>(take((E + 1) * 4));
  b.perm = reinterpret_cast<int32_t*>(take(N * 4));
  b.inv_perm = reinterpret_cast<int32_t*>(take(N * 4));
  b.topk_idx = reinterpret_cast<int32_t*>(take(N * 4));
  b.topk_w = reinterpret_cast<float*>(take(N * 4));
  b.logits = reinterpret_cast<float*>(take(T * E * 4));
  b.x_stage = take(T * H * 2);
  b.out_stage = take(T * H * 2);
  b.scan = reinterpret_cast<int32_t*>(take(moe::layout_scratch_ints((int64_t)N, (int)E) * 4));
  b.xq = take(f8 * N * H);
  b.sx = reinterpret_cast<float*>(take(f8 * N * 4));
  b.aq = take(f8 * N * I);
  b.sa = reinterpret_cast<float*>(take(f8 * N * 4));
  b.xq_tok = take(f8 * T * H);
  b.sx_tok = reinterpret_cast<float*>(take(f8 * T * 4));
  b.aq_shared = take(f8 * T * Is);
  b.sa_shared = reinterpret_cast<float*>(take(f8 * (c.n_shared ? T * 4 : 0)));
  if (out) *out = b;
  return off;
}

// One more staging slot of the pipelined host path (the first slots are the staging buffers of the context's
// buffer sets); with base == nullptr it only measures.
size_t carve_staging(const moe_config& c, char* base, BufferSet* out) {
  const size_t T = (size_t)c.max_tokens, H = (size_t)c.hidden, E = (size_t)c.n_experts;
  const size_t a = align_up(T * E * 4, 256), b = align_up(T * H * 2, 256);
  if (base && out) {
    out->logits = reinterpret_cast<float*>(base);
    out->x_stage = base + a;
    out->out_stage = base + a + b;
  }
  return a + 2 * b;
}

const char* validate_config(const moe_config* c) {
  if (!c) return "config is NULL";
  if (c->hidden <= 0 || c->hidden % 64) return "hidden must be a positive multiple of 64";
  if (c->inter <= 0 || c->inter % 64) return "inter must be a positive multiple of 64";
  if (c->n_experts < 1 || c->n_experts > 1024) return "n_experts must be in 1..1024";
  if (c->top_k < 1 || c->top_k > 32 || c->top_k > c->n_experts) return "top_k must be in 1..min(n_experts,32)";
  if (c->n_shared < 0 || c->n_shared > 1) return "n_shared must be 0 or 1";
  if (c->n_shared && (c->shared_inter <= 0 || c->shared_inter % 64)) return "shared_inter must be a positive multiple of 64";
  if (c->max_tokens < 1) return "max_tokens must be >= 1";
  if ((int64_t)c->max_tokens * c->top_k > (int64_t)1 << 30) return "max_tokens * top_k too large";
  if (c->phase != MOE_PHASE_PREFILL && c->phase != MOE_PHASE_DECODE) return "phase must be MOE_PHASE_PREFILL or MOE_PHASE_DECODE";
  if (c->sm_budget < 0) return "sm_budget must be >= 0";
  if (c->gemm_variant < MOE_GEMM_AUTO || c->gemm_variant > MOE_GEMM_VALIDATION) return "unknown gemm_variant";
  if (c->row_gather != 0 && c->row_gather != 1) return "row_gather must be 0 or 1";
  if (!(c->routed_scale == c->routed_scale)) return "routed_scale is NaN";
  if (c->weight_format != MOE_WEIGHTS_BF16 && c->weight_format != MOE_WEIGHTS_FP8_E4M3) return "unknown weight_format";
  if (c->weight_format == MOE_WEIGHTS_FP8_E4M3) {
    if (c->hidden > 8192 || c->inter > 8192 || (c->n_shared && c->shared_inter > 8192))
      return "FP8 weights: hidden, inter and shared_inter may not exceed 8192";
    if (c->gemm_variant == MOE_GEMM_VALIDATION) return "FP8 weights need a tensor-core gemm_variant";
    if (c->row_gather) return "the row gather does not apply to FP8 weights";
  }
  return nullptr;
}

Layout measure(const moe_config& c) {
  Layout l;
  l.n_sets = (c.phase == MOE_PHASE_DECODE) ? 2 : 1;
  l.set_bytes = carve_set(c, nullptr, nullptr);
  l.total_bytes = kStatusBlock + l.set_bytes * (size_t)l.n_sets +
                  (size_t)(MOE_HOST_SLOTS - l.n_sets) * carve_staging(c, nullptr, nullptr);
  return l;
}

thread_local char g_create_error[256] = "";

}  // namespace

struct moe_ctx {
  moe_config cfg;
  cudaStream_t stream;
  char* ws;
  size_t ws_bytes;
  int device;
  int n_sms;
  int* status;  // device status word (first int of the status block)
  BufferSet sets[2];
  int n_sets;
  int cur;  // double-buffer index (always 0 for a PREFILL context)
  StepState state;
  int T;  // tokens of the step in progress
  // arrays of the step in progress (the caller's or the context's own)
  int32_t* counts;
  int32_t* offsets;
  int32_t* perm;
  int32_t* inv_perm;
  cudaEvent_t done;  // recorded after the last enqueue of every call
  int64_t launches;
  // pending-dispatch record of a split dispatch: what the second half needs (the arrays above, T) and the
  // stream position of the first half; at most one per context
  bool pending_dispatch;
  cudaEvent_t notified;
  bool split_step;   // the step in progress went through the split entry points (boundary numbering)
  unsigned gemm_seq = 0;  // GEMM launches so far: selects the tile-counter pair of the next one
  // prefill segmentation (off by default)
  int seg_experts;
  moe_boundary_fn boundary_fn;
  void* boundary_user;
  // per-stage timing (off by default): event pairs recorded around each stage's launches
  bool profiling;
  struct Span { cudaEvent_t beg, end; int stage; };
  std::vector<Span> spans;
  size_t spans_used;
  // pipelined host path: staging slots and two copy streams (created by the first moe_layer_host_submit)
  struct HostSlot {
    float* logits;
    char* x;
    char* out;
    cudaEvent_t h2d, comp, done;
    bool in_flight;
  } slots[MOE_HOST_SLOTS];
  cudaStream_t h2d_stream, d2h_stream;
  bool host_pipeline;
  // preemption of prefill GEMM passes at tile granularity (off by default)
  bool preemptible;
  int* yield_src;     // pinned host words {0, 1}: the sources of the copies that lower / raise the request
  int* yield_dev;     // the request word in the status block
  cudaStream_t yield_stream;  // private stream of those copies (any host thread may raise a request)
  std::mutex* yield_mu;
  int* stopped_host;  // pinned host word: CTAs that stopped in the last launch
  int64_t yields;     // launches that ended on a yield request
  unsigned long long wait_limit_ns;  // time limit of every bounded device-side wait (0 = the kernels' default)
  bool debug_stall;                  // failure-detection hook: the GEMM producers issue no copies
  char err[256];
};

namespace {

std::mutex g_registry_mutex;
std::vector<moe_ctx*> g_registry;

moe_status fail(moe_ctx* ctx, moe_status st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(ctx ? ctx->err : g_create_error, 256, fmt, ap);
  va_end(ap);
  return st;
}

moe_status cuda_fail(moe_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, e == cudaErrorNotSupported ? MOE_ERR_UNSUPPORTED : MOE_ERR_CUDA, "%s: %s", what,
              cudaGetErrorString(e));
}

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    cudaGetDevice(&prev);
    if (prev != dev) cudaSetDevice(dev);
    else prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

bool capturing(const moe_ctx* ctx) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(ctx->stream, &st) != cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  return st != cudaStreamCaptureStatusNone;
}

// After the last enqueue of a call: count the launches and mark the stream position.  While the stream is
// being captured into a CUDA graph nothing executes, so there is no position to mark (and an event recorded
// during capture could not be queried later).
void mark(moe_ctx* ctx, int n) {
  ctx->launches += n;
  if (!capturing(ctx)) cudaEventRecord(ctx->done, ctx->stream);
}

// Brackets the launches of one stage with events when profiling is on.
struct StageTimer {
  moe_ctx* ctx;
  moe_ctx::Span* span = nullptr;
  StageTimer(moe_ctx* c, int stage) : ctx(c) {
    if (!c->profiling || capturing(c)) return;  // event timing is meaningless inside a capture
    if (c->spans_used == c->spans.size()) {
      moe_ctx::Span s;
      if (cudaEventCreate(&s.beg) != cudaSuccess) return;
      if (cudaEventCreate(&s.end) != cudaSuccess) {
        cudaEventDestroy(s.beg);
        return;
      }
      c->spans.push_back(s);
    }
    span = &c->spans[c->spans_used++];
    span->stage = stage;
    cudaEventRecord(span->beg, c->stream);
  }
  ~StageTimer() {
    if (span) cudaEventRecord(span->end, ctx->stream);
  }
};

int gemm_ctas(const moe_ctx* ctx) {
  return (ctx->cfg.sm_budget > 0 && ctx->cfg.sm_budget < ctx->n_sms) ? ctx->cfg.sm_budget : ctx->n_sms;
}

// The choice between the two tensor-core variants for a PREFILL context, per pass, from the rows per expert
// R = rows / experts and the pass's K.  Measured on a B200 with the variants interleaved in long blocks
// (DeepSeek-V3- and Qwen3-30B-shaped layers, uniform and Zipf routing, whole steps and per-pass stage times):
//  * with tiles of up to 256 tokens the small-M kernel moves fewer bytes through shared memory per flop than the
//    large-M kernel (one CTA's MMA operands come from shared memory, whose bandwidth both end up waiting for), but
//    its tiles of more than 128 tokens fill tensor memory, so their epilogue is exposed: the longer K is, the less
//    that weighs;
//  * gated pass: K = 7168 -- small-M ahead by 4-13 % at every R up to 1024; K = 2048 -- level or ahead from R = 448
//    to 1024, behind by 3-10 % below that;
//  * down pass: K = 2048 -- small-M ahead up to R ~ 320 and 10-17 % behind above; K = 768 (12 k-blocks per tile: an
//    exposed epilogue is a quarter of a tile) -- behind by 9-25 % at every R;
//  * problems of up to 8192 rows, whose launches overlap with their neighbours, are 1.5-6 % faster on the small-M
//    kernel at any shape: it builds its tile list and fetches weights before the previous kernel has finished;
//  * FP8 (half the operand bytes per flop, so the issue cost of two MMAs per 16 K-elements shows): small-M up to
//    R = 256 (gated, K >= 4096) and 128 (down, K >= 1536); with shorter K (half as many k-blocks per tile as bf16)
//    large-M is 8-10 % ahead above the launch-overlap regime.
constexpr int64_t kSmallMRowsGated = 1024, kSmallMRowsGatedShortKFrom = 448, kSmallMRowsDown = 320;
constexpr int64_t kSmallMRowsFp8Gated = 256, kSmallMRowsFp8Down = 128;
constexpr int kLongK = 4096, kShortDownK = 1536;

// AUTO: a DECODE context always streams; a PREFILL context chooses per launch from the problem's rows (T * top_k
// rows over n_experts; T rows over one group for the shared expert by itself) and K: the choice is a function of T
// alone, so it is the same on every replay of a graph.
int gemm_variant_of(const moe_ctx* ctx, const moe::GemmProblem& p) {
  const int v = ctx->cfg.gemm_variant;
  if (v != MOE_GEMM_AUTO) return v;
  if (ctx->cfg.phase == MOE_PHASE_DECODE) return MOE_GEMM_SMALL_M;
  if (ctx->cfg.row_gather == 1) return MOE_GEMM_LARGE_M;  // only the large-M kernel gathers its rows itself
  if (ctx->preemptible) return MOE_GEMM_SMALL_M;          // only the small-M kernel can stop between tiles
  const int64_t E = p.E;  // 1 for a dense problem
  bool small;
  if (p.rows_bound <= moe::kGemmOverlapMaxRows) {
    small = true;
  } else if (p.fp8) {
    small = p.K >= (p.gated ? kLongK : kShortDownK) && p.rows_bound <= (p.gated ? kSmallMRowsFp8Gated : kSmallMRowsFp8Down) * E;
  } else if (p.gated) {
    small = p.rows_bound <= kSmallMRowsGated * E && (p.K >= kLongK || p.rows_bound >= kSmallMRowsGatedShortKFrom * E);
  } else {
    small = p.K >= kShortDownK && p.rows_bound <= kSmallMRowsDown * E;
  }
  return small ? MOE_GEMM_SMALL_M : MOE_GEMM_LARGE_M;
}

// GEMM1 gathers its rows itself only on the large-M tensor-core variant.
bool gathers_rows(const moe_ctx* ctx) {
  const int v = ctx->cfg.gemm_variant;
  return ctx->cfg.row_gather == 1 &&
         (v == MOE_GEMM_LARGE_M || (v == MOE_GEMM_AUTO && ctx->cfg.phase == MOE_PHASE_PREFILL));
}

// `dense` (the shared expert's pass, or nullptr) rides in the same launch on the tensor-core path.
cudaError_t run_gemm(moe_ctx* ctx, moe::GemmProblem p, const moe::GemmDenseGroup* dense, int T, int* n) {
  const int variant = gemm_variant_of(ctx, p);
  p.wait_limit_ns = ctx->wait_limit_ns;
  p.debug_stall = ctx->debug_stall;
  // Every GEMM launch comes after the step's row movement (or after another GEMM launch or a quantisation of the
  // same step), which in turn waited for the layout kernels: the offsets are older than the previous kernel.
  p.offsets_settled = true;
  p.tile_counters = reinterpret_cast<int*>(ctx->ws + kTileCounterOffset) + 2 * (ctx->gemm_seq++ % kTileCounterPairs);
  p.max_group_rows = T;
  if (variant == MOE_GEMM_VALIDATION) {
    cudaError_t e = moe::launch_gemm_validation(p, ctx->stream, n);
    if (e == cudaSuccess && dense != nullptr) {
      moe::GemmProblem d{dense->A, dense->W, dense->out, nullptr, dense->rows, dense->rows, dense->rows, 1,
                         dense->n_feat, dense->K, p.gated};
      e = moe::launch_gemm_validation(d, ctx->stream, n);
    }
    return e;
  }
  if (variant == MOE_GEMM_SMALL_M && ctx->preemptible && !capturing(ctx)) {
    // A pass that can be asked to stop between tiles: launch, wait on the host for the launch to end, and if
    // CTAs stopped on a yield request report the boundary and launch again with the same tile counter, which
    // goes on with the tiles not yet taken.
    int* stopped = ctx->status + 1;
    p.stopped = stopped;
    p.resumable = true;
    cudaError_t e = cudaMemsetAsync(p.tile_counters, 0, 2 * sizeof(int), ctx->stream);  // (an abandoned pass may have left them)
    for (int attempt = 0; e == cudaSuccess; ++attempt) {
      // a request that is still up after the hook has returned is honoured once more, then overridden: the pass
      // must end even with a controller that never clears its request
      p.yield_req = attempt < 64 ? ctx->yield_dev : nullptr;
      e = cudaMemsetAsync(stopped, 0, sizeof(int), ctx->stream);
      if (e == cudaSuccess) e = moe::launch_gemm_stream(p, dense, gemm_ctas(ctx), ctx->status, ctx->stream, n);
      if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stopped_host, stopped, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream);
      if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
      if (e != cudaSuccess || *ctx->stopped_host == 0) break;
      ++ctx->yields;
      if (ctx->boundary_fn) ctx->boundary_fn(ctx->boundary_user, MOE_BOUNDARY_YIELD, 0);
    }
    return e;
  }
  if (variant == MOE_GEMM_SMALL_M) return moe::launch_gemm_stream(p, dense, gemm_ctas(ctx), ctx->status, ctx->stream, n);
  return moe::launch_gemm_tc(p, dense, gemm_ctas(ctx), ctx->status, ctx->stream, n);
}

}  // namespace

namespace moe {

cudaError_t ensure_dynamic_smem_impl(const void* kern, size_t bytes) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, size_t> configured;  // (kernel, device) -> largest size set
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  std::lock_guard<std::mutex> lock(mu);
  size_t& have = configured[{kern, dev}];
  if (bytes <= have) return cudaSuccess;
  if (bytes > 48 * 1024) {
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (err != cudaSuccess) return err;
  }
  have = bytes;
  return cudaSuccess;
}

}  // namespace moe

extern "C" {

const char* moe_version(void) { return "moe_pd 0.1 (sm_100a)"; }

size_t moe_ctx_workspace_bytes(const moe_config* cfg) {
  if (validate_config(cfg)) return 0;
  return measure(*cfg).total_bytes;
}

moe_status moe_ctx_create(const moe_config* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream,
                          moe_ctx** out) {
  if (!out) return fail(nullptr, MOE_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (const char* why = validate_config(cfg)) return fail(nullptr, MOE_ERR_INVALID_ARG, "%s", why);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return fail(nullptr, MOE_ERR_INVALID_ARG, "workspace must be a 256-byte aligned device pointer");
  const Layout l = measure(*cfg);
  if (workspace_bytes < l.total_bytes)
    return fail(nullptr, MOE_ERR_CAPACITY, "workspace has %zu bytes, %zu needed", workspace_bytes, l.total_bytes);

  cudaPointerAttributes attr;
  cudaError_t e = cudaPointerGetAttributes(&attr, workspace);
  if (e != cudaSuccess || attr.type != cudaMemoryTypeDevice) {
    (void)cudaGetLastError();
    return fail(nullptr, MOE_ERR_INVALID_ARG, "workspace is not device memory");
  }
  const char* why = nullptr;
  if (cfg->gemm_variant != MOE_GEMM_VALIDATION && !moe::gemm_tc_init(&why))
    return fail(nullptr, MOE_ERR_UNSUPPORTED, "%s", why ? why : "tensor-map encoding unavailable");

  moe_ctx* ctx = new (std::nothrow) moe_ctx();
  if (!ctx) return fail(nullptr, MOE_ERR_CUDA, "host allocation failed");
  ctx->cfg = *cfg;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->ws = static_cast<char*>(workspace);
  ctx->ws_bytes = l.total_bytes;
  ctx->device = attr.device;
  ctx->n_sets = l.n_sets;
  ctx->cur = 0;
  ctx->state = ST_IDLE;
  ctx->T = 0;
  ctx->launches = 0;
  ctx->pending_dispatch = false;
  ctx->split_step = false;
  ctx->profiling = false;
  ctx->spans_used = 0;
  ctx->seg_experts = 0;
  ctx->boundary_fn = nullptr;
  ctx->boundary_user = nullptr;
  ctx->err[0] = 0;
  ctx->status = reinterpret_cast<int*>(ctx->ws);
  for (int s = 0; s < l.n_sets; ++s) carve_set(*cfg, ctx->ws + kStatusBlock + (size_t)s * l.set_bytes, &ctx->sets[s]);
  ctx->host_pipeline = false;
  ctx->wait_limit_ns = 0;
  ctx->debug_stall = false;
  ctx->preemptible = false;
  ctx->yield_src = ctx->yield_dev = ctx->stopped_host = nullptr;
  ctx->yield_stream = nullptr;
  ctx->yield_mu = nullptr;
  ctx->yields = 0;
  const size_t staging_bytes = carve_staging(*cfg, nullptr, nullptr);
  for (int s = 0; s < MOE_HOST_SLOTS; ++s) {
    BufferSet st = ctx->sets[s < l.n_sets ? s : 0];
    if (s >= l.n_sets)
      carve_staging(*cfg, ctx->ws + kStatusBlock + l.set_bytes * (size_t)l.n_sets + (size_t)(s - l.n_sets) * staging_bytes,
                    &st);
    ctx->slots[s].logits = st.logits;
    ctx->slots[s].x = st.x_stage;
    ctx->slots[s].out = st.out_stage;
    ctx->slots[s].in_flight = false;
  }

  {
    // Isolation is validated at construction: no two live contexts may share a mutable byte, and a
    // stream serves contexts of one phase only.
    std::lock_guard<std::mutex> lock(g_registry_mutex);
    for (const moe_ctx* o : g_registry) {
      if (o->device == ctx->device && ctx->ws < o->ws + o->ws_bytes && o->ws < ctx->ws + ctx->ws_bytes) {
        delete ctx;
        return fail(nullptr, MOE_ERR_STATE, "workspace overlaps the workspace of a live context");
      }
      if (o->device == ctx->device && o->stream == ctx->stream && o->cfg.phase != ctx->cfg.phase) {
        delete ctx;
        return fail(nullptr, MOE_ERR_STATE, "stream is already bound to a live context of the other phase");
      }
    }
    g_registry.push_back(ctx);
  }

  DeviceGuard guard(ctx->device);
  int sms = 0;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->done, cudaEventDisableTiming);
  if (e == cudaSuccess) {
    e = cudaEventCreateWithFlags(&ctx->notified, cudaEventDisableTiming);
    if (e != cudaSuccess) cudaEventDestroy(ctx->done);
  }
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->ws, 0, kStatusBlock, ctx->stream);
  if (e == cudaSuccess) e = cudaEventRecord(ctx->done, ctx->stream);
  if (e != cudaSuccess) {
    std::lock_guard<std::mutex> lock(g_registry_mutex);
    for (size_t i = 0; i < g_registry.size(); ++i)
      if (g_registry[i] == ctx) {
        g_registry.erase(g_registry.begin() + i);
        break;
      }
    moe_status st = cuda_fail(nullptr, e, "context set-up");
    delete ctx;
    return st;
  }
  ctx->n_sms = sms;
  *out = ctx;
  return MOE_OK;
}

moe_status moe_ctx_destroy(moe_ctx* ctx) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaError_t q = cudaEventQuery(ctx->done);
  if (q == cudaErrorNotReady) return fail(ctx, MOE_ERR_STATE, "work is still in flight on the context's stream");
  if (q != cudaSuccess) (void)cudaGetLastError();
  for (int s = 0; s < MOE_HOST_SLOTS; ++s)
    if (ctx->slots[s].in_flight && cudaEventQuery(ctx->slots[s].done) == cudaErrorNotReady)
      return fail(ctx, MOE_ERR_STATE, "a moe_layer_host_submit slot is still in flight");
  (void)cudaGetLastError();
  if (ctx->host_pipeline) {
    for (int s = 0; s < MOE_HOST_SLOTS; ++s) {
      cudaEventDestroy(ctx->slots[s].h2d);
      cudaEventDestroy(ctx->slots[s].comp);
      cudaEventDestroy(ctx->slots[s].done);
    }
    cudaStreamDestroy(ctx->h2d_stream);
    cudaStreamDestroy(ctx->d2h_stream);
  }
  {
    std::lock_guard<std::mutex> lock(g_registry_mutex);
    for (size_t i = 0; i < g_registry.size(); ++i)
      if (g_registry[i] == ctx) {
        g_registry.erase(g_registry.begin() + i);
        break;
      }
  }
  cudaEventDestroy(ctx->done);
  cudaEventDestroy(ctx->notified);
  if (ctx->yield_src) cudaFreeHost(ctx->yield_src);
  if (ctx->stopped_host) cudaFreeHost(ctx->stopped_host);
  if (ctx->yield_stream) cudaStreamDestroy(ctx->yield_stream);
  delete ctx->yield_mu;
  for (auto& sp : ctx->spans) {
    cudaEventDestroy(sp.beg);
    cudaEventDestroy(sp.end);
  }
  delete ctx;
  return MOE_OK;
}

moe_status moe_ctx_abandon_step(moe_ctx* ctx) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state == ST_IDLE) return MOE_OK;
  ctx->state = ST_IDLE;
  ctx->T = 0;
  ctx->pending_dispatch = false;  // a pending dispatch is retired with the step
  ctx->split_step = false;
  if (ctx->n_sets == 2) ctx->cur ^= 1;  // D: the abandoned step's buffer set rests for one whole step
  return MOE_OK;
}

moe_status moe_ctx_status(moe_ctx* ctx, int32_t* device_status) {
  if (!ctx || !device_status) return MOE_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  int32_t v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, ctx->status, sizeof v, cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status, 0, sizeof(int), ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_ctx_status");
  *device_status = v;
  return MOE_OK;
}

const char* moe_last_error(const moe_ctx* ctx) { return ctx ? ctx->err : g_create_error; }

int64_t moe_ctx_launch_count(const moe_ctx* ctx) { return ctx ? ctx->launches : 0; }

moe_status moe_route(moe_ctx* ctx, const float* logits, const float* select_bias, int32_t T, int32_t* topk_idx,
                     float* topk_w) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state != ST_IDLE && ctx->state != ST_ROUTED)
    return fail(ctx, MOE_ERR_STATE, "moe_route called in the middle of a step");
  if (T < 0) return fail(ctx, MOE_ERR_INVALID_ARG, "T < 0");
  if (T > ctx->cfg.max_tokens) return fail(ctx, MOE_ERR_CAPACITY, "T = %d exceeds max_tokens = %d", T, ctx->cfg.max_tokens);
  if (T > 0 && (!logits || !topk_idx || !topk_w)) return fail(ctx, MOE_ERR_INVALID_ARG, "NULL pointer");
  if (misaligned(logits) || misaligned(select_bias) || misaligned(topk_idx) || misaligned(topk_w))
    return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  DeviceGuard guard(ctx->device);
  int n = 0;
  cudaError_t e;
  {
    StageTimer tm(ctx, 0);
    e = moe::launch_route(logits, select_bias, T, ctx->cfg.n_experts, ctx->cfg.top_k, ctx->cfg.routed_scale, topk_idx,
                          topk_w, ctx->stream, &n);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_route");
  ctx->state = ST_ROUTED;
  mark(ctx, n);
  return MOE_OK;
}

}  // extern "C"

namespace {

// First half of a dispatch: counts, exclusive scan, stable permutation (no rows move).
moe_status enqueue_layout(moe_ctx* ctx, const char* who, const int32_t* topk_idx, int32_t T, int32_t* counts,
                          int32_t* offsets, int32_t* perm, int32_t* inv_perm) {
  if (T < 0) return fail(ctx, MOE_ERR_INVALID_ARG, "T < 0");
  if (T > ctx->cfg.max_tokens) return fail(ctx, MOE_ERR_CAPACITY, "T = %d exceeds max_tokens = %d", T, ctx->cfg.max_tokens);
  if (T > 0 && !topk_idx) return fail(ctx, MOE_ERR_INVALID_ARG, "topk_idx is NULL");
  if (misaligned(topk_idx) || misaligned(counts) || misaligned(offsets) || misaligned(perm) || misaligned(inv_perm))
    return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  BufferSet& b = ctx->sets[ctx->cur];
  ctx->counts = counts ? counts : b.counts;
  ctx->offsets = offsets ? offsets : b.offsets;
  ctx->perm = perm ? perm : b.perm;
  ctx->inv_perm = inv_perm ? inv_perm : b.inv_perm;
  int n = 0;
  cudaError_t e;
  {
    StageTimer tm(ctx, 1);
    e = moe::launch_layout(topk_idx, (int64_t)T * ctx->cfg.top_k, ctx->cfg.n_experts, ctx->counts, ctx->offsets,
                           ctx->perm, ctx->inv_perm, b.scan, ctx->status, ctx->stream, &n);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, who);
  ctx->T = T;
  ctx->launches += n;
  return MOE_OK;
}

// Second half: the routed data movement (an FP8 context quantises each token row once and moves the codes).
moe_status enqueue_row_movement(moe_ctx* ctx, const char* who, const void* x) {
  BufferSet& b = ctx->sets[ctx->cur];
  const int32_t T = ctx->T;
  const bool fp8 = ctx->cfg.weight_format == MOE_WEIGHTS_FP8_E4M3;
  int n = 0;
  cudaError_t e = cudaSuccess;
  if (T > 0 && fp8) {
    {
      StageTimer tm(ctx, 8);
      e = moe::launch_quantize_rows(x, T, ctx->cfg.hidden, b.xq_tok, b.sx_tok, ctx->stream, &n);
    }
    if (e == cudaSuccess) {
      StageTimer tm(ctx, 2);
      e = moe::launch_permute(b.xq_tok, ctx->inv_perm, b.xq, T, ctx->cfg.top_k, ctx->cfg.hidden / 2, ctx->status,
                              ctx->stream, &n, b.sx_tok, b.sx, ctx->wait_limit_ns);
    }
  } else if (T > 0 && !gathers_rows(ctx)) {
    StageTimer tm(ctx, 2);
    e = moe::launch_permute(x, ctx->inv_perm, b.x_perm, T, ctx->cfg.top_k, ctx->cfg.hidden, ctx->status, ctx->stream,
                            &n, nullptr, nullptr, ctx->wait_limit_ns);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, who);
  ctx->launches += n;
  return MOE_OK;
}

// Boundaries moe_grouped_ffn / moe_grouped_ffn_fp8 report with the current segmentation.
int ffn_boundaries(const moe_ctx* ctx) {
  const moe_config& c = ctx->cfg;
  const bool shared = c.n_shared != 0;
  const int span = (ctx->seg_experts > 0 && ctx->seg_experts < c.n_experts) ? ctx->seg_experts : c.n_experts;
  const int routed_segs = (c.n_experts + span - 1) / span;
  const bool fuse_shared = shared && ctx->seg_experts == 0;
  if (c.weight_format == MOE_WEIGHTS_FP8_E4M3) return 2 * routed_segs + 1 + ((shared && !fuse_shared) ? 2 : 0);
  return 2 * routed_segs + (shared ? 2 : 0);
}

}  // namespace

extern "C" {

moe_status moe_dispatch_layout(moe_ctx* ctx, const int32_t* topk_idx, int32_t T, const void* x, int32_t* counts,
                               int32_t* offsets, int32_t* perm, int32_t* inv_perm) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state == ST_NOTIFIED)
    return fail(ctx, MOE_ERR_STATE, "a dispatch is pending on this context: move its rows or abandon the step");
  if (ctx->state != ST_IDLE && ctx->state != ST_ROUTED && ctx->state != ST_LAYOUT_ONLY)
    return fail(ctx, MOE_ERR_STATE, "moe_dispatch_layout called in the middle of a step");
  if (misaligned(x)) return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  DeviceGuard guard(ctx->device);
  moe_status st = enqueue_layout(ctx, "moe_dispatch_layout", topk_idx, T, counts, offsets, perm, inv_perm);
  if (st == MOE_OK && x != nullptr) st = enqueue_row_movement(ctx, "moe_dispatch_layout", x);
  if (st != MOE_OK) return st;
  ctx->state = (x != nullptr || T == 0) ? ST_LAID_OUT : ST_LAYOUT_ONLY;  // an empty batch has no rows to move
  ctx->split_step = false;
  mark(ctx, 0);
  return MOE_OK;
}

moe_status moe_dispatch_notify(moe_ctx* ctx, const int32_t* topk_idx, int32_t T, int32_t* counts, int32_t* offsets,
                               int32_t* perm, int32_t* inv_perm) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->pending_dispatch || ctx->state == ST_NOTIFIED)
    return fail(ctx, MOE_ERR_STATE, "a dispatch is already pending on this context (at most one per context)");
  if (ctx->state != ST_IDLE && ctx->state != ST_ROUTED)
    return fail(ctx, MOE_ERR_STATE, "moe_dispatch_notify called in the middle of a step");
  DeviceGuard guard(ctx->device);
  moe_status st = enqueue_layout(ctx, "moe_dispatch_notify", topk_idx, T, counts, offsets, perm, inv_perm);
  if (st != MOE_OK) return st;
  ctx->state = ST_NOTIFIED;
  ctx->pending_dispatch = true;
  ctx->split_step = true;
  mark(ctx, 0);
  if (!capturing(ctx)) cudaEventRecord(ctx->notified, ctx->stream);  // the record's stream position
  // boundary 0 of a segmented step: after notification, before any row moves
  if (ctx->seg_experts > 0 && ctx->boundary_fn) ctx->boundary_fn(ctx->boundary_user, 0, 1 + ffn_boundaries(ctx));
  return MOE_OK;
}

moe_status moe_dispatch_move(moe_ctx* ctx, const void* x) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state != ST_NOTIFIED || !ctx->pending_dispatch)
    return fail(ctx, MOE_ERR_STATE, "moe_dispatch_move needs a pending dispatch (moe_dispatch_notify) on this context");
  if (ctx->T > 0 && !x) return fail(ctx, MOE_ERR_INVALID_ARG, "x is NULL");
  if (misaligned(x)) return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  DeviceGuard guard(ctx->device);
  moe_status st = enqueue_row_movement(ctx, "moe_dispatch_move", x);
  if (st != MOE_OK) return st;  // the dispatch stays pending: retry, or abandon the step
  ctx->state = ST_LAID_OUT;
  ctx->pending_dispatch = false;
  mark(ctx, 0);
  return MOE_OK;
}

moe_status moe_ctx_pending_dispatch(moe_ctx* ctx, int32_t* pending, int32_t* tokens, int32_t* notified_done) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (pending) *pending = ctx->pending_dispatch ? 1 : 0;
  if (tokens) *tokens = ctx->pending_dispatch ? ctx->T : 0;
  if (notified_done) {
    *notified_done = 0;
    if (ctx->pending_dispatch) {
      DeviceGuard guard(ctx->device);
      const cudaError_t q = cudaEventQuery(ctx->notified);
      if (q == cudaSuccess) *notified_done = 1;
      else (void)cudaGetLastError();
    }
  }
  return MOE_OK;
}

moe_status moe_grouped_ffn(moe_ctx* ctx, const void* w_gate_up, const void* w_down, const void* x,
                           const void* ws_gate_up, const void* ws_down, int32_t T) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->cfg.weight_format != MOE_WEIGHTS_BF16)
    return fail(ctx, MOE_ERR_STATE, "the context was created for FP8 weights: call moe_grouped_ffn_fp8");
  if (ctx->state != ST_LAID_OUT)
    return fail(ctx, MOE_ERR_STATE, "moe_grouped_ffn needs a moe_dispatch_layout with x in the same step");
  if (T != ctx->T) return fail(ctx, MOE_ERR_INVALID_ARG, "T = %d differs from the layout's T = %d", T, ctx->T);
  if (!w_gate_up || !w_down) return fail(ctx, MOE_ERR_INVALID_ARG, "routed weights are NULL");
  const bool shared = ctx->cfg.n_shared != 0;
  if (shared && (!ws_gate_up || !ws_down || (!x && T > 0)))
    return fail(ctx, MOE_ERR_INVALID_ARG, "the shared expert needs ws_gate_up, ws_down and x");
  if (gathers_rows(ctx) && !x && T > 0) return fail(ctx, MOE_ERR_INVALID_ARG, "the row gather needs x");
  if (misaligned(w_gate_up) || misaligned(w_down) || misaligned(x) || misaligned(ws_gate_up) || misaligned(ws_down))
    return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  DeviceGuard guard(ctx->device);
  BufferSet& b = ctx->sets[ctx->cur];
  const moe_config& c = ctx->cfg;
  const int64_t N = (int64_t)T * c.top_k, Ncap = (int64_t)c.max_tokens * c.top_k;
  int n = 0;
  cudaError_t e = cudaSuccess;
  if (T > 0) {
    // One launch per pass, or one per group of seg_experts experts with a boundary call after each.
    const int span = (ctx->seg_experts > 0 && ctx->seg_experts < c.n_experts) ? ctx->seg_experts : c.n_experts;
    const int routed_segs = (c.n_experts + span - 1) / span;
    const int first = ctx->split_step ? 1 : 0;  // a split dispatch reported boundary 0 after its notification
    const int n_bound = first + 2 * routed_segs + (shared ? 2 : 0);
    int bound = first;
    auto boundary = [&]() {
      if (ctx->seg_experts > 0 && ctx->boundary_fn) {
        if (!capturing(ctx)) cudaEventRecord(ctx->done, ctx->stream);
        ctx->boundary_fn(ctx->boundary_user, bound, n_bound);
      }
      ++bound;
    };
    moe::GemmProblem g1{b.x_perm, w_gate_up, b.act, ctx->offsets, 0, Ncap, N, c.n_experts, c.inter, c.hidden, true};
    moe::GemmProblem g2{b.act, w_down, b.y_perm, ctx->offsets, 0, Ncap, N, c.n_experts, c.hidden, c.inter, false};
    if (gathers_rows(ctx)) {
      g1.gather_src = x;
      g1.perm = ctx->perm;
      g1.top_k = c.top_k;
    }
    moe::GemmDenseGroup s1{x, ws_gate_up, b.act_shared, T, c.shared_inter, c.hidden};
    moe::GemmDenseGroup s2{b.act_shared, ws_down, b.y_shared, T, c.hidden, c.shared_inter};
    // Unsegmented: the shared expert's two passes ride in the routed launches (two launches in all).
    // Segmented: they are segments of their own, after the routed ones.
    const bool fuse_shared = shared && ctx->seg_experts == 0;
    for (int pass = 0; pass < 2 && e == cudaSuccess; ++pass) {
      moe::GemmProblem& g = pass == 0 ? g1 : g2;
      for (int e0 = 0; e0 < c.n_experts && e == cudaSuccess; e0 += span) {
        g.e_begin = e0;
        g.e_end = e0 + span < c.n_experts ? e0 + span : c.n_experts;
        {
          StageTimer tm(ctx, pass == 0 ? 3 : 4);
          e = run_gemm(ctx, g, fuse_shared ? (pass == 0 ? &s1 : &s2) : nullptr, T, &n);
        }
        if (e == cudaSuccess) boundary();
      }
    }
    if (e == cudaSuccess && shared && !fuse_shared) {
      moe::GemmProblem d1{s1.A, s1.W, s1.out, nullptr, T, T, T, 1, s1.n_feat, s1.K, true};
      {
        StageTimer tm(ctx, 5);
        e = run_gemm(ctx, d1, nullptr, T, &n);
      }
      if (e == cudaSuccess) {
        boundary();
        moe::GemmProblem d2{s2.A, s2.W, s2.out, nullptr, T, T, T, 1, s2.n_feat, s2.K, false};
        {
          StageTimer tm(ctx, 6);
          e = run_gemm(ctx, d2, nullptr, T, &n);
        }
        if (e == cudaSuccess) boundary();
      }
    }
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_grouped_ffn");
  ctx->state = ST_FFN_DONE;
  mark(ctx, n);
  return MOE_OK;
}

moe_status moe_grouped_ffn_fp8(moe_ctx* ctx, const void* wq_gate_up, const float* sw_gate_up, const void* wq_down,
                               const float* sw_down, const void* wsq_gate_up, const float* sws_gate_up,
                               const void* wsq_down, const float* sws_down, int32_t T) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->cfg.weight_format != MOE_WEIGHTS_FP8_E4M3)
    return fail(ctx, MOE_ERR_STATE, "the context was not created with weight_format = MOE_WEIGHTS_FP8_E4M3");
  if (ctx->state != ST_LAID_OUT)
    return fail(ctx, MOE_ERR_STATE, "moe_grouped_ffn_fp8 needs a moe_dispatch_layout with x in the same step");
  if (T != ctx->T) return fail(ctx, MOE_ERR_INVALID_ARG, "T = %d differs from the layout's T = %d", T, ctx->T);
  if (!wq_gate_up || !sw_gate_up || !wq_down || !sw_down)
    return fail(ctx, MOE_ERR_INVALID_ARG, "routed weights or scales are NULL");
  const bool shared = ctx->cfg.n_shared != 0;
  if (shared && (!wsq_gate_up || !sws_gate_up || !wsq_down || !sws_down))
    return fail(ctx, MOE_ERR_INVALID_ARG, "the shared expert needs its weights and scales");
  if (misaligned(wq_gate_up) || misaligned(sw_gate_up) || misaligned(wq_down) || misaligned(sw_down) ||
      misaligned(wsq_gate_up) || misaligned(sws_gate_up) || misaligned(wsq_down) || misaligned(sws_down))
    return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  DeviceGuard guard(ctx->device);
  BufferSet& b = ctx->sets[ctx->cur];
  const moe_config& c = ctx->cfg;
  const int64_t N = (int64_t)T * c.top_k, Ncap = (int64_t)c.max_tokens * c.top_k;
  int n = 0;
  cudaError_t e = cudaSuccess;
  if (T > 0) {
    // GEMM1 + SwiGLU on the rows moe_dispatch_layout quantised -> quantise the activation -> GEMM2.
    // Unsegmented: the shared expert's passes ride in the routed launches.  Segmented (moe_ctx_set_segments): one
    // launch per group of experts and pass, the shared expert's passes and the activation's quantisation are
    // segments of their own, and the boundary hook runs after each.
    const int span = (ctx->seg_experts > 0 && ctx->seg_experts < c.n_experts) ? ctx->seg_experts : c.n_experts;
    const int routed_segs = (c.n_experts + span - 1) / span;
    const bool fuse_shared = shared && ctx->seg_experts == 0;
    const int first = ctx->split_step ? 1 : 0;
    const int n_bound = first + 2 * routed_segs + 1 + ((shared && !fuse_shared) ? 2 : 0);
    int bound = first;
    auto boundary = [&]() {
      if (ctx->seg_experts > 0 && ctx->boundary_fn) {
        if (!capturing(ctx)) cudaEventRecord(ctx->done, ctx->stream);
        ctx->boundary_fn(ctx->boundary_user, bound, n_bound);
      }
      ++bound;
    };
    moe::GemmProblem g1{b.xq, wq_gate_up, b.act, ctx->offsets, 0, Ncap, N, c.n_experts, c.inter, c.hidden, true};
    g1.fp8 = true;
    g1.row_scale = b.sx;
    g1.w_scale = sw_gate_up;
    moe::GemmProblem g2{b.aq, wq_down, b.y_perm, ctx->offsets, 0, Ncap, N, c.n_experts, c.hidden, c.inter, false};
    g2.fp8 = true;
    g2.row_scale = b.sa;
    g2.w_scale = sw_down;
    moe::GemmDenseGroup s1{b.xq_tok, wsq_gate_up, b.act_shared, T, c.shared_inter, c.hidden, b.sx_tok, sws_gate_up};
    moe::GemmDenseGroup s2{b.aq_shared, wsq_down, b.y_shared, T, c.hidden, c.shared_inter, b.sa_shared, sws_down};
    auto dense_problem = [&](const moe::GemmDenseGroup& d, bool gated) {
      moe::GemmProblem q{d.A, d.W, d.out, nullptr, T, T, T, 1, d.n_feat, d.K, gated};
      q.fp8 = true;
      q.row_scale = d.row_scale;
      q.w_scale = d.w_scale;
      return q;
    };
    for (int pass = 0; pass < 2 && e == cudaSuccess; ++pass) {
      moe::GemmProblem& g = pass == 0 ? g1 : g2;
      for (int e0 = 0; e0 < c.n_experts && e == cudaSuccess; e0 += span) {
        g.e_begin = e0;
        g.e_end = e0 + span < c.n_experts ? e0 + span : c.n_experts;
        {
          StageTimer tm(ctx, pass == 0 ? 3 : 4);
          e = run_gemm(ctx, g, fuse_shared ? (pass == 0 ? &s1 : &s2) : nullptr, T, &n);
        }
        if (e == cudaSuccess) boundary();
      }
      if (pass == 0 && e == cudaSuccess && shared && !fuse_shared) {
        moe::GemmProblem d1 = dense_problem(s1, true);
        {
          StageTimer tm(ctx, 5);
          e = run_gemm(ctx, d1, nullptr, T, &n);
        }
        if (e == cudaSuccess) boundary();
      }
      if (pass == 0 && e == cudaSuccess) {
        {
          StageTimer tm(ctx, 9);
          e = moe::launch_quantize_rows(b.act, N, c.inter, b.aq, b.sa, ctx->stream, &n);
          if (e == cudaSuccess && shared)
            e = moe::launch_quantize_rows(b.act_shared, T, c.shared_inter, b.aq_shared, b.sa_shared, ctx->stream, &n);
        }
        if (e == cudaSuccess) boundary();
      }
    }
    if (e == cudaSuccess && shared && !fuse_shared) {
      moe::GemmProblem d2 = dense_problem(s2, false);
      {
        StageTimer tm(ctx, 6);
        e = run_gemm(ctx, d2, nullptr, T, &n);
      }
      if (e == cudaSuccess) boundary();
    }
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_grouped_ffn_fp8");
  ctx->state = ST_FFN_DONE;
  mark(ctx, n);
  return MOE_OK;
}

moe_status moe_combine(moe_ctx* ctx, const float* topk_w, const int32_t* inv_perm, int32_t T, void* out) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state != ST_FFN_DONE) return fail(ctx, MOE_ERR_STATE, "moe_combine needs moe_grouped_ffn in the same step");
  if (T != ctx->T) return fail(ctx, MOE_ERR_INVALID_ARG, "T = %d differs from the layout's T = %d", T, ctx->T);
  if (T > 0 && (!topk_w || !out)) return fail(ctx, MOE_ERR_INVALID_ARG, "NULL pointer");
  if (misaligned(topk_w) || misaligned(inv_perm) || misaligned(out))
    return fail(ctx, MOE_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
  DeviceGuard guard(ctx->device);
  BufferSet& b = ctx->sets[ctx->cur];
  int n = 0;
  cudaError_t e;
  {
    StageTimer tm(ctx, 7);
    e = moe::launch_combine(b.y_perm, ctx->cfg.n_shared ? b.y_shared : nullptr, inv_perm ? inv_perm : ctx->inv_perm,
                            topk_w, out, T, ctx->cfg.top_k, ctx->cfg.hidden, ctx->status, ctx->stream, &n,
                            ctx->wait_limit_ns);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_combine");
  ctx->state = ST_IDLE;
  ctx->split_step = false;
  if (ctx->n_sets == 2) ctx->cur ^= 1;  // D: the next step works in the other buffer set
  mark(ctx, n);
  return MOE_OK;
}

moe_status moe_layer_host(moe_ctx* ctx, const float* logits_host, const float* select_bias, const void* x_host,
                          int32_t T, const void* w_gate_up, const void* w_down, const void* ws_gate_up,
                          const void* ws_down, void* out_host) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state != ST_IDLE) return fail(ctx, MOE_ERR_STATE, "moe_layer_host called in the middle of a step");
  if (T < 0) return fail(ctx, MOE_ERR_INVALID_ARG, "T < 0");
  if (T > ctx->cfg.max_tokens) return fail(ctx, MOE_ERR_CAPACITY, "T = %d exceeds max_tokens = %d", T, ctx->cfg.max_tokens);
  if (T > 0 && (!logits_host || !x_host || !out_host)) return fail(ctx, MOE_ERR_INVALID_ARG, "NULL host pointer");
  DeviceGuard guard(ctx->device);
  BufferSet& b = ctx->sets[ctx->cur];
  const moe_config& c = ctx->cfg;
  const size_t x_bytes = (size_t)T * c.hidden * 2;
  cudaError_t e = cudaSuccess;
  if (T > 0) {
    e = cudaMemcpyAsync(b.logits, logits_host, (size_t)T * c.n_experts * 4, cudaMemcpyHostToDevice, ctx->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.x_stage, x_host, x_bytes, cudaMemcpyHostToDevice, ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "host-to-device copy");
  }
  moe_status st = moe_route(ctx, b.logits, select_bias, T, b.topk_idx, b.topk_w);
  if (st == MOE_OK) st = moe_dispatch_layout(ctx, b.topk_idx, T, b.x_stage, nullptr, nullptr, nullptr, nullptr);
  if (st == MOE_OK) st = moe_grouped_ffn(ctx, w_gate_up, w_down, b.x_stage, ws_gate_up, ws_down, T);
  if (st == MOE_OK) st = moe_combine(ctx, b.topk_w, nullptr, T, b.out_stage);
  if (st != MOE_OK) {
    ctx->state = ST_IDLE;
    return st;
  }
  if (T > 0) e = cudaMemcpyAsync(out_host, b.out_stage, x_bytes, cudaMemcpyDeviceToHost, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "device-to-host copy");
  return MOE_OK;
}

moe_status moe_layer_host_submit(moe_ctx* ctx, int32_t slot, const float* logits_host, const float* select_bias,
                                 const void* x_host, int32_t T, const void* w_gate_up, const void* w_down,
                                 const void* ws_gate_up, const void* ws_down, void* out_host) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (slot < 0 || slot >= MOE_HOST_SLOTS) return fail(ctx, MOE_ERR_INVALID_ARG, "slot must be in [0, %d)", MOE_HOST_SLOTS);
  if (ctx->cfg.weight_format != MOE_WEIGHTS_BF16)
    return fail(ctx, MOE_ERR_STATE, "the host path serves contexts created for BF16 weights");
  if (ctx->state != ST_IDLE) return fail(ctx, MOE_ERR_STATE, "moe_layer_host_submit called in the middle of a step");
  if (ctx->slots[slot].in_flight) return fail(ctx, MOE_ERR_STATE, "slot %d has not been waited for", slot);
  if (T < 0) return fail(ctx, MOE_ERR_INVALID_ARG, "T < 0");
  if (T > ctx->cfg.max_tokens) return fail(ctx, MOE_ERR_CAPACITY, "T = %d exceeds max_tokens = %d", T, ctx->cfg.max_tokens);
  if (T > 0 && (!logits_host || !x_host || !out_host)) return fail(ctx, MOE_ERR_INVALID_ARG, "NULL host pointer");
  DeviceGuard guard(ctx->device);
  cudaError_t e = cudaSuccess;
  if (!ctx->host_pipeline) {
    constexpr int kEvents = 3 * MOE_HOST_SLOTS;
    cudaEvent_t ev[kEvents] = {};
    cudaStream_t st[2] = {};
    for (int i = 0; i < kEvents && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaStreamCreateWithFlags(&st[i], cudaStreamNonBlocking);
    if (e != cudaSuccess) {
      for (int i = 0; i < kEvents; ++i)
        if (ev[i]) cudaEventDestroy(ev[i]);
      for (int i = 0; i < 2; ++i)
        if (st[i]) cudaStreamDestroy(st[i]);
      return cuda_fail(ctx, e, "moe_layer_host_submit set-up");
    }
    for (int s = 0; s < MOE_HOST_SLOTS; ++s) {
      ctx->slots[s].h2d = ev[3 * s];
      ctx->slots[s].comp = ev[3 * s + 1];
      ctx->slots[s].done = ev[3 * s + 2];
    }
    ctx->h2d_stream = st[0];
    ctx->d2h_stream = st[1];
    ctx->host_pipeline = true;
  }
  moe_ctx::HostSlot& hs = ctx->slots[slot];
  BufferSet& b = ctx->sets[ctx->cur];
  const moe_config& c = ctx->cfg;
  const size_t x_bytes = (size_t)T * c.hidden * 2;
  if (T > 0) {
    e = cudaMemcpyAsync(hs.logits, logits_host, (size_t)T * c.n_experts * 4, cudaMemcpyHostToDevice, ctx->h2d_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(hs.x, x_host, x_bytes, cudaMemcpyHostToDevice, ctx->h2d_stream);
  }
  if (e == cudaSuccess) e = cudaEventRecord(hs.h2d, ctx->h2d_stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->stream, hs.h2d, 0);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "host-to-device copy");
  moe_status st = moe_route(ctx, hs.logits, select_bias, T, b.topk_idx, b.topk_w);
  if (st == MOE_OK) st = moe_dispatch_layout(ctx, b.topk_idx, T, hs.x, nullptr, nullptr, nullptr, nullptr);
  if (st == MOE_OK) st = moe_grouped_ffn(ctx, w_gate_up, w_down, hs.x, ws_gate_up, ws_down, T);
  if (st == MOE_OK) st = moe_combine(ctx, b.topk_w, nullptr, T, hs.out);
  if (st != MOE_OK) {
    ctx->state = ST_IDLE;
    return st;
  }
  e = cudaEventRecord(hs.comp, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->d2h_stream, hs.comp, 0);
  if (e == cudaSuccess && T > 0) e = cudaMemcpyAsync(out_host, hs.out, x_bytes, cudaMemcpyDeviceToHost, ctx->d2h_stream);
  if (e == cudaSuccess) e = cudaEventRecord(hs.done, ctx->d2h_stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "device-to-host copy");
  hs.in_flight = true;
  return MOE_OK;
}

moe_status moe_layer_host_wait(moe_ctx* ctx, int32_t slot) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (slot < 0 || slot >= MOE_HOST_SLOTS) return fail(ctx, MOE_ERR_INVALID_ARG, "slot must be in [0, %d)", MOE_HOST_SLOTS);
  if (!ctx->slots[slot].in_flight) return MOE_OK;
  DeviceGuard guard(ctx->device);
  cudaError_t e = cudaEventSynchronize(ctx->slots[slot].done);
  ctx->slots[slot].in_flight = false;
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_layer_host_wait");
  return MOE_OK;
}

moe_status moe_ctx_set_segments(moe_ctx* ctx, int32_t experts_per_segment, moe_boundary_fn fn, void* user) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (experts_per_segment < 0) return fail(ctx, MOE_ERR_INVALID_ARG, "experts_per_segment < 0");
  if (ctx->state != ST_IDLE) return fail(ctx, MOE_ERR_STATE, "segmentation can only change between steps");
  ctx->seg_experts = experts_per_segment;
  ctx->boundary_fn = fn;
  ctx->boundary_user = user;
  return MOE_OK;
}

moe_status moe_ctx_set_preemption(moe_ctx* ctx, int32_t enabled) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->state != ST_IDLE) return fail(ctx, MOE_ERR_STATE, "preemption can only change between steps");
  if (enabled && ctx->cfg.phase != MOE_PHASE_PREFILL)
    return fail(ctx, MOE_ERR_INVALID_ARG, "only a PREFILL context can be made preemptible");
  if (enabled && ctx->yield_src == nullptr) {
    DeviceGuard guard(ctx->device);
    void *y = nullptr, *st = nullptr;
    cudaStream_t ys = nullptr;
    cudaError_t e = cudaHostAlloc(&y, 64, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaHostAlloc(&st, 64, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ys, cudaStreamNonBlocking);
    std::mutex* mu = new (std::nothrow) std::mutex();
    if (e != cudaSuccess || mu == nullptr) {
      if (y) cudaFreeHost(y);
      if (st) cudaFreeHost(st);
      if (ys) cudaStreamDestroy(ys);
      delete mu;
      return e != cudaSuccess ? cuda_fail(ctx, e, "moe_ctx_set_preemption") : fail(ctx, MOE_ERR_CUDA, "host allocation failed");
    }
    memset(y, 0, 64);
    memset(st, 0, 64);
    static_cast<int*>(y)[1] = 1;
    ctx->yield_src = static_cast<int*>(y);
    ctx->yield_dev = ctx->status + 2;
    ctx->stopped_host = static_cast<int*>(st);
    ctx->yield_stream = ys;
    ctx->yield_mu = mu;
  }
  ctx->preemptible = enabled != 0;
  if (ctx->yield_src) return moe_ctx_request_yield(ctx, 0);
  return MOE_OK;
}

moe_status moe_ctx_request_yield(moe_ctx* ctx, int32_t on) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->yield_src == nullptr) return MOE_ERR_STATE;  // preemption was never switched on (no message: any thread may call)
  DeviceGuard guard(ctx->device);
  std::lock_guard<std::mutex> lock(*ctx->yield_mu);
  cudaError_t e = cudaMemcpyAsync(ctx->yield_dev, ctx->yield_src + (on ? 1 : 0), sizeof(int), cudaMemcpyHostToDevice,
                                  ctx->yield_stream);
  // lowering is complete when this returns, so that a pass launched afterwards does not see a stale request
  if (e == cudaSuccess && !on) e = cudaStreamSynchronize(ctx->yield_stream);
  return e == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int64_t moe_ctx_yield_count(const moe_ctx* ctx) { return ctx ? ctx->yields : 0; }

moe_status moe_ctx_set_wait_limit(moe_ctx* ctx, int64_t limit_us) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (limit_us < 0) return fail(ctx, MOE_ERR_INVALID_ARG, "limit_us < 0");
  ctx->wait_limit_ns = (unsigned long long)limit_us * 1000ull;
  return MOE_OK;
}

moe_status moe_ctx_debug_inject_stall(moe_ctx* ctx, int32_t enabled) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->debug_stall = enabled != 0;
  return MOE_OK;
}

moe_status moe_ctx_set_profiling(moe_ctx* ctx, int32_t enabled) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->profiling = enabled != 0;
  return MOE_OK;
}

moe_status moe_ctx_read_profile(moe_ctx* ctx, moe_stage_times* out) {
  if (!ctx || !out) return MOE_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  memset(out, 0, sizeof *out);
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "moe_ctx_read_profile");
  for (size_t i = 0; i < ctx->spans_used; ++i) {
    const moe_ctx::Span& sp = ctx->spans[i];
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, sp.beg, sp.end) == cudaSuccess && sp.stage >= 0 && sp.stage < MOE_N_STAGES) {
      out->ms[sp.stage] += ms;
      out->calls[sp.stage] += 1;
    } else {
      (void)cudaGetLastError();
    }
  }
  ctx->spans_used = 0;
  return MOE_OK;
}

moe_status moe_ctx_debug_ptrs(moe_ctx* ctx, void** x_perm, void** act, void** y_perm, void** y_shared,
                              int32_t** counts, int32_t** offsets) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  // after moe_combine a DECODE context has already flipped; report the set the last step used
  const int set = (ctx->n_sets == 2 && ctx->state == ST_IDLE) ? (ctx->cur ^ 1) : ctx->cur;
  BufferSet& b = ctx->sets[set];
  if (x_perm) *x_perm = b.x_perm;
  if (act) *act = b.act;
  if (y_perm) *y_perm = b.y_perm;
  if (y_shared) *y_shared = b.y_shared;
  if (counts) *counts = b.counts;
  if (offsets) *offsets = b.offsets;
  return MOE_OK;
}

moe_status moe_ctx_debug_ptrs_fp8(moe_ctx* ctx, void** xq, float** sx, void** aq, float** sa) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  if (ctx->cfg.weight_format != MOE_WEIGHTS_FP8_E4M3)
    return fail(ctx, MOE_ERR_STATE, "the context was not created with weight_format = MOE_WEIGHTS_FP8_E4M3");
  const int set = (ctx->n_sets == 2 && ctx->state == ST_IDLE) ? (ctx->cur ^ 1) : ctx->cur;
  BufferSet& b = ctx->sets[set];
  if (xq) *xq = b.xq;
  if (sx) *sx = b.sx;
  if (aq) *aq = b.aq;
  if (sa) *sa = b.sa;
  return MOE_OK;
}

}  // extern "C"
