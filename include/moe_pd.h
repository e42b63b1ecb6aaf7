/*
 * moe_pd.h -- C ABI of the phase-owned MoE layer for in-place prefill/decode multiplexing.
 *
 * The layer is the one prefill (P) and decode (D) both execute on shared devices:
 *   route -> dispatch layout (counts, exclusive scan, stable permutation, row movement)
 *         -> grouped SwiGLU expert FFN (+ shared expert) -> weighted combine.
 * The paper's Section "DeepEP Communication-State Isolation" requires that everything a
 * communication/layout kernel MODIFIES (buffers, counters, workspace, stream, events,
 * D's double-buffer index) is owned by exactly one phase, while initialisation and the
 * model weights are shared (Table "Ownership in the concurrent DeepEP runtime").  Here
 * that is one `moe_ctx` per phase: two contexts never share a mutable byte, and the
 * only memory reachable from both is the read-only weights the caller passes in.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned,
 *     dense row-major.  The library never frees or keeps them beyond the stream work
 *     of the step they belong to.  Only `moe_layer_host` and `moe_layer_host_submit` take HOST pointers.
 *   - Calls validate on the host, enqueue kernels on the context's stream and return.
 *     They do not synchronise, allocate device memory or read device memory back
 *     (except `moe_ctx_status`, `moe_ctx_destroy`, `moe_layer_host` and `moe_layer_host_wait`, which say so).
 *   - Host threads: calls on ONE context must not overlap in time (a context is not locked; give each phase's
 *     context to one thread, or serialise).  Calls on different contexts, creation and destruction included,
 *     may run concurrently from different threads; the turnstile controller is thread-safe by itself.
 *   - Every function returns a `moe_status`; no exception crosses the boundary.
 *     `moe_last_error` gives a human-readable reason for the last failure on a context.
 *   - Problems only the device can see (an expert index outside [0,E), a bounded wait
 *     that ran out) make the kernel skip the offending work and record a code in the
 *     context's device status word; nothing traps.  `moe_ctx_status` reads it.
 *   - bf16 tensors are passed as `const void*` / `void*`.
 *
 * Per step, in order:  moe_route (optional) -> moe_dispatch_layout (or its two halves moe_dispatch_notify ->
 * moe_dispatch_move) -> moe_grouped_ffn -> moe_combine.  Any other order returns MOE_ERR_STATE.
 *
 * CUDA graphs.  The four step calls only enqueue kernels, so a step may be recorded while the
 * context's stream is being captured and replayed later (D keeps stable graph addresses: the
 * graph holds the buffer set that was current at capture, whatever the double-buffer index
 * does afterwards).  Run one step eagerly first (it configures the kernels), keep every
 * array the step touches alive and in place, and do not capture moe_layer_host,
 * moe_ctx_status or moe_ctx_read_profile (they synchronise).
 */
#ifndef MOE_PD_H_
#define MOE_PD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct moe_ctx moe_ctx; /* opaque; one per phase */

/* Explicit phase identity: it selects state and kernel variant, and is never inferred
 * from a host thread or a stream (Section "End-to-End Integration"). */
typedef enum { MOE_PHASE_PREFILL = 0, MOE_PHASE_DECODE = 1 } moe_phase;

typedef enum {
  MOE_OK = 0,
  MOE_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, bad shape                        */
  MOE_ERR_CAPACITY = 2,    /* T > max_tokens, or workspace too small                      */
  MOE_ERR_STATE = 3,       /* call out of order, overlapping workspaces, destroy while busy */
  MOE_ERR_UNSUPPORTED = 4, /* shape outside what the kernels handle                       */
  MOE_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed                           */
  MOE_ERR_TIMEOUT = 6,     /* device: a bounded wait gave up                              */
  MOE_ERR_BAD_INDEX = 7    /* device: an expert index was outside [0, E)                  */
} moe_status;

/* GEMM kernel variants.  AUTO: a DECODE context uses small-M; a PREFILL context chooses per step and pass from
 * the step's rows per expert R = T * top_k / n_experts and the pass's K (hidden for the gated pass, inter for the
 * down pass): small-M for every problem of up to 8192 rows; above that, the gated pass up to R = 1024 (with
 * K < 4096 only from R = 448 on) and the down pass up to R = 320 when its K is at least 1536; with FP8 weights
 * up to R = 256 (K >= 4096) and 128 (K >= 1536); large-M otherwise -- a function of T alone, so a step captured in a CUDA graph replays
 * the kernels it was captured with. */
typedef enum {
  MOE_GEMM_AUTO = 0,
  MOE_GEMM_LARGE_M = 1,  /* tokens fill the 128-row MMA dimension; for experts of many hundreds of rows,
                            where the pass is bound by the tensor cores                            */
  MOE_GEMM_SMALL_M = 2,  /* swap-AB: weight rows fill the MMA M dimension, an expert's tokens sit in N
                            (16..256 per tile, following the expert's row count), so each expert's
                            weights enter an SM once per 256 tokens -- for experts of few rows, where
                            the pass is bound by streaming the weights                             */
  MOE_GEMM_VALIDATION = 3 /* plain CUDA-core kernel, slow; exists to localise tensor-core bugs   */
} moe_gemm_variant;

/* Precision of the expert weights a context will be given.  BF16 is the path the whole library is measured
 * on; FP8_E4M3 enables moe_grouped_ffn_fp8 (the paper evaluates its models in BF16 and in FP8, Section
 * "Evaluation", "Methodology"). */
typedef enum { MOE_WEIGHTS_BF16 = 0, MOE_WEIGHTS_FP8_E4M3 = 1 } moe_weight_format;

typedef struct {
  int32_t hidden;       /* H, multiple of 64                                            */
  int32_t n_experts;    /* E, 1..1024                                                   */
  int32_t top_k;        /* k, 1..min(E,32)                                              */
  int32_t inter;        /* I, routed expert intermediate size, multiple of 64           */
  int32_t n_shared;     /* S in {0,1}: number of shared experts                         */
  int32_t shared_inter; /* I_s, multiple of 64 (ignored when S = 0)                     */
  int32_t max_tokens;   /* capacity; T of a call may be anything in [0, max_tokens]     */
  int32_t phase;        /* moe_phase                                                    */
  int32_t sm_budget;    /* 0 = all SMs; else the most CTAs a persistent kernel of this
                           context may occupy (the analogue of the paper's separate
                           communication-SM budgets per phase)                          */
  int32_t gemm_variant; /* moe_gemm_variant                                             */
  int32_t row_gather;   /* 0: moe_dispatch_layout writes x_perm (stage a5 is its own kernel).
                           1: with the large-M GEMM variant, GEMM1 gathers its rows from x
                              through perm while it runs; x_perm is not written, and x must
                              be passed to moe_grouped_ffn.  Ignored by the other variants. */
  float routed_scale;   /* multiplies the routed weights; 1.0f unless the model says so */
  int32_t weight_format; /* moe_weight_format; FP8 adds the quantisation buffers to the workspace */
} moe_config;

/* Bytes of device workspace `moe_ctx_create` needs for this configuration (0 on a bad config).
 * A DECODE context holds two buffer sets, selected by a double-buffer index that flips at
 * every moe_combine, so that its addresses stay stable across steps. */
size_t moe_ctx_workspace_bytes(const moe_config* cfg);

/* Creates a phase context bound to `cuda_stream` (a cudaStream_t; NULL = the legacy default
 * stream) that owns [workspace, workspace + workspace_bytes) -- device memory the caller
 * allocated (256-byte aligned) and keeps alive until moe_ctx_destroy.  The range is
 * registered process-wide: a range overlapping a live context's, or a stream already bound
 * to a live context of the other phase, is refused with MOE_ERR_STATE (construction
 * validates isolation before any kernel runs).  Enqueues one memset on the stream; if the workspace was
 * allocated or last used on another stream (a stream-ordered or caching allocator may hand out a block that
 * still has work pending there), order the two streams before this call. */
moe_status moe_ctx_create(const moe_config* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream,
                          moe_ctx** out);

/* Destroys a context at a quiescent point.  If work may still be in flight on its stream
 * it returns MOE_ERR_STATE and the context stays valid (an abandoned operation retires its
 * buffer only at quiescent cleanup); otherwise it unregisters the workspace and frees the
 * host object.  Device memory is the caller's and is not freed. */
moe_status moe_ctx_destroy(moe_ctx* ctx);

/* Abandons the step in progress (after a failed call, or because the caller changed its plan) and returns the
 * context to the state between steps; a no-op when no step is in progress.  Kernels already enqueued for the
 * step still run.  Following the paper's lifetime rule that an abandoned operation retires its buffer until a
 * quiescent point (Section "Network and Lifetime Isolation"), a DECODE context moves on to its other buffer
 * set, so the abandoned step's buffers are written again only after one more whole step has been enqueued
 * behind them on the stream.  Enqueues nothing and does not synchronise. */
moe_status moe_ctx_abandon_step(moe_ctx* ctx);

/* Time limit of every bounded device-side wait of this context's kernels, in microseconds (0 restores the
 * default of 2 s).  A wait that runs out makes the kernel record MOE_ERR_TIMEOUT in the status word and return
 * (the paper's controller likewise detects protocol violations instead of waiting forever, Section "Rank-Aligned
 * Segment Boundaries"); a service that prefers to fail fast on a wedged device sets a few milliseconds. */
moe_status moe_ctx_set_wait_limit(moe_ctx* ctx, int64_t limit_us);

/* Test hook of the failure-detection path (the paper has no counterpart): while enabled, the copy-issuing warp
 * of this context's GEMM kernels issues nothing, so every consumer wait runs into the limit set by
 * moe_ctx_set_wait_limit, the kernels report MOE_ERR_TIMEOUT through the status word, free their tensor
 * memory and return.  The outputs of such a step are undefined.  Use a short limit with it. */
moe_status moe_ctx_debug_inject_stall(moe_ctx* ctx, int32_t enabled);

/* Synchronises the context's stream and returns the device status word (a moe_status:
 * MOE_OK, MOE_ERR_TIMEOUT or MOE_ERR_BAD_INDEX) in *device_status, then clears it. */
moe_status moe_ctx_status(moe_ctx* ctx, int32_t* device_status);

/* Reason for the last non-OK return on this context (static storage inside the context;
 * valid until the next call on it).  Never NULL.  With ctx == NULL: the reason for the
 * last failed moe_ctx_create on this thread. */
const char* moe_last_error(const moe_ctx* ctx);

/* Stage a1 -- top-k routing over given router logits.
 *   key[e]      = logits[t,e] + select_bias[e]  (one fp32 add; select_bias NULL: key = logits)
 *   topk_idx[t] = the k experts of largest key, descending; equal keys (IEEE ==, so +0 and -0
 *                 tie) go to the lower expert index
 *   topk_w[t,j] = routed_scale * softmax over the k selected UNBIASED logits
 * logits [T,E] fp32, select_bias [E] fp32 or NULL, topk_idx [T,k] int32, topk_w [T,k] fp32.
 * Inputs must be finite; with NaN/Inf the selection is unspecified but still k distinct
 * in-range indices.  T = 0 is a legal no-op. */
moe_status moe_route(moe_ctx* ctx, const float* logits, const float* select_bias, int32_t T, int32_t* topk_idx,
                     float* topk_w);

/* Stages a2-a5 -- the local part of a dispatch: per-expert counts (the "receive counts"),
 * their exclusive scan (the "tensor allocation"), the stable token-to-expert permutation and
 * the routed row movement (Section "Exposing a Safe Prefill Boundary" lists these stages).
 * With flat slot f = t*k + j and N = T*k:
 *   counts[e]  = #{f : topk_idx[f] == e};   offsets[0] = 0, offsets[e+1] = offsets[e] + counts[e]
 *   perm[p] = f and inv_perm[f] = p, where slots of one expert keep ascending f (stable)
 *   x_perm[p,:] = x[perm[p] / k, :]   (bit copy into the context's workspace; with row_gather = 1 the copy is
 *                 skipped and GEMM1 reads x through perm; a context created for FP8 weights quantises each row
 *                 of x once and moves the E4M3 codes and the row scales instead, see moe_grouped_ffn_fp8)
 * topk_idx [T,k] int32 (the caller's own routing is welcome; moe_route is optional);
 * x [T,H] bf16, or NULL to build the layout only (then moe_grouped_ffn is not allowed);
 * counts [E], offsets [E+1], perm [N], inv_perm [N] int32 -- each may be NULL, in which
 * case the context keeps that array privately.  Arrays the caller does pass must stay
 * untouched until moe_combine of the same step has been enqueued.
 * A slot whose index is outside [0,E) is dropped (inv_perm[f] = -1), the device status
 * becomes MOE_ERR_BAD_INDEX, and the slot contributes nothing to the output.
 * T = 0 zero-fills counts and offsets. */
moe_status moe_dispatch_layout(moe_ctx* ctx, const int32_t* topk_idx, int32_t T, const void* x, int32_t* counts,
                               int32_t* offsets, int32_t* perm, int32_t* inv_perm);

/* Split-phase dispatch.  The paper splits a normal (prefill) dispatch AFTER notification: expert notification and
 * the receive counts come first; the routed data movement happens only after the counts are there AND the
 * boundary controller has given its permit, so that a ready decode iteration can be ordered in between; the backend
 * keeps a pending-dispatch record (the tensors and the stream state the second half needs), allows at most one
 * pending dispatch per prefill buffer and makes every transition explicit (Section "Exposing a Safe Prefill
 * Boundary").  On one GPU the two halves of moe_dispatch_layout are:
 *   moe_dispatch_notify   stages a2-a4 only (counts, exclusive scan, stable permutation; arguments as for
 *                         moe_dispatch_layout without x).  The context then holds a pending dispatch: the arrays, T
 *                         and the stream position of this half.  With prefill segmentation on, the boundary hook is
 *                         called here as boundary 0 of 1 + (the boundaries of moe_grouped_ffn), which then
 *                         reports its own as 1, 2, ...: the first safe point of a prefill step lies before any
 *                         row has moved.
 *   moe_dispatch_move     stage a5, the routed data movement of the pending dispatch (x [T,H] bf16; an FP8 context
 *                         quantises and moves codes, a row_gather context moves nothing).  The counts need no
 *                         host round trip here -- they stay on the device and the stream orders the two halves --
 *                         so calling this function IS the permit.  Afterwards the step continues with
 *                         moe_grouped_ffn as after moe_dispatch_layout.
 * Transitions: idle/routed --notify--> pending --move--> laid out.  A second moe_dispatch_notify or a
 * moe_dispatch_layout while a dispatch is pending returns MOE_ERR_STATE, as does moe_dispatch_move without one;
 * moe_ctx_abandon_step retires a pending dispatch together with the step (kernels already enqueued still run).
 * If moe_dispatch_move fails the dispatch stays pending.  moe_ctx_pending_dispatch reports whether a dispatch is
 * pending, its T, and whether the first half has already finished on the device (an event query; no wait). */
moe_status moe_dispatch_notify(moe_ctx* ctx, const int32_t* topk_idx, int32_t T, int32_t* counts, int32_t* offsets,
                               int32_t* perm, int32_t* inv_perm);
moe_status moe_dispatch_move(moe_ctx* ctx, const void* x);
moe_status moe_ctx_pending_dispatch(moe_ctx* ctx, int32_t* pending, int32_t* tokens, int32_t* notified_done);

/* Stages a6-a8 -- grouped SwiGLU expert FFN over the permuted rows, plus the shared expert:
 *   act[p,i]    = silu(x_perm[p,:] . W_gate_up[e,i,:]) * (x_perm[p,:] . W_gate_up[e,I+i,:])
 *   y_perm[p,c] = act[p,:] . W_down[e,c,:]          for p in expert e's segment
 *   y_shared    = the same FFN with the shared weights on x[t,:] for every token (S = 1)
 * bf16 operands, fp32 accumulation on the tensor cores, silu(z) = z / (1 + exp(-z)) in fp32;
 * act, y_perm and y_shared are stored as bf16 (round to nearest even) in the workspace.
 * w_gate_up [E,2I,H] bf16 (rows 0..I-1 gate, I..2I-1 up), w_down [E,H,I] bf16,
 * ws_gate_up [2I_s,H], ws_down [H,I_s] bf16 (required iff S = 1), x [T,H] bf16 (read by the
 * shared expert and by the row gather; required iff S = 1 or row_gather = 1; it must be the x
 * that moe_dispatch_layout was given).  Weights are read-only and may be shared by contexts. */
moe_status moe_grouped_ffn(moe_ctx* ctx, const void* w_gate_up, const void* w_down, const void* x,
                           const void* ws_gate_up, const void* ws_down, int32_t T);

/* Stages a6-a8 with FP8 weights and activations (context created with weight_format = MOE_WEIGHTS_FP8_E4M3;
 * same place in the step as moe_grouped_ffn, which such a context refuses).  The paper names FP8 runs but
 * prints no recipe; this one is W8A8 with OCP E4M3 codes (1-4-3 bits, bias 7, largest finite value 448, no
 * infinities):
 *   weights      wq_* hold E4M3 codes, sw_* one fp32 scale per output channel (weight row):
 *                W[e,r,:] = sw[e,r] * decode(wq[e,r,:])
 *   activations  every bf16 row v entering a GEMM is quantised on the fly, per row:
 *                amax = max(max|v|, 2^-100), scale = amax / 448, code_i = e4m3(v_i * (448 / amax)), all in
 *                IEEE fp32, conversion round-to-nearest-even saturating at +-448
 *   GEMM1        g, u = (sum_h x_code * w_code) * scale_x[p] * sw[e,row], act = silu(g) * u stored as bf16
 *   GEMM2        act is quantised per row as above; y = (sum_i a_code * w_code) * scale_a[p] * sw[e,c], bf16
 * The sums run on the tensor cores (tcgen05 kind::f8f6f4) with fp32 accumulation.  On such a context
 * moe_dispatch_layout quantises each row of x once (stage 8 of the profile) and moves the codes and the row
 * scales instead of the bf16 rows, so the workspace holds no bf16 x_perm.  The shared expert (S = 1) is computed
 * the same way from the quantised x with its own codes and scales.
 * wq_gate_up [E,2I,H] uint8, sw_gate_up [E,2I] fp32, wq_down [E,H,I] uint8, sw_down [E,H] fp32;
 * wsq_gate_up [2I_s,H], sws_gate_up [2I_s], wsq_down [H,I_s], sws_down [H] (required iff S = 1).
 * H, I and I_s may not exceed 8192.  Prefill segmentation (moe_ctx_set_segments) applies as to moe_grouped_ffn,
 * the quantisation of the activation being one more segment between the two passes; the row gather and the
 * host-buffer entry points do not apply to an FP8 context.  Errors as for moe_grouped_ffn; MOE_ERR_STATE if the context was created for BF16 weights. */
moe_status moe_grouped_ffn_fp8(moe_ctx* ctx, const void* wq_gate_up, const float* sw_gate_up, const void* wq_down,
                               const float* sw_down, const void* wsq_gate_up, const float* sws_gate_up,
                               const void* wsq_down, const float* sws_down, int32_t T);

/* Prefill segmentation.  A single P execution spans several D iterations, so the paper divides P into
 * segments delimited by backend-provided boundaries (Section "In-Place P/D Execution"; the span K of Section
 * "Prefill Policy Interface").  With experts_per_segment > 0, moe_grouped_ffn enqueues each routed GEMM pass
 * as one launch per group of that many experts (the shared-expert passes are segments of their own) and
 * calls `fn(user, i, n)` on the calling host thread right after segment i of n has been enqueued: a safe
 * point at which the caller's controller may enqueue a D step on another context and order the streams (for
 * instance make this context's stream wait for an event of the D stream) before the next segment is
 * enqueued.  The callback must not call into THIS context.  Results are bit-identical to the unsegmented
 * call.  experts_per_segment = 0 switches segmentation off; fn may be NULL. */
typedef void (*moe_boundary_fn)(void* user, int32_t boundary, int32_t n_boundaries);
moe_status moe_ctx_set_segments(moe_ctx* ctx, int32_t experts_per_segment, moe_boundary_fn fn, void* user);

/* Preemption of a prefill step at tile granularity -- boundaries without cutting P into many launches.
 * The paper lets successive D iterations advance through one long P execution at backend-provided boundaries
 * (Section "In-Place P/D Execution"); on one GPU, where P and D compete for the same SMs and the same HBM, the
 * finest boundary that costs nothing while no D is waiting is the end of a GEMM tile.  With preemption on (PREFILL
 * contexts only), every GEMM pass of moe_grouped_ffn uses the small-M kernel, whose CTAs take their tiles from a
 * counter in the context's workspace and look at a yield request before they take one (tens of microseconds
 * apart).  moe_ctx_request_yield(ctx, 1) -- callable from any host thread, typically the one about to enqueue a D
 * step -- raises the request: every CTA finishes the tiles it has taken (the one it is in and at most the next) and
 * exits, so the SMs are free within a tile or two.  moe_grouped_ffn, which in this mode WAITS
 * ON THE HOST for each of its launches (eager variable-length P; it cannot be captured in a graph and costs a
 * host round trip of ~10 us per launch), then calls the boundary hook as fn(user, MOE_BOUNDARY_YIELD, 0) and,
 * when the hook returns, launches the pass again: the counter goes on with the tiles not yet taken.  The hook is the permit
 * wait: it should return once the D step has finished on the device and the request has been lowered
 * (moe_ctx_request_yield(ctx, 0)); a request still up is honoured again (up to 64 launches per pass, after which
 * the pass runs to its end regardless).  Results are bit-identical to the unpreempted pass.  The request is a
 * word in the context's workspace; raising it is a 4-byte asynchronous copy on a private stream of the context
 * (it reaches the kernels within microseconds), lowering it also waits for that copy, so that a pass launched
 * after the call returns cannot see a stale request.  The first moe_ctx_set_preemption(ctx, 1) creates that
 * stream and two small pinned host buffers (host resources, released by moe_ctx_destroy).
 * moe_ctx_yield_count: launches that ended on a request since the context was created. */
#define MOE_BOUNDARY_YIELD (-1)
moe_status moe_ctx_set_preemption(moe_ctx* ctx, int32_t enabled);
moe_status moe_ctx_request_yield(moe_ctx* ctx, int32_t on);
int64_t moe_ctx_yield_count(const moe_ctx* ctx);

/* Segment turnstile -- the host-side boundary controller (Sections "Rank-Aligned Segment Boundaries" and
 * "Distributed Segment Turnstile").  Host-only: it orders host enqueue, never waits for GPU work and launches
 * nothing.  One controller per rank keeps the current P epoch e, the largest reached boundary r (-1 at the start
 * of an epoch), the permitted endpoint p, the positive span K and the task state.
 *   P side   moe_turnstile_begin_epoch(e, d_already_enqueued): r = -1; p = K if a D iteration is already
 *            enqueued, else 0 (so that a ready D is ordered before P enters CUDA).
 *            moe_turnstile_publish(e, i): step P1/P2 -- publish boundary i (r = i), then wait while i >= p.
 *            Call it with i = 0 before the first segment is enqueued and with i + 1 after segment i has been
 *            (the boundary hook of moe_ctx_set_segments is the place).  moe_turnstile_task_done(e) after the
 *            final segment.
 *   D side   moe_turnstile_d_enter: step D1 -- if p > 0 wait until r >= p or the epoch is done; *p_active says
 *            whether a P epoch is running.  The caller then runs its PreDRendezvous over all ranks (any CPU
 *            barrier), enqueues the D calls (D2), runs its PostDRendezvous (D3) and calls
 *            moe_turnstile_d_release: step D4 -- p <- p + K for an active epoch, without waiting for P's GPU work.
 * Rejected with MOE_ERR_STATE: a stale or duplicate epoch, a publication or completion for an epoch that was
 * never begun (missing producer), a boundary that is not larger than the last one, a boundary beyond the
 * current permit, beginning an epoch while one is active, destroying a controller with an active epoch.
 * Every wait takes timeout_ms (negative = unbounded) and returns MOE_ERR_TIMEOUT when it runs out. */
typedef struct moe_turnstile moe_turnstile;
moe_status moe_turnstile_create(int32_t span, moe_turnstile** out);
moe_status moe_turnstile_destroy(moe_turnstile* ts);
moe_status moe_turnstile_set_span(moe_turnstile* ts, int32_t span);
moe_status moe_turnstile_begin_epoch(moe_turnstile* ts, int64_t epoch, int32_t d_already_enqueued);
moe_status moe_turnstile_publish(moe_turnstile* ts, int64_t epoch, int32_t boundary, int32_t timeout_ms);
moe_status moe_turnstile_task_done(moe_turnstile* ts, int64_t epoch);
moe_status moe_turnstile_d_enter(moe_turnstile* ts, int32_t timeout_ms, int32_t* p_active);
moe_status moe_turnstile_d_release(moe_turnstile* ts);
moe_status moe_turnstile_state(moe_turnstile* ts, int64_t* epoch, int32_t* reached, int32_t* permit, int32_t* span,
                               int32_t* active);

/* Stage a9 -- weighted combine back to token order:
 *   out[t,:] = sum_j topk_w[t,j] * y_perm[inv_perm[t*k+j],:]  (+ y_shared[t,:]),  fp32 sum, bf16 store.
 * topk_w [T,k] fp32; inv_perm [N] int32 or NULL to use the layout of this step kept by the
 * context; out [T,H] bf16.  Deterministic: fixed summation order, no atomics.
 * Ends the step; a DECODE context then flips its double-buffer index. */
moe_status moe_combine(moe_ctx* ctx, const float* topk_w, const int32_t* inv_perm, int32_t T, void* out);

/* The same layout (stages a2-a4, no row movement) for callers that cannot allocate device memory and so
 * cannot supply a context with a workspace: code that runs inside another framework's memory pool, a
 * runtime that has handed every byte of the device to its own allocator, or any place where cudaMalloc is
 * forbidden.  (The paper has no counterpart of this entry point; it exists for such embedders.)
 * The scratch the large-T path needs lives in a 256 KiB array inside the library image, which each GPU that
 * loads the library holds until the process exits.  Limit: ceil(T*top_k / 256) * n_experts <= 65536
 * (e.g. T*top_k <= 65536 at 256 experts); beyond it the call returns MOE_ERR_CAPACITY and does nothing.
 * The call allocates nothing and frees nothing.  It works on the device that is current when it is called:
 * the pointers and the stream must belong to that device.  The first call on each device looks up the
 * array's device address (a host-side set-up step); make that first call before any stream capture begins.
 * A call with more experts than any earlier call on that device (single-launch path, T*top_k <= 16384) also
 * raises a kernel's shared-memory limit on the host, so it too should come before capture.
 * All calls on one device share the array: two calls whose kernels can overlap on the GPU (different
 * streams without an ordering between them) race on it -- order them.  Nothing in the array needs clearing
 * between calls: every cell is written before it is read within a call.
 * Arguments and results are those of moe_dispatch_layout with x == NULL; all four output arrays are
 * required (perm and inv_perm may be NULL only when T == 0).  An out-of-range expert index is dropped
 * (inv_perm[f] = -1); there is no status word to report it to. */
moe_status moe_dispatch_layout_static(const int32_t* topk_idx, int32_t T, int32_t top_k, int32_t n_experts,
                                      int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                                      void* cuda_stream);

/* One whole step with HOST activations: copies logits_host [T,E] fp32 and x_host [T,H] bf16
 * to the device (cudaMemcpyAsync into context-owned staging), runs a1..a9, copies out
 * [T,H] bf16 back to out_host and synchronises the stream before returning.  Pinned host
 * memory is recommended.  select_bias and all weights are DEVICE pointers as above. */
moe_status moe_layer_host(moe_ctx* ctx, const float* logits_host, const float* select_bias, const void* x_host,
                          int32_t T, const void* w_gate_up, const void* w_down, const void* ws_gate_up,
                          const void* ws_down, void* out_host);

/* Pipelined form of moe_layer_host: MOE_HOST_SLOTS staging slots, so that the host<->device copies of one step
 * overlap the kernels and the copies of others (host-to-device, kernels and device-to-host run as a three-stage
 * pipeline; with three or more slots in rotation each stage stays busy).  moe_layer_host_submit(slot) enqueues the
 * host-to-device copies of logits_host and x_host on a copy stream of the context, the step's kernels on the
 * context's stream behind them, and the copy of the result to out_host on a second copy stream behind the
 * kernels; it returns without synchronising.  moe_layer_host_wait(slot) blocks the calling thread until that
 * slot's result has arrived in out_host (a no-op for a slot with nothing in flight).  A slot must be waited for
 * before it is submitted again (MOE_ERR_STATE otherwise); the host buffers of a submitted slot must stay valid
 * and untouched until its wait returns, and must be pinned for the copies to overlap anything.  Steps execute in
 * submission order.  The two copy streams and the events are created by the first submit on a context (host
 * resources, no device memory) and belong to that context alone; moe_ctx_destroy refuses while a slot is in
 * flight.  Device-side arguments as for moe_layer_host.  Not for contexts created for FP8 weights. */
#define MOE_HOST_SLOTS 4
moe_status moe_layer_host_submit(moe_ctx* ctx, int32_t slot, const float* logits_host, const float* select_bias,
                                 const void* x_host, int32_t T, const void* w_gate_up, const void* w_down,
                                 const void* ws_gate_up, const void* ws_down, void* out_host);
moe_status moe_layer_host_wait(moe_ctx* ctx, int32_t slot);

/* Test/inspection only: device pointers into the buffer set of the step in progress (between steps: of
 * the step that finished last).  Rows
 * [0, T*k) of x_perm [.,H], act [.,I], y_perm [.,H] and rows [0,T) of y_shared [.,H] are
 * defined after the respective stage.  Any out-pointer may be NULL. */
moe_status moe_ctx_debug_ptrs(moe_ctx* ctx, void** x_perm, void** act, void** y_perm, void** y_shared,
                              int32_t** counts, int32_t** offsets);

/* Test/inspection only, FP8 variant: the quantised GEMM1 input rows and activation rows of the same buffer set
 * (codes [N,H] / [N,I] uint8, scales [N] fp32).  Any out-pointer may be NULL. */
moe_status moe_ctx_debug_ptrs_fp8(moe_ctx* ctx, void** xq, float** sx, void** aq, float** sa);

/* Per-stage device timing (measurement aid; off by default).  While enabled, every stage's launches are
 * bracketed by CUDA events on the context's stream.  moe_ctx_read_profile synchronises the stream, returns
 * the summed device time and the number of bracketed launches per stage since the last read, and resets.
 * Stage order: 0 route, 1 layout (counts+scan+permutation), 2 permute rows, 3 routed GEMM1+SwiGLU,
 * 4 routed GEMM2, 5 shared GEMM1+SwiGLU, 6 shared GEMM2, 7 combine.  Without prefill segmentation the shared
 * expert's passes ride in the routed launches, so their time is part of stages 3 and 4 and stages 5 and 6
 * stay empty.  FP8 variant only: 8 quantise the GEMM1 input rows, 9 quantise the activation rows. */
#define MOE_N_STAGES 10
typedef struct {
  double ms[MOE_N_STAGES];
  int64_t calls[MOE_N_STAGES];
} moe_stage_times;
moe_status moe_ctx_set_profiling(moe_ctx* ctx, int32_t enabled);
moe_status moe_ctx_read_profile(moe_ctx* ctx, moe_stage_times* out);

/* Kernels launched on this context since creation (for launch accounting in benchmarks). */
int64_t moe_ctx_launch_count(const moe_ctx* ctx);

/* Library version string, e.g. "moe_pd 0.1 (sm_100a)". */
const char* moe_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MOE_PD_H_ */
