// Segment turnstile: the host-side boundary controller that lets successive D iterations advance through a
// long P execution (paper, Sections "Rank-Aligned Segment Boundaries" and "Distributed Segment Turnstile").
// Host-only: it orders host ENQUEUE, never waits for GPU completion, and launches nothing.
//
// State per controller: current P epoch e, largest reached boundary r (-1 at the start of an epoch), permitted
// endpoint p, positive span K, task state.  P publishes monotone boundaries i = 0, 1, ... and stops at i = p;
// a D iteration waits until P has reached the endpoint (r >= p) or the epoch is done, enqueues its own calls,
// and then moves the endpoint: p <- p + K.  The two all-rank rendezvous around the D enqueue are the caller's
// (any CPU barrier); this object is one rank's controller.
#include <chrono>
#include <condition_variable>
#include <cstdint>
#include <mutex>
#include <new>

#include "../../include/moe_pd.h"

struct moe_turnstile {
  std::mutex mu;
  std::condition_variable cv;
  int32_t K = 1;
  int64_t epoch = -1;      // current (or last) P epoch
  int64_t last_epoch = -1; // largest epoch ever begun: older or equal ones are stale / duplicate
  bool active = false;     // an epoch has begun and has not reported TaskDone
  int32_t r = -1;          // largest reached boundary
  int32_t p = 0;           // permitted endpoint
  int64_t d_steps = 0;     // D iterations released so far (diagnostics)
};

namespace {
using Clock = std::chrono::steady_clock;

template <typename Pred>
bool wait_bounded(moe_turnstile* ts, std::unique_lock<std::mutex>& lock, int32_t timeout_ms, Pred pred) {
  if (timeout_ms < 0) {
    ts->cv.wait(lock, pred);
    return true;
  }
  return ts->cv.wait_for(lock, std::chrono::milliseconds(timeout_ms), pred);
}
}  // namespace

extern "C" {

moe_status moe_turnstile_create(int32_t span, moe_turnstile** out) {
  if (!out) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  if (span < 1) return MOE_ERR_INVALID_ARG;
  moe_turnstile* ts = new (std::nothrow) moe_turnstile();
  if (!ts) return MOE_ERR_CUDA;
  ts->K = span;
  *out = ts;
  return MOE_OK;
}

moe_status moe_turnstile_destroy(moe_turnstile* ts) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  {
    std::lock_guard<std::mutex> lock(ts->mu);
    if (ts->active) return MOE_ERR_STATE;  // an epoch is still running
  }
  delete ts;
  return MOE_OK;
}

moe_status moe_turnstile_set_span(moe_turnstile* ts, int32_t span) {
  if (!ts || span < 1) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(ts->mu);
  ts->K = span;  // takes effect at the next release (the segment policy may change it between rounds)
  return MOE_OK;
}

moe_status moe_turnstile_begin_epoch(moe_turnstile* ts, int64_t epoch, int32_t d_already_enqueued) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(ts->mu);
  if (epoch <= ts->last_epoch) return MOE_ERR_STATE;  // stale or duplicate epoch
  if (ts->active) return MOE_ERR_STATE;               // the previous epoch never reported TaskDone
  ts->epoch = ts->last_epoch = epoch;
  ts->active = true;
  ts->r = -1;
  ts->p = d_already_enqueued ? ts->K : 0;  // p = 0 orders a ready D before P enters CUDA
  ts->cv.notify_all();
  return MOE_OK;
}

moe_status moe_turnstile_publish(moe_turnstile* ts, int64_t epoch, int32_t boundary, int32_t timeout_ms) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  std::unique_lock<std::mutex> lock(ts->mu);
  if (!ts->active || epoch != ts->epoch) return MOE_ERR_STATE;  // no producer registered for this epoch / stale
  if (boundary <= ts->r) return MOE_ERR_STATE;                    // non-monotone publication
  if (boundary > ts->p) return MOE_ERR_STATE;                     // P ran past its permitted endpoint
  ts->r = boundary;
  ts->cv.notify_all();
  // P2: stop at the endpoint until a D iteration has moved it
  const bool ok = wait_bounded(ts, lock, timeout_ms, [&] { return boundary < ts->p || !ts->active; });
  return ok ? MOE_OK : MOE_ERR_TIMEOUT;
}

moe_status moe_turnstile_task_done(moe_turnstile* ts, int64_t epoch) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(ts->mu);
  if (!ts->active || epoch != ts->epoch) return MOE_ERR_STATE;
  ts->active = false;
  ts->cv.notify_all();
  return MOE_OK;
}

moe_status moe_turnstile_d_enter(moe_turnstile* ts, int32_t timeout_ms, int32_t* p_active) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  std::unique_lock<std::mutex> lock(ts->mu);
  // D1: endpoint 0 needs no publication; otherwise wait until P stands at the endpoint or the epoch is over
  const bool ok = wait_bounded(ts, lock, timeout_ms, [&] { return !ts->active || ts->p == 0 || ts->r >= ts->p; });
  if (p_active) *p_active = ts->active ? 1 : 0;
  return ok ? MOE_OK : MOE_ERR_TIMEOUT;
}

moe_status moe_turnstile_d_release(moe_turnstile* ts) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(ts->mu);
  ts->d_steps += 1;
  if (ts->active) ts->p += ts->K;  // D4: admit the next P segment; completed epochs follow the no-work path
  ts->cv.notify_all();
  return MOE_OK;
}

moe_status moe_turnstile_state(moe_turnstile* ts, int64_t* epoch, int32_t* reached, int32_t* permit, int32_t* span,
                               int32_t* active) {
  if (!ts) return MOE_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(ts->mu);
  if (epoch) *epoch = ts->epoch;
  if (reached) *reached = ts->r;
  if (permit) *permit = ts->p;
  if (span) *span = ts->K;
  if (active) *active = ts->active ? 1 : 0;
  return MOE_OK;
}

}  // extern "C"
