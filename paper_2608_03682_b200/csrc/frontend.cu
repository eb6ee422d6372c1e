// Data-parallel serving front-end, host side (paper, Sec. "Parallel Execution": the scheduler assigns independent
// requests to data-parallel runners that exchange no state; appendix on eight-GPU serving: rank 0 collects at most
// `max_batch` pending observations, waits up to `window_ms` for a batch to fill, splits it over the workers with a
// fixed local batch each -- the shape their CUDA graph was captured for --, pads the local inputs to that shape and
// drops the padded outputs after the gather).
//
// Two pieces, no device code:
//   * the batcher: a thread-safe queue with the batching window.  A batch is due when `max_batch` requests are
//     pending, or when `window_ms` have passed since the OLDEST pending request arrived (reading: the wait starts
//     with the first observation of a batch, not with the previous batch).
//   * the plan: which (worker, slot) every request of a batch goes to and which slots are padding.  Requests fill the
//     workers in order, `local_batch` each (reading: contiguous blocks, so the gather is a concatenation); workers
//     past the last request run an all-padding batch or, if the caller prefers, nothing (`active_workers`).
#include <chrono>
#include <condition_variable>
#include <deque>
#include <mutex>
#include <new>

#include "../../include/phyai.h"

struct phyai_batcher {
  phyai_batcher_config_t cfg;
  std::mutex mu;
  std::condition_variable cv;
  struct Item {
    uint64_t id;
    std::chrono::steady_clock::time_point t;
  };
  std::deque<Item> q;
};

namespace {
bool config_ok(const phyai_batcher_config_t* c) {
  return c && c->struct_size == sizeof(phyai_batcher_config_t) && c->max_batch && c->n_workers && c->local_batch &&
         (uint64_t)c->n_workers * c->local_batch >= c->max_batch && c->window_ms >= 0.0;
}
}  // namespace

extern "C" {

phyai_status_t phyai_batcher_create(const phyai_batcher_config_t* cfg, phyai_batcher_t** out) {
  if (!out) return PHYAI_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg)) return PHYAI_ERR_INVALID_ARG;
  phyai_batcher* b = new (std::nothrow) phyai_batcher();
  if (!b) return PHYAI_ERR_OOM;
  b->cfg = *cfg;
  *out = b;
  return PHYAI_OK;
}

void phyai_batcher_destroy(phyai_batcher_t* b) { delete b; }

phyai_status_t phyai_batcher_submit(phyai_batcher_t* b, uint64_t request_id) {
  if (!b) return PHYAI_ERR_INVALID_ARG;
  {
    std::lock_guard<std::mutex> lock(b->mu);
    b->q.push_back({request_id, std::chrono::steady_clock::now()});
  }
  b->cv.notify_all();
  return PHYAI_OK;
}

phyai_status_t phyai_batcher_next(phyai_batcher_t* b, double timeout_ms, uint64_t* ids, uint32_t* n) {
  if (!b || !ids || !n) return PHYAI_ERR_INVALID_ARG;
  using clock = std::chrono::steady_clock;
  const auto ms = [](double v) { return std::chrono::duration_cast<clock::duration>(std::chrono::duration<double, std::milli>(v)); };
  const auto give_up = clock::now() + ms(timeout_ms < 0 ? 0 : timeout_ms);
  std::unique_lock<std::mutex> lock(b->mu);
  *n = 0;
  for (;;) {
    const auto now = clock::now();
    if (b->q.size() >= b->cfg.max_batch) break;                                   // full
    if (!b->q.empty() && now >= b->q.front().t + ms(b->cfg.window_ms)) break;    // the oldest request has waited long enough
    if (now >= give_up) return PHYAI_OK;                                         // nothing due: n = 0
    auto until = give_up;
    if (!b->q.empty()) {
      const auto due = b->q.front().t + ms(b->cfg.window_ms);
      if (due < until) until = due;
    }
    b->cv.wait_until(lock, until);
  }
  while (*n < b->cfg.max_batch && !b->q.empty()) {
    ids[(*n)++] = b->q.front().id;
    b->q.pop_front();
  }
  return PHYAI_OK;
}

uint32_t phyai_batcher_pending(phyai_batcher_t* b) {
  if (!b) return 0;
  std::lock_guard<std::mutex> lock(b->mu);
  return (uint32_t)b->q.size();
}

phyai_status_t phyai_batcher_plan(const phyai_batcher_config_t* cfg, uint32_t n, int32_t* slots, uint32_t* active_workers) {
  if (!config_ok(cfg) || !slots || n > cfg->max_batch) return PHYAI_ERR_INVALID_ARG;
  const uint32_t total = cfg->n_workers * cfg->local_batch;
  for (uint32_t i = 0; i < total; ++i) slots[i] = i < n ? (int32_t)i : -1;   // slot (w, j) = index w * local_batch + j
  if (active_workers) *active_workers = (n + cfg->local_batch - 1) / cfg->local_batch;
  return PHYAI_OK;
}

}  // extern "C"
