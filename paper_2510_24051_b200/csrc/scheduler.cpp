// Batch scheduler of the control layer (Section 5.2 "Batch scheduler", Section 6.1 "Adaptive batch
// scheduling"): per-command-queue FIFOs of pending API calls, batches formed by vertical batching
// (consecutive same-type calls at the head of a queue that do not write the same KvPage) and
// horizontal batching (same type across queues), higher-priority queues first, truncated from the
// tail at the backend's maximum batch size; among API types the one whose oldest eligible call has
// waited longest goes first.  Work-conserving: the embedding runtime asks for the next batch the
// moment the GPU reports idle.  Pure host code.
#include <algorithm>
#include <cstdint>
#include <deque>
#include <new>
#include <unordered_set>
#include <vector>

#include "pie_b200.h"

namespace {
struct Call {
  int32_t type;
  int64_t arrival_ns, tag;
  std::vector<int32_t> writes;
};
struct Queue {
  int priority = 0;
  bool live = false;
  std::deque<Call> calls;
};
}  // namespace

struct pie_sched {
  int max_batch = 1;
  std::vector<Queue> queues;
};

extern "C" {

int pie_sched_create(int32_t max_batch_calls, pie_sched** out) {
  if (!out || max_batch_calls < 1) return PIE_ERR_INVALID;
  pie_sched* s = new (std::nothrow) pie_sched();
  if (!s) return PIE_ERR_INVALID;
  s->max_batch = max_batch_calls;
  *out = s;
  return PIE_OK;
}

int pie_sched_destroy(pie_sched* s) {
  if (!s) return PIE_ERR_INVALID;
  delete s;
  return PIE_OK;
}

int pie_sched_create_queue(pie_sched* s, int32_t priority, int32_t* out_queue) {
  if (!s || !out_queue) return PIE_ERR_INVALID;
  s->queues.emplace_back();
  s->queues.back().priority = priority;
  s->queues.back().live = true;
  *out_queue = (int32_t)s->queues.size() - 1;
  return PIE_OK;
}

int pie_sched_set_queue_priority(pie_sched* s, int32_t queue, int32_t priority) {
  if (!s || queue < 0 || queue >= (int32_t)s->queues.size() || !s->queues[queue].live) return PIE_ERR_INVALID;
  s->queues[queue].priority = priority;
  return PIE_OK;
}

int pie_sched_submit(pie_sched* s, int32_t queue, int32_t type, int32_t n_write, const int32_t* write_pages,
                     int64_t arrival_ns, int64_t tag) {
  if (!s || queue < 0 || queue >= (int32_t)s->queues.size() || !s->queues[queue].live) return PIE_ERR_INVALID;
  if (type < 0 || type >= PIE_SCHED_MAX_TYPES || n_write < 0 || (n_write > 0 && !write_pages)) return PIE_ERR_INVALID;
  Call c;
  c.type = type;
  c.arrival_ns = arrival_ns;
  c.tag = tag;
  c.writes.assign(write_pages, write_pages + n_write);
  s->queues[queue].calls.push_back(std::move(c));
  return PIE_OK;
}

int pie_sched_pending(const pie_sched* s, int32_t* out) {
  if (!s || !out) return PIE_ERR_INVALID;
  int64_t n = 0;
  for (const Queue& q : s->queues) n += (int64_t)q.calls.size();
  *out = (int32_t)std::min<int64_t>(n, 0x7FFFFFFF);
  return PIE_OK;
}

int pie_sched_next_batch(pie_sched* s, int32_t* out_type, int32_t cap, int64_t* out_tags, int32_t* out_queues,
                         int32_t* out_n) {
  if (!s || !out_type || !out_n || cap < 0 || (cap > 0 && !out_tags)) return PIE_ERR_INVALID;
  *out_n = 0;
  *out_type = -1;
  // the API type whose oldest eligible call (a head-of-queue run) has waited longest
  int64_t oldest[PIE_SCHED_MAX_TYPES];
  for (int t = 0; t < PIE_SCHED_MAX_TYPES; ++t) oldest[t] = INT64_MAX;
  for (const Queue& q : s->queues) {
    if (q.calls.empty()) continue;
    const int t = q.calls.front().type;
    for (const Call& c : q.calls) {  // the run of consecutive calls of the head's type
      if (c.type != t) break;
      oldest[t] = std::min(oldest[t], c.arrival_ns);
    }
  }
  int type = -1;
  for (int t = 0; t < PIE_SCHED_MAX_TYPES; ++t)
    if (oldest[t] != INT64_MAX && (type < 0 || oldest[t] < oldest[type])) type = t;
  if (type < 0) return PIE_OK;  // nothing pending

  // queues in priority order (higher first; ties by queue id), each contributing its head run up
  // to the first call that writes a KvPage already written in this batch
  std::vector<int32_t> order;
  for (int32_t qi = 0; qi < (int32_t)s->queues.size(); ++qi)
    if (!s->queues[qi].calls.empty() && s->queues[qi].calls.front().type == type) order.push_back(qi);
  std::stable_sort(order.begin(), order.end(),
                   [&](int32_t a, int32_t b) { return s->queues[a].priority > s->queues[b].priority; });
  const int limit = std::min<int>(s->max_batch, cap);
  std::unordered_set<int32_t> written;
  int n = 0;
  for (int32_t qi : order) {
    Queue& q = s->queues[qi];
    while (n < limit && !q.calls.empty() && q.calls.front().type == type) {  // tail truncation at the limit
      const Call& c = q.calls.front();
      bool conflict = false;
      for (int32_t pg : c.writes) conflict |= written.count(pg) != 0;
      if (conflict) break;  // stays queued (and blocks the rest of its queue) until a later batch
      for (int32_t pg : c.writes) written.insert(pg);
      out_tags[n] = c.tag;
      if (out_queues) out_queues[n] = qi;
      ++n;
      q.calls.pop_front();
    }
    if (n >= limit) break;
  }
  *out_type = type;
  *out_n = n;
  return PIE_OK;
}

}  // extern "C"
