// Host batch planner: the control-layer side of one coalesced `forward` batch (Section 5.2
// "Batch scheduler": a batch is a set of same-type calls that do not conflict; Section 4.2
// "Forward API": explicit boolean masks or masks inferred from positions).
//
// Turns per-request page lists and masks into what the kernels read: per-request records,
// bit-packed masks, a page list with fully masked pages removed, append destinations, and a
// work partition that gives every SM an equal share of page visits.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstring>
#include <condition_variable>
#include <functional>
#include <mutex>
#include <thread>
#if defined(__SSE2__)
#include <emmintrin.h>
#endif

#include "pie_internal.h"

// A context's worker threads: `run(n, fn)` calls fn(0) .. fn(n - 1), each once, on the calling thread and the
// workers, and returns when all are done.  (Starting threads for every batch cost more than the packing of
// a long-context batch's masks gained: ~0.4 ms against ~0.7 ms.)
struct PieWorkers {
  std::vector<std::thread> threads;
  std::mutex m;
  std::condition_variable wake, done;
  const std::function<void(int)>* fn = nullptr;
  std::atomic<int> next{0}, generation{0}, busy{0};
  std::atomic<bool> stop{false};
  int n_tasks = 0;

  explicit PieWorkers(int n_workers) {
    for (int t = 0; t < n_workers; ++t) threads.emplace_back([this] { loop(); });
  }
  ~PieWorkers() {
    {
      std::lock_guard<std::mutex> lk(m);
      stop.store(true);
    }
    wake.notify_all();
    for (auto& t : threads) t.join();
  }
  // Waiting: a short spin first (the planner calls run() several times per batch, some tens of microseconds
  // apart: a sleeping thread takes longer than that to wake up), then the condition variable.
  template <class Pred>
  static bool spin_for(Pred pred) {
    const auto t0 = std::chrono::steady_clock::now();
    for (int k = 0;; ++k) {
      if (pred()) return true;
#if defined(__SSE2__)
      _mm_pause();
#endif
      if ((k & 63) == 63 && std::chrono::steady_clock::now() - t0 > std::chrono::microseconds(200)) return false;
    }
  }
  void drain() {
    for (int k = next.fetch_add(1); k < n_tasks; k = next.fetch_add(1)) (*fn)(k);
  }
  void loop() {
    int seen = 0;
    for (;;) {
      auto ready = [&] { return stop.load(std::memory_order_acquire) || generation.load(std::memory_order_acquire) != seen; };
      if (!spin_for(ready)) {
        std::unique_lock<std::mutex> lk(m);
        wake.wait(lk, ready);
      }
      if (stop.load()) return;
      seen = generation.load(std::memory_order_acquire);
      drain();
      if (busy.fetch_sub(1, std::memory_order_acq_rel) == 1) {
        std::lock_guard<std::mutex> lk(m);
        done.notify_one();
      }
    }
  }
  void run(int n, const std::function<void(int)>& f) {
    fn = &f;
    n_tasks = n;
    next.store(0);
    busy.store((int)threads.size());
    {
      std::lock_guard<std::mutex> lk(m);   // (a worker between its check and its wait holds the mutex: no wake-up is lost)
      generation.fetch_add(1, std::memory_order_release);
    }
    wake.notify_all();
    drain();
    auto idle = [&] { return busy.load(std::memory_order_acquire) == 0; };
    if (!spin_for(idle)) {
      std::unique_lock<std::mutex> lk(m);
      done.wait(lk, idle);
    }
  }
};
void pie_workers_destroy(PieWorkers* w) { delete w; }

// fn(0) .. fn(n - 1): on the context's worker threads when `parallel`, else in order on this thread.
// (Half the hardware threads, at most 16: with all of them the sibling threads of a core slow each other
//  and the serial parts of the planner.)
static int pie_host_threads(int n) {
  return (int)std::min<int64_t>({(int64_t)std::max(1u, std::thread::hardware_concurrency() / 2), 16, (int64_t)n});
}
static void pie_run_tasks(pie_ctx* ctx, int n, bool parallel, const std::function<void(int)>& fn) {
  const int nt = parallel ? pie_host_threads(n) : 1;
  if (nt <= 1) {
    for (int k = 0; k < n; ++k) fn(k);
    return;
  }
  if (!ctx->workers) ctx->workers = new PieWorkers(nt - 1);
  ctx->workers->run(n, fn);
}

namespace {

// Pack `n` bool bytes (each 0 or 1) into bits, LSB first, and zero the rest of the row: all
// `row_words` words of `dst` are written (the destination need not be cleared beforehand).
// Returns false on a byte > 1.
bool pack_row(const uint8_t* src, int64_t n, uint32_t* dst, int row_words) {
  int64_t j = 0;
  uint8_t bad = 0;
#if defined(__SSE2__)
  // 32 bytes -> one word: bit 0 of every byte moved to its sign bit, then gathered by movemask
  __m128i bad_v = _mm_setzero_si128();
  const __m128i not_bool = _mm_set1_epi8((char)0xFE);
  for (; j + 32 <= n; j += 32) {
    const __m128i a = _mm_loadu_si128((const __m128i*)(src + j)), c = _mm_loadu_si128((const __m128i*)(src + j + 16));
    bad_v = _mm_or_si128(bad_v, _mm_and_si128(_mm_or_si128(a, c), not_bool));
    const uint32_t lo = (uint32_t)_mm_movemask_epi8(_mm_slli_epi16(a, 7)), hi = (uint32_t)_mm_movemask_epi8(_mm_slli_epi16(c, 7));
    dst[j >> 5] = lo | (hi << 16);
  }
  bad |= _mm_movemask_epi8(_mm_cmpeq_epi8(bad_v, _mm_setzero_si128())) != 0xFFFF;
#endif
  int64_t k = j >> 5;   // next word to write (j is a multiple of 32 here)
  while (j < n) {
    uint32_t word = 0;
    const int64_t word_end = std::min<int64_t>(j + 32, n);
    int sh = 0;
    for (; j + 8 <= word_end; j += 8, sh += 8) {
      uint64_t x;
      std::memcpy(&x, src + j, 8);
      bad |= (x & 0xFEFEFEFEFEFEFEFEull) != 0;
      // gather the low bit of each byte into one byte (byte k -> bit k)
      word |= ((uint32_t)((x * 0x0102040810204080ull) >> 56) & 0xFFu) << sh;
    }
    for (; j < word_end; ++j, ++sh) {
      bad |= src[j] > 1;
      word |= (uint32_t)(src[j] & 1) << sh;
    }
    dst[k++] = word;
  }
  for (; k < row_words; ++k) dst[k] = 0u;
  return bad == 0;
}

// One bit per page: does the OR of all mask rows (`any_w`, `row_words` words, a multiple of four) have a bit
// in the page's P positions?  Bits for pages [first, first + 64) (first a multiple of 64; P = 8, 16 or 32).
// Which pages an application keeps is not predictable, so the kept-page list is built by walking the set
// bits of these words instead of testing page after page.
uint64_t page_any_bits(const uint32_t* any_w, int row_words, int P, int first) {
  uint64_t out = 0;
  const int w0 = (int)(((int64_t)first * P) >> 5), nw = 2 * P;   // 64 pages span 64 P / 32 words
#if defined(__SSE2__)
  const __m128i zero = _mm_setzero_si128();
  for (int k = 0; k < nw; k += 4) {   // 128 bits: 16 / 8 / 4 pages
    if (w0 + k + 4 > row_words) break;
    const __m128i v = _mm_loadu_si128((const __m128i*)(any_w + w0 + k));
    uint32_t none;
    int per;
    if (P == 8) {
      none = (uint32_t)_mm_movemask_epi8(_mm_cmpeq_epi8(v, zero));
      per = 16;
    } else if (P == 16) {
      const __m128i z = _mm_cmpeq_epi16(v, zero);
      none = (uint32_t)_mm_movemask_epi8(_mm_packs_epi16(z, z)) & 0xFFu;
      per = 8;
    } else {
      none = (uint32_t)_mm_movemask_ps(_mm_castsi128_ps(_mm_cmpeq_epi32(v, zero)));
      per = 4;
    }
    const uint64_t some = (uint64_t)(~none & ((1u << per) - 1u));
    out |= some << ((k / 4) * per);
  }
#else
  const uint32_t full = P == 32 ? 0xFFFFFFFFu : ((1u << P) - 1u);
  for (int i = 0; i < 64; ++i) {
    const int64_t bit = (int64_t)(first + i) * P;
    if ((bit >> 5) >= row_words) break;
    if ((any_w[bit >> 5] >> (bit & 31)) & full) out |= 1ull << i;
  }
#endif
  return out;
}

struct Unit {
  int32_t req, kv_head, row0, nrows, page_begin, page_end;
  // shared-prefix cascade (defaults: a plain unit)
  int32_t x_slot0 = -1, x_nslots = 0, x_row0 = 0;  // cascade partials that cover this unit's rows
  bool force_partial = false;                      // write fp32 partials even when the unit is not cut
  bool cascade = false;                            // the unit IS a cascade piece: slots, but no merge group of its own
};
typedef std::vector<std::pair<int32_t, int32_t>> UnitSlots;  // per unit: (first slot, slots), (-1, 0) if none

PieItem make_item(const Unit& u, int32_t page_begin, int32_t page_end) {
  PieItem it{};
  it.req = u.req;
  it.kv_head = u.kv_head;
  it.row0 = u.row0;
  it.nrows = u.nrows;
  it.page_begin = page_begin;
  it.page_end = page_end;
  it.partial_slot = -1;
  return it;
}

// Give each of `grid` CTAs (or warps) a share of the page visits of `units`.
//  * Many units, none of them large against a share: whole units are dealt out in order, each to
//    the least-loaded CTA (equal units => round robin).  Units that are neighbours in the batch
//    (heads of one request, branches that share a prefix) then run at the same time on different
//    SMs, so shared pages are fetched from HBM once and served from L2 afterwards; nothing is
//    split, so nothing needs merging.
//  * Otherwise: contiguous equal shares; a unit cut by a share boundary becomes several items
//    whose fp32 partials are merged.
void partition(const std::vector<Unit>& units, int grid_max, int min_pages_per_cta, int slot_rows,
               bool allow_whole_units, PieLaunchList& ll, UnitSlots* slots_out = nullptr) {
  if (slots_out) slots_out->assign(units.size(), std::make_pair(-1, 0));
  ll.items.clear();
  ll.merges.clear();
  ll.cta_ptr.clear();
  ll.n_slots = 0;
  ll.slot_rows = slot_rows;
  ll.grid = 0;
  ll.n_static = 0;
  if (units.empty()) return;
  int64_t W = 0, max_unit = 0;
  for (const Unit& u : units) {
    W += u.page_end - u.page_begin;
    max_unit = std::max<int64_t>(max_unit, u.page_end - u.page_begin);
  }
  const int grid = (int)std::min<int64_t>(grid_max, std::max<int64_t>(1, W / std::max(1, min_pages_per_cta)));
  ll.grid = grid;

  // Whole units also when there are only a few per CTA (or fewer units than CTAs), as long as dealing them out
  // (largest first then) leaves the fullest CTA within 12 % of the average or within 200 page visits (~45 us of
  // a row-tile CTA) of it: a cut unit costs fp32 partials of up to 256 rows, more and shorter items and the merge
  // launch, which on a short launch is more than that imbalance (8 prefill chunks of 512 tokens: 137 -> 78 us;
  // one prompt of 2,048 tokens: 90 -> 46 us although only 64 of 148 CTAs get a unit).
  const bool many_small = (int64_t)units.size() >= 4 * (int64_t)grid && max_unit * 8 <= W / grid;
  const bool few_whole = !many_small && allow_whole_units && W > 0;
  if (allow_whole_units && (many_small || few_whole)) {
    // least-loaded-first list scheduling (binary heap keyed on (load, cta)), then a counting sort
    std::vector<std::pair<int64_t, int>> heap(grid);
    for (int c = 0; c < grid; ++c) heap[c] = {0, c};
    auto cmp = [](const std::pair<int64_t, int>& a, const std::pair<int64_t, int>& b) { return a > b; };
    std::make_heap(heap.begin(), heap.end(), cmp);
    std::vector<int32_t> owner(units.size());
    std::vector<int32_t> order(units.size());
    for (size_t k = 0; k < units.size(); ++k) order[k] = (int32_t)k;
    if (few_whole)   // largest first (stable: equal units keep the batch order)
      std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
        return units[a].page_end - units[a].page_begin > units[b].page_end - units[b].page_begin;
      });
    ll.cta_ptr.assign(grid + 1, 0);
    int64_t max_load = 0;
    for (size_t o = 0; o < units.size(); ++o) {
      const size_t k = (size_t)order[o];
      std::pop_heap(heap.begin(), heap.end(), cmp);
      auto& top = heap.back();
      owner[k] = top.second;
      ++ll.cta_ptr[top.second + 1];
      top.first += std::max<int64_t>(1, units[k].page_end - units[k].page_begin);
      max_load = std::max(max_load, top.first);
      std::push_heap(heap.begin(), heap.end(), cmp);
    }
    if (few_whole && max_load * grid * 100 > W * 112 && max_load > W / grid + 200) goto contiguous;   // too uneven: cut the units instead
    for (int c = 0; c < grid; ++c) ll.cta_ptr[c + 1] += ll.cta_ptr[c];
    std::vector<int32_t> fill(ll.cta_ptr.begin(), ll.cta_ptr.end() - 1);
    ll.items.resize(units.size());
    for (size_t k = 0; k < units.size(); ++k) {
      const Unit& u = units[k];
      PieItem it = make_item(u, u.page_begin, u.page_end);
      if (u.force_partial || u.cascade) {
        it.partial_slot = ll.n_slots;
        if (slots_out) (*slots_out)[k] = {ll.n_slots, 1};
        if (!u.cascade) ll.merges.push_back(PieMerge{u.req, u.kv_head, u.row0, u.nrows, ll.n_slots, 1, u.x_slot0, u.x_nslots, u.x_row0});
        ++ll.n_slots;
      }
      ll.items[fill[owner[k]]++] = it;
    }
    return;
  }

contiguous:
  ll.cta_ptr.clear();
  // Contiguous shares.  Walking the units in order visits the shares in order too, so the items
  // come out already grouped by CTA; share c covers page visits [c W / grid, (c + 1) W / grid),
  // and its end is recomputed only when the walk crosses it (no division per piece).
  ll.items.reserve(units.size() + grid);
  ll.merges.reserve(std::min<size_t>(units.size(), (size_t)grid));
  ll.cta_ptr.reserve(grid + 1);
  ll.cta_ptr.push_back(0);
  int cur = 0;  // CTA whose item range is open
  auto open_cta = [&](int c) {
    while (cur < c) {
      ll.cta_ptr.push_back((int32_t)ll.items.size());
      ++cur;
    }
  };
  int c = 0;                                             // share that holds the walk's position
  // end of share c = floor((c + 1) W / grid) = (c + 1) q + floor((c + 1) r / grid): stepped, one division per list
  const int64_t q_share = W / grid, r_share = W % grid;
  int64_t c_end = grid == 1 ? W : q_share, acc = r_share;
  auto advance_to = [&](int64_t x) {                     // make c the share that holds page visit x
    while (c + 1 < grid && x >= c_end) {
      ++c;
      acc += r_share;
      c_end += q_share;
      if (acc >= grid) {
        acc -= grid;
        ++c_end;
      }
      if (c + 1 == grid) c_end = W;
    }
  };
  int64_t off = 0;
  for (size_t ui = 0; ui < units.size(); ++ui) {
    const Unit& u = units[ui];
    const int64_t n = u.page_end - u.page_begin;
    if (n == 0) {
      advance_to(std::min(off, W > 0 ? W - 1 : 0));
      open_cta(std::max(cur, c));
      ll.items.push_back(make_item(u, u.page_begin, u.page_begin));
      continue;
    }
    const int first_item = (int)ll.items.size();
    int64_t x = off;
    while (x < off + n) {  // pieces: cut at share boundaries strictly inside (off, off+n)
      advance_to(x);
      int64_t end = c_end;
      if (end <= x) end = x + 1;
      end = std::min(end, off + n);
      open_cta(c);
      ll.items.push_back(make_item(u, (int32_t)(u.page_begin + (x - off)), (int32_t)(u.page_begin + (end - off))));
      x = end;
    }
    const int np = (int)ll.items.size() - first_item;
    if (np > 1 || u.force_partial || u.cascade) {
      for (int k = 0; k < np; ++k) ll.items[first_item + k].partial_slot = ll.n_slots + k;
      if (slots_out) (*slots_out)[ui] = {ll.n_slots, np};
      if (!u.cascade) ll.merges.push_back(PieMerge{u.req, u.kv_head, u.row0, u.nrows, ll.n_slots, np, u.x_slot0, u.x_nslots, u.x_row0});
      ll.n_slots += np;
    }
    off += n;
  }
  open_cta(grid - 1);
  ll.cta_ptr.push_back((int32_t)ll.items.size());
}

// Split-KV decode, short launches: fixed shares with block-local merges.  Whole units are first
// dealt to thread blocks (largest first, each to the least-loaded block, then units are moved from
// the fullest block to the emptiest while that lowers the maximum); inside a block its units'
// page visits are cut into one contiguous equal share per warp.  A unit cut by a share boundary
// therefore has all its pieces in one block, and the kernel merges them itself (PIE_ITEM_LOCAL_*):
// no partial needs the merge launch.  Returns false (and leaves `ll` unusable) when whole units
// cannot be dealt evenly enough - few or very unequal units - where cutting them across blocks
// balances better than the merge launch costs.
bool partition_local(const std::vector<Unit>& units, int ctas_max, int NW, int min_pages_per_warp, int slot_rows,
                     PieLaunchList& ll) {
  ll.merges.clear();
  ll.n_slots = 0;
  ll.slot_rows = slot_rows;
  ll.grid = 0;
  ll.n_static = 0;
  if (units.empty()) {
    ll.items.clear();
    ll.cta_ptr.clear();
    return true;
  }
  auto size_of = [&](int32_t k) { return (int64_t)std::max(1, units[k].page_end - units[k].page_begin); };
  int64_t W = 0, largest = 0;
  for (size_t k = 0; k < units.size(); ++k) {
    W += size_of((int32_t)k);
    largest = std::max(largest, size_of((int32_t)k));
  }
  const int n_ctas = (int)std::min<int64_t>(ctas_max, std::max<int64_t>(1, W / std::max(1, min_pages_per_warp * NW)));
  // (some block holds the largest unit whole: when that alone is beyond what the test at the end accepts, there is
  //  nothing to deal - the common case of a few long requests)
  if (largest * n_ctas * 100 > W * 108 && largest > W / n_ctas + 100) return false;
  // Largest first.  Units arrive in runs of equal size (the kv heads of one request), so the runs
  // are sorted, not the units: equivalent to a stable sort of the units by size, descending.
  const int n_units = (int)units.size();
  std::vector<uint64_t> runs;   // (~size) << 32 | first unit of the run
  runs.reserve(n_units / 4 + 1);
  for (int k = 0; k < n_units;) {
    int e = k + 1;
    while (e < n_units && size_of(e) == size_of(k)) ++e;
    runs.push_back(((uint64_t)(0xFFFFFFFFu - (uint32_t)size_of(k)) << 32) | (uint32_t)k);
    k = e;
  }
  std::sort(runs.begin(), runs.end());
  // Min-heap of (load << 16 | block) keys; dealing a unit replaces the top key and sifts it down.
  std::vector<uint64_t> heap(n_ctas);
  for (int c = 0; c < n_ctas; ++c) heap[c] = (uint64_t)c;   // all loads zero: already a heap
  std::vector<int64_t> load(n_ctas, 0);
  std::vector<int32_t> head(n_ctas, -1), next(n_units, -1);   // members of a block: singly linked lists
  for (uint64_t run : runs) {
    const int k0 = (int)(uint32_t)run;
    const int64_t sz = size_of(k0);
    for (int k = k0; k < n_units && size_of(k) == sz; ++k) {
      const int c = (int)(heap[0] & 0xFFFF);
      next[k] = head[c];
      head[c] = k;
      load[c] += sz;
      const uint64_t key = ((uint64_t)load[c] << 16) | (uint64_t)c;
      int i = 0;
      for (;;) {   // sift down
        int ch = 2 * i + 1;
        if (ch >= n_ctas) break;
        if (ch + 1 < n_ctas && heap[ch + 1] < heap[ch]) ++ch;
        if (heap[ch] >= key) break;
        heap[i] = heap[ch];
        i = ch;
      }
      heap[i] = key;
    }
  }
  // refinement: move a unit from the fullest block to the emptiest one while that lowers the maximum
  for (int iter = 0; iter < 48; ++iter) {
    int hi = 0, lo = 0;
    for (int c = 1; c < n_ctas; ++c) {
      if (load[c] > load[hi]) hi = c;
      if (load[c] < load[lo]) lo = c;
    }
    if (load[hi] * n_ctas * 100 <= W * 101) break;   // within 1 % of the average: good enough
    const int64_t gap = load[hi] - load[lo];
    int best = -1, best_prev = -1;
    int64_t best_sz = 0;
    for (int k = head[hi], prev = -1; k >= 0; prev = k, k = next[k]) {   // the largest unit that still leaves `lo` below the old maximum
      const int64_t sz = size_of(k);
      if (sz < gap && sz > best_sz) {
        best = k;
        best_prev = prev;
        best_sz = sz;
      }
    }
    if (best < 0) break;
    if (best_prev < 0) head[hi] = next[best];
    else next[best_prev] = next[best];
    next[best] = head[lo];
    head[lo] = best;
    load[hi] -= best_sz;
    load[lo] += best_sz;
  }
  int64_t max_load = 0;
  for (int c = 0; c < n_ctas; ++c) max_load = std::max(max_load, load[c]);
  // the fullest block may hold up to 8 % or 100 page visits above the average: beyond that, cutting units across blocks
  // and paying the merge launch (+4-5 us on a 55 us launch) is faster (batches at 6 % measured 58.9 vs 60.9 us, at 7 %
  // 60.9 vs 65.8 us; 32 and 48 requests, inside the 100 visits: 37.3 vs 40.2 and 46.5 vs 51.1 us; 16 requests and fewer
  // lose with whole units: too few blocks get one)
  if (max_load * n_ctas * 100 > W * 108 && max_load > W / n_ctas + 100) return false;

  // (items and warp ranges are written through plain pointers into arrays sized for the worst case,
  //  every unit whole plus one extra piece per warp; a reused plan keeps the arrays, and every field
  //  of an item is written here or when the request records are copied in, so nothing is cleared)
  ll.items.resize(units.size() + (size_t)n_ctas * NW);
  ll.cta_ptr.resize((size_t)n_ctas * NW + 1);
  PieItem* const items = ll.items.data();
  int32_t* const ptr = ll.cta_ptr.data();
  int32_t n_items = 0, n_ptr = 0, n_slots = 0;
  ptr[n_ptr++] = 0;
  auto emit = [&](const Unit& u, int32_t page_begin, int32_t page_end) {
    PieItem& it = items[n_items++];
    it.req = u.req;
    it.kv_head = u.kv_head;
    it.row0 = u.row0;
    it.nrows = u.nrows;
    it.page_begin = page_begin;
    it.page_end = page_end;
    it.partial_slot = -1;
    it.flags = 0;
  };
  std::vector<int32_t> members;
  for (int c = 0; c < n_ctas; ++c) {
    members.clear();
    for (int k = head[c]; k >= 0; k = next[k]) members.push_back(k);
    std::sort(members.begin(), members.end());      // batch order inside a block
    const int64_t Wc = load[c];
    const int nw = (int)std::min<int64_t>(NW, std::max<int64_t>(1, Wc / std::max(1, min_pages_per_warp)));
    int w = 0;                                      // warp whose item range is open
    // share w ends at floor((w + 1) Wc / nw) = (w + 1) q + floor((w + 1) rem / nw): stepped, one division per block
    const int64_t q_share = Wc / nw, rem_share = Wc % nw;
    int64_t w_end = q_share, acc = rem_share, off = 0;
    int local_groups = 0;
    auto advance_to = [&](int64_t x) {
      while (w + 1 < nw && x >= w_end) {
        ptr[n_ptr++] = n_items;
        ++w;
        acc += rem_share;
        w_end += q_share;
        if (acc >= nw) {
          acc -= nw;
          ++w_end;
        }
      }
    };
    for (int32_t ui : members) {
      const Unit& u = units[ui];
      const int64_t n = size_of(ui);
      const int first_item = n_items;
      if (u.page_end == u.page_begin) {
        advance_to(off);
        emit(u, u.page_begin, u.page_begin);
      } else {
        int64_t x = off;
        while (x < off + n) {
          advance_to(x);
          const int64_t end = std::min(std::max(w_end, x + 1), off + n);
          emit(u, (int32_t)(u.page_begin + (x - off)), (int32_t)(u.page_begin + (end - off)));
          x = end;
        }
      }
      const int np = n_items - first_item;
      if (np > 1) {   // (at most NW - 1 cut units per block, np <= NW)
        for (int k = 0; k < np; ++k) {
          PieItem& it = items[first_item + k];
          it.partial_slot = n_slots + k;
          it.flags |= PIE_ITEM_LOCAL_PIECE | (k == 0 ? PIE_ITEM_LOCAL_MERGER : 0u) | PIE_ITEM_LOCAL_BITS(local_groups, np);
        }
        n_slots += np;
        ++local_groups;
      }
      off += n;
    }
    for (; w < NW; ++w) ptr[n_ptr++] = n_items;   // close this block's warps (idle ones: empty ranges)
  }
  ll.items.resize((size_t)n_items);
  ll.n_slots = n_slots;
  ll.grid = n_ctas * NW;
  return true;
}

// Block-local merge groups (PIE_ITEM_LOCAL_*) all of whose pieces are the last items of their warps leave
// their partials in shared memory: mark them.  `ll.cta_ptr` holds one item range per warp; the pieces of a
// group are consecutive items, the merging one first.
void mark_smem_groups(PieLaunchList& ll) {
  const int n_w = (int)ll.cta_ptr.size() - 1;
  auto is_last = [&](int32_t idx, int& w) {   // (groups come in warp order: w only moves forward)
    while (w < n_w && ll.cta_ptr[w + 1] <= idx) ++w;
    return w < n_w && ll.cta_ptr[w + 1] == idx + 1;
  };
  int w = 0;
  for (size_t k = 0; k < ll.items.size(); ++k) {
    const uint32_t f = ll.items[k].flags;
    if (!(f & PIE_ITEM_LOCAL_MERGER)) continue;
    const int np = (int)PIE_ITEM_LOCAL_NP(f);
    bool all_last = k + np <= ll.items.size();
    int wk = w;
    for (int c = 0; c < np && all_last; ++c) all_last = is_last((int32_t)(k + c), wk);
    w = wk;
    if (all_last)
      for (int c = 0; c < np; ++c) ll.items[k + c].flags |= PIE_ITEM_LOCAL_SMEM;
  }
}

// Split-KV decode: cut every unit into chunks that the warps of the grid take from a global
// counter at run time.  Units in the first 80 % of the page visits get large chunks (about a
// third of a warp's fair share), the rest small ones, and the large chunks come first in the
// list, so the end of the launch is filled with short pieces of work.
void chunk_units(const std::vector<Unit>& units, int n_warps, PieLaunchList& ll) {
  if (units.empty()) ll.items.clear();
  ll.merges.clear();
  ll.cta_ptr.clear();
  ll.n_slots = 0;
  ll.slot_rows = 1;
  ll.grid = 0;
  ll.n_static = 0;
  if (units.empty()) return;
  int64_t W = 0;
  for (const Unit& u : units) {
    W += u.page_end - u.page_begin;
    ll.slot_rows = std::max(ll.slot_rows, u.nrows);
  }
  const int64_t share = std::max<int64_t>(1, W / std::max(1, n_warps));
  const int c_big = (int)std::min<int64_t>(128, std::max<int64_t>(4, share / 3));
  const int c_small = std::min(16, std::max(2, c_big / 4));
  const int64_t tail_start = W - W / 5;
  // first pass: how many large and small chunks there will be (the small ones go behind the large ones)
  size_t n_big = 0, n_small = 0, n_groups = 0;
  {
    int64_t off = 0;
    for (const Unit& u : units) {
      const int n = u.page_end - u.page_begin;
      const bool tail = off >= tail_start;
      const int c = tail ? c_small : c_big;
      const int nchunks = (n + c - 1) / c;
      (tail ? n_small : n_big) += (size_t)nchunks;
      n_groups += (nchunks > 1 || u.force_partial) ? 1 : 0;
      off += n;
    }
  }
  ll.items.resize(n_big + n_small);   // (every field of an item is written here or when the request records are copied in)
  ll.merges.reserve(n_groups);
  PieItem* big = ll.items.data();
  PieItem* small = ll.items.data() + n_big;
  int64_t off = 0;
  for (const Unit& u : units) {
    const int n = u.page_end - u.page_begin;
    const bool tail = off >= tail_start;
    const int c = tail ? c_small : c_big;
    const int nchunks = (n + c - 1) / c;
    PieItem*& dst = tail ? small : big;
    const bool partial = nchunks > 1 || u.force_partial;
    // chunks of equal size (+-1 page): chunk k covers [floor(n k / nchunks), floor(n (k + 1) / nchunks)), stepped without divisions
    const int base = nchunks ? n / nchunks : 0, rem = nchunks ? n % nchunks : 0;
    int bgn = 0, acc = 0;
    for (int k = 0; k < nchunks; ++k) {
      int end = bgn + base;
      acc += rem;
      if (acc >= nchunks) {
        acc -= nchunks;
        ++end;
      }
      PieItem& it = *dst++;
      it.req = u.req;
      it.kv_head = u.kv_head;
      it.row0 = u.row0;
      it.nrows = u.nrows;
      it.page_begin = u.page_begin + bgn;
      it.page_end = u.page_begin + end;
      it.partial_slot = partial ? ll.n_slots + k : -1;
      it.flags = 0;
      bgn = end;
    }
    if (partial) {
      ll.merges.push_back(PieMerge{u.req, u.kv_head, u.row0, u.nrows, ll.n_slots, nchunks, u.x_slot0, u.x_nslots, u.x_row0});
      ll.n_slots += nchunks;
    }
    off += n;
  }
  ll.grid = (int)std::min<int64_t>(n_warps, (int64_t)ll.items.size());
}

}  // namespace

static int build_plan_core(pie_ctx* ctx, const pie_batch_desc* b, pie_plan* plan);

// Scratch pages a plan holds for requests without output KvPages go back to the free list.
void pie_free_pages(pie_ctx* ctx, const std::vector<int32_t>& ids) {
  for (int32_t id : ids) {
    if (ctx->page_mask[id] != 0xFFFFFFFFu) {
      ctx->page_mask[id] = 0xFFFFFFFFu;
      --ctx->n_masked_pages;
    }
    ctx->allocated[id] = 0;
    ctx->free_list.push_back(id);
  }
}

void pie_plan_release_scratch(pie_plan* plan) {
  pie_free_pages(plan->ctx, plan->scratch_pages);
  plan->scratch_pages.clear();
  plan->pre_copies.clear();
}

// Requests WITHOUT output KvPages (Section 4.2: a forward call takes input KvPages and / or Embeds and fills
// output Embeds and / or KvPages; `forward(kv, iemb[-1:], oemb)` in its listing): the new rows are attended
// but must not land in the caller's pages.  The kernels read K/V from pool pages only, so such a request
// gets pages of the library's own for the lifetime of the plan: the rows of a partly filled last input page
// are copied into the first of them (a token-range page copy that pie_forward runs before the append), the
// new rows are appended behind, and the request's page list becomes  full input pages ++ scratch pages.
// Logical positions do not change, so masks and inferred causality stay as they are.
int pie_build_plan(pie_ctx* ctx, const pie_batch_desc* b, pie_plan* plan) {
  plan->ctx = ctx;
  pie_plan_release_scratch(plan);   // (a reused plan object)
  const int R = b->num_requests;
  bool any = false;
  if (b->no_store && R > 0 && R <= ctx->cfg.max_requests)
    for (int r = 0; r < R; ++r) any = any || b->no_store[r] != 0;
  if (!any) return build_plan_core(ctx, b, plan);
  if (!b->qo_indptr || !b->page_indptr || !b->last_page_len || b->qo_indptr[0] != 0 || b->page_indptr[0] != 0) return PIE_ERR_INVALID;
  const int P = ctx->cfg.page_size;
  pie_reclaim_pages(ctx, false);   // pages of earlier such batches whose forward is over
  std::vector<int32_t>& ip = plan->int_page_indptr;
  std::vector<int32_t>& idx = plan->int_page_indices;
  std::vector<int32_t>& lpl = plan->int_last_page_len;
  ip.assign(1, 0);
  idx.clear();
  lpl.clear();
  int rc = PIE_OK;
  for (int r = 0; r < R && rc == PIE_OK; ++r) {
    const int q_len = b->qo_indptr[r + 1] - b->qo_indptr[r];
    const int np = b->page_indptr[r + 1] - b->page_indptr[r];
    if (q_len < 1 || np < 0 || (np > 0 && !b->page_indices)) {
      rc = PIE_ERR_INVALID;
      break;
    }
    const int32_t* pages = b->page_indices + b->page_indptr[r];
    if (!b->no_store[r]) {
      idx.insert(idx.end(), pages, pages + np);
      lpl.push_back(b->last_page_len[r]);
    } else {
      const int last_in = np > 0 ? b->last_page_len[r] : P;
      if (last_in < 1 || last_in > P) {
        rc = PIE_ERR_INVALID;
        break;
      }
      for (int k = 0; k < np; ++k)
        if (pages[k] < 0 || pages[k] >= ctx->cfg.num_pages || !ctx->allocated[pages[k]]) rc = PIE_ERR_BAD_PAGE;
      if (rc != PIE_OK) break;
      const int carry = (np > 0 && last_in < P) ? last_in : 0;   // rows of the partly filled last input page
      const int keep = carry ? np - 1 : np;                      // input pages that stay in the list
      const int n_scratch = (carry + q_len + P - 1) / P;
      if ((size_t)n_scratch > ctx->free_list.size()) pie_reclaim_pages(ctx, true);   // wait for the forwards that still hold borrowed pages
      if ((size_t)n_scratch > ctx->free_list.size()) {
        rc = PIE_ERR_NO_PAGES;
        break;
      }
      idx.insert(idx.end(), pages, pages + keep);
      for (int k = 0; k < n_scratch; ++k) {
        const int32_t id = ctx->free_list.back();
        ctx->free_list.pop_back();
        ctx->allocated[id] = 1;
        plan->scratch_pages.push_back(id);
        idx.push_back(id);
        if (k == 0 && carry) {
          plan->pre_copies.insert(plan->pre_copies.end(), {pages[np - 1], id, 0, 0, carry});
          const uint32_t pm = ctx->page_mask[pages[np - 1]];   // a page mask travels with the copied rows
          if (pm != 0xFFFFFFFFu) {
            ctx->page_mask[id] = pm | ~((1u << carry) - 1u);
            if (ctx->page_mask[id] != 0xFFFFFFFFu) ++ctx->n_masked_pages;
          }
        }
      }
      lpl.push_back(carry + q_len - (n_scratch - 1) * P);
    }
    ip.push_back((int32_t)idx.size());
  }
  if (rc == PIE_OK) {
    pie_batch_desc bb = *b;
    bb.page_indptr = ip.data();
    bb.page_indices = idx.data();
    bb.last_page_len = lpl.data();
    bb.no_store = nullptr;
    rc = build_plan_core(ctx, &bb, plan);
    // (the fused append would be fine, but the copies must run first: keep the separate launches in order)
  }
  if (rc != PIE_OK) pie_plan_release_scratch(plan);
  return rc;
}

static int build_plan_core(pie_ctx* ctx, const pie_batch_desc* b, pie_plan* plan) {
  const pie_config& cfg = ctx->cfg;
  const int P = cfg.page_size, G = ctx->G;
  const int R = b->num_requests;
  if (R < 0) return PIE_ERR_INVALID;
  if (R > cfg.max_requests) return PIE_ERR_BATCH_TOO_LARGE;
  if (R > 0 && (!b->qo_indptr || !b->page_indptr || !b->page_indices || !b->last_page_len))
    return PIE_ERR_INVALID;
  plan->R = R;
  plan->flags = b->flags;
  plan->T = 0;
  if (R == 0) {
    plan->info = pie_plan_info{};
    return PIE_OK;
  }
  if (b->qo_indptr[0] != 0 || b->page_indptr[0] != 0) return PIE_ERR_INVALID;
  for (int r = 0; r < R; ++r) {
    if (b->qo_indptr[r + 1] <= b->qo_indptr[r]) return PIE_ERR_INVALID;      // q_len >= 1
    if (b->page_indptr[r + 1] <= b->page_indptr[r]) return PIE_ERR_INVALID;  // >= 1 page
  }
  const int T = b->qo_indptr[R];
  if (T > cfg.max_query_tokens) return PIE_ERR_BATCH_TOO_LARGE;
  plan->T = T;

  // ---- per-request validation (the passes over the page lists - here and in the next step - run on the
  // context's worker threads when the batch lists many pages; the first failing request, in batch order,
  // decides the error)
  plan->reqs.assign(R, PieReq{});
  const bool many_pages = b->page_indptr[R] >= 65536;
  std::vector<int32_t>& req_note = plan->req_note;
  req_note.assign((size_t)R, PIE_OK);
  pie_run_tasks(ctx, R, many_pages, [&](int r) {
    const int q_len = b->qo_indptr[r + 1] - b->qo_indptr[r];
    const int np = b->page_indptr[r + 1] - b->page_indptr[r];
    const int last = b->last_page_len[r];
    const int64_t kv_len64 = (int64_t)(np - 1) * P + last;
    if (last < 1 || last > P || kv_len64 > 0x3FFFFFFF || kv_len64 < q_len ||
        (b->out_len && (b->out_len[r] < 0 || b->out_len[r] > q_len))) {
      req_note[r] = PIE_ERR_INVALID;
      return;
    }
    const int32_t* pages = b->page_indices + b->page_indptr[r];
    uint32_t max_id = 0;   // (negative ids wrap to large values)
    for (int k = 0; k < np; ++k) max_id = std::max(max_id, (uint32_t)pages[k]);
    if (max_id >= (uint32_t)cfg.num_pages) {
      req_note[r] = PIE_ERR_BAD_PAGE;
      return;
    }
    // (whether every page is allocated is looked up further down, in the same pass over the page lists that looks
    //  for pages another request of the batch writes: one random access per listed page instead of two)
    PieReq& q = plan->reqs[r];
    q.q_start = b->qo_indptr[r];
    q.q_len = q_len;
    q.kv_len = (int32_t)kv_len64;
    q.last_logical = np - 1;
    q.last_page_len = last;
  });
  for (int r = 0; r < R; ++r)
    if (req_note[r] != PIE_OK) return req_note[r];

  bool cross_read = false;  // some request lists a page that another request of the batch appends to
  // ---- conflict rule: no slot is written twice, and no request reads a slot that a later request
  // of the batch writes (rows appended by an earlier request are visible: append precedes attention)
  {
    std::vector<int32_t> touched;
    struct SharedWrite { int32_t page, req; uint32_t mask; };
    std::vector<SharedWrite> shared;  // pages written by more than one request: who wrote which slots
    int status = PIE_OK;
    cross_read = false;
    auto slot_mask = [&](int lo, int hi) -> uint32_t {  // bits [lo, hi)
      uint32_t m = (hi >= 32) ? 0xFFFFFFFFu : ((1u << hi) - 1u);
      return m & ~((1u << lo) - 1u);
    };
    for (int r = 0; r < R && status == PIE_OK; ++r) {
      const PieReq& q = plan->reqs[r];
      const int32_t* pages = b->page_indices + b->page_indptr[r];
      const int first = q.kv_len - q.q_len;
      for (int lp = first / P; lp <= q.last_logical; ++lp) {
        int lo = std::max(first - lp * P, 0), hi = std::min(q.kv_len - lp * P, P);
        uint32_t m = slot_mask(lo, hi);
        int32_t pg = pages[lp];
        if (ctx->wmask[pg] & m) { status = PIE_ERR_CONFLICT; break; }
        if (ctx->wmask[pg] == 0) {
          touched.push_back(pg);
          ctx->writer[pg] = r;
          ctx->allocated[pg] |= 2;   // "written in this batch", next to the allocation flag (cleared again below)
        } else {
          if (ctx->writer[pg] >= 0) {  // second writer of this page: start the per-writer record
            shared.push_back(SharedWrite{pg, ctx->writer[pg], ctx->wmask[pg]});
            ctx->writer[pg] = -2;
          }
          shared.push_back(SharedWrite{pg, r, m});
        }
        ctx->wmask[pg] |= m;
      }
    }
    // one look per listed page: allocated?  written by a request of this batch?
    // (note bit 0: some page is not allocated; bit 1: some page the request only reads is written by somebody)
    pie_run_tasks(ctx, R, many_pages, [&](int r) {
      const PieReq& q = plan->reqs[r];
      const int32_t* pages = b->page_indices + b->page_indptr[r];
      const int first_written = (q.kv_len - q.q_len) / P;
      uint8_t all_a = 0xFF, any_a = 0;
      for (int lp = 0; lp < first_written; ++lp) {
        const uint8_t a = ctx->allocated[pages[lp]];
        all_a &= a;
        any_a |= a;
      }
      for (int lp = first_written; lp <= q.last_logical; ++lp) all_a &= ctx->allocated[pages[lp]];
      req_note[r] = ((all_a & 1) ? 0 : 1) | ((any_a & 2) ? 2 : 0);
    });
    bool bad_page = false;   // (reported before a conflict, as when the pages were checked first)
    for (int r = 0; r < R && !bad_page; ++r) {
      const PieReq& q = plan->reqs[r];
      const int32_t* pages = b->page_indices + b->page_indptr[r];
      const int first_written = (q.kv_len - q.q_len) / P;
      if (req_note[r] & 1) {
        bad_page = true;
        break;
      }
      if (status != PIE_OK) continue;
      // (common case: none of the pages the request only reads is written by anybody)
      const bool any_written = (req_note[r] & 2) != 0;
      for (int lp = any_written ? 0 : first_written; lp <= q.last_logical; ++lp) {
        int32_t pg = pages[lp];
        uint32_t w = ctx->wmask[pg];
        if (w == 0) continue;
        if (ctx->writer[pg] == r) {
          // the request's own page: listed a second time below the rows it appends, the copy is read by
          // another warp than the one that would write the new row in a fused append
          if (lp < first_written) cross_read = true;
          continue;
        }
        cross_read = true;  // a page one request appends to is in another request's list
        if (ctx->writer[pg] >= 0 && ctx->writer[pg] < r) continue;  // written by an earlier request: visible
        uint32_t rd = slot_mask(0, lp == q.last_logical ? q.last_page_len : P);
        if (ctx->writer[pg] == -2) {  // several writers: only slots written by LATER requests conflict
          w = 0;
          for (const SharedWrite& sw : shared)
            if (sw.page == pg && sw.req > r) w |= sw.mask;
        }
        if (w & rd) { status = PIE_ERR_CONFLICT; break; }
      }
    }
    for (int32_t pg : touched) {
      ctx->wmask[pg] = 0;
      ctx->writer[pg] = -1;
      ctx->allocated[pg] &= 1;
    }
    if (bad_page) return PIE_ERR_BAD_PAGE;
    if (status != PIE_OK) return status;
  }

  // ---- masks: pack explicit ones, classify pages, build the kept-page list.
  // Word offsets are fixed first; then requests are independent, so large batches (tens of MB of
  // mask bytes) are packed by several host threads, each writing its own requests' slices.
  plan->kept.clear();
  const uint32_t full_bits = (P >= 32) ? 0xFFFFFFFFu : ((1u << P) - 1u);
  int64_t n_words = 0, mask_bytes_total = 0;
  const bool bits_in = (b->flags & PIE_PLAN_MASK_BITS) != 0;   // the caller packed the masks itself
  for (int r = 0; r < R; ++r) {
    PieReq& q = plan->reqs[r];
    int64_t m0 = 0, m1 = 0;
    if (b->mask_indptr) { m0 = b->mask_indptr[r]; m1 = b->mask_indptr[r + 1]; }
    if (m1 < m0) return PIE_ERR_MASK;
    bool page_masked = false;  // some page of the request carries a mask_kvpage mask
    if (ctx->n_masked_pages > 0) {
      const int32_t* pages = b->page_indices + b->page_indptr[r];
      for (int lp = 0; lp <= q.last_logical && !page_masked; ++lp) page_masked = ctx->page_mask[pages[lp]] != 0xFFFFFFFFu;
    }
    // explicit mask: q_len x kv_len bool bytes, or (PIE_PLAN_MASK_BITS) q_len rows of ceil(kv_len / 32) words
    const int64_t mask_units = bits_in ? (int64_t)q.q_len * ((q.kv_len + 31) / 32) : (int64_t)q.q_len * q.kv_len;
    if (m1 > m0 && (!b->mask || m1 - m0 != mask_units)) return PIE_ERR_MASK;
    if (m1 > m0 || page_masked) {  // the request gets packed mask rows (given, or causal AND page masks)
      q.mask_row_words = ((q.kv_len + 127) / 128) * 4;
      q.mask_word_off = n_words;
      n_words += (int64_t)q.mask_row_words * q.q_len;
      mask_bytes_total += (m1 - m0) * (bits_in ? 4 : 1);
    } else {
      q.mask_row_words = 0;
      q.mask_word_off = 0;
    }
  }
  plan->mask_words.resize((size_t)n_words);   // (every row is written in full below: nothing to clear)
  // every request first writes its kept pages into its own slice of a scratch array (sized for
  // "all pages kept"); the slices are then packed together in request order
  int n_threads = 1;
  if (mask_bytes_total > (4 << 20)) {
    n_threads = pie_host_threads(R);
  }
  // (one thread: the requests are visited in order, so each writes straight behind its predecessor
  //  in the final list and nothing is packed afterwards)
  std::vector<int32_t>& scratch = n_threads > 1 ? plan->kept_scratch : plan->kept;
  scratch.resize(2 * (size_t)b->page_indptr[R]);
  std::atomic<int> bad_mask{0};
  plan->clean_kept.resize(R);
  size_t kept_at = 0;   // single-threaded: pages kept so far
  auto do_request = [&](int r) {
    PieReq& q = plan->reqs[r];
    const int32_t* pages = b->page_indices + b->page_indptr[r];
    const int np = q.last_logical + 1;
    int32_t* kept = scratch.data() + 2 * (n_threads > 1 ? (size_t)b->page_indptr[r] : kept_at);
    int nk = 0, first_flagged = -1;   // (first kept page some row sees only in part: explicit masks)
    if (q.mask_row_words) {
      const int row_words = q.mask_row_words;
      uint32_t* w = plan->mask_words.data() + q.mask_word_off;
      const bool given = b->mask_indptr && b->mask_indptr[r + 1] > b->mask_indptr[r];
      if (given && bits_in) {   // rows of ceil(kv_len / 32) words, LSB first: copied into the 128-bit padded rows
        const int words_in = (q.kv_len + 31) / 32;
        const uint32_t tail = (q.kv_len & 31) ? ((1u << (q.kv_len & 31)) - 1u) : 0xFFFFFFFFu;   // bits past kv_len are ignored
        const uint32_t* src = reinterpret_cast<const uint32_t*>(b->mask) + b->mask_indptr[r];
        for (int i = 0; i < q.q_len; ++i) {
          uint32_t* row = w + (size_t)i * row_words;
          std::memcpy(row, src + (int64_t)i * words_in, (size_t)words_in * 4);
          row[words_in - 1] &= tail;
          for (int k = words_in; k < row_words; ++k) row[k] = 0u;
        }
      } else if (given) {
        const uint8_t* src = b->mask + b->mask_indptr[r];
        for (int i = 0; i < q.q_len; ++i)
          if (!pack_row(src + (int64_t)i * q.kv_len, q.kv_len, w + (size_t)i * row_words, row_words)) bad_mask.store(1);
      } else {  // inferred causal rows, written out because page masks will be ANDed in
        for (int i = 0; i < q.q_len; ++i) {
          const int nbits = q.kv_len - q.q_len + i + 1;  // positions 0 .. lim
          uint32_t* row = w + (size_t)i * row_words;
          int k = 0;
          for (; k < nbits / 32; ++k) row[k] = 0xFFFFFFFFu;
          if (nbits & 31) row[k++] = (1u << (nbits & 31)) - 1u;
          for (; k < row_words; ++k) row[k] = 0u;
        }
      }
      if (ctx->n_masked_pages > 0) {
        for (int lp = 0; lp < np; ++lp) {
          const uint32_t pm = ctx->page_mask[pages[lp]];
          if (pm == 0xFFFFFFFFu) continue;
          const int bit = lp * P;
          const uint32_t clear = ~pm & full_bits;
          for (int i = 0; i < q.q_len; ++i) w[(size_t)i * row_words + (bit >> 5)] &= ~(clear << (bit & 31));
        }
      }
      // OR and AND of all rows, word by word (contiguous passes over the rows), then one look per page
      static thread_local std::vector<uint32_t> col;
      col.resize(2 * (size_t)row_words);
      uint32_t* const any_w = col.data();
      uint32_t* const all_w = col.data() + row_words;
      for (int k = 0; k < row_words; ++k) {
        any_w[k] = 0u;
        all_w[k] = 0xFFFFFFFFu;
      }
      for (int i = 0; i < q.q_len; ++i) {
        const uint32_t* row = w + (size_t)i * row_words;
        for (int k = 0; k < row_words; ++k) {
          any_w[k] |= row[k];
          all_w[k] &= row[k];
        }
      }
      for (int lp0 = 0; lp0 < np; lp0 += 64) {
        // (a page no query row attends to is never fetched: only the others are visited)
        uint64_t some = page_any_bits(any_w, row_words, P, lp0);
        if (np - lp0 < 64) some &= (1ull << (np - lp0)) - 1ull;
        while (some) {
          const int lp = lp0 + __builtin_ctzll(some);
          some &= some - 1;
          const int bit = lp * P;
          const uint32_t all = (all_w[bit >> 5] >> (bit & 31)) & full_bits;
          kept[2 * nk] = pages[lp];
          kept[2 * nk + 1] = (int32_t)((uint32_t)lp | (all == full_bits ? 0u : PIE_KEPT_NEEDS_MASK));
          if (all != full_bits && first_flagged < 0) first_flagged = nk;
          ++nk;
        }
      }
    } else {
      const int lim0 = q.kv_len - q.q_len;  // last position the first query token sees
      for (int lp = 0; lp < np; ++lp) {
        kept[2 * lp] = pages[lp];
        kept[2 * lp + 1] = (int32_t)((uint32_t)lp | (lp * P + P - 1 <= lim0 ? 0u : PIE_KEPT_NEEDS_MASK));
      }
      nk = np;
    }
    q.kept_count = nk;
    plan->clean_kept[r] = first_flagged < 0 ? nk : first_flagged;
    if (n_threads <= 1) {
      q.kept_start = (int32_t)kept_at;
      kept_at += (size_t)nk;
    }
  };
  pie_run_tasks(ctx, R, n_threads > 1, do_request);
  if (bad_mask.load()) return PIE_ERR_MASK;
  if (n_threads <= 1) {
    plan->kept.resize(2 * kept_at);
  } else {
    size_t total = 0;
    for (int r = 0; r < R; ++r) total += (size_t)plan->reqs[r].kept_count;
    plan->kept.resize(2 * total);
    size_t at = 0;
    for (int r = 0; r < R; ++r) {
      PieReq& q = plan->reqs[r];
      q.kept_start = (int32_t)at;
      std::memcpy(plan->kept.data() + 2 * at, scratch.data() + 2 * (size_t)b->page_indptr[r], 8 * (size_t)q.kept_count);
      at += (size_t)q.kept_count;
    }
  }

  // ---- append destinations
  plan->append_dst.resize(T);
  plan->tok_req.resize(T);
  plan->positions.clear();
  if (cfg.rope_theta > 0.f) plan->positions.resize(T);
  for (int r = 0; r < R; ++r) {
    const PieReq& q = plan->reqs[r];
    const int32_t* pages = b->page_indices + b->page_indptr[r];
    for (int i = 0; i < q.q_len; ++i) {
      int pos = q.kv_len - q.q_len + i;
      plan->append_dst[q.q_start + i] = pages[pos / P] * P + pos % P;
      plan->tok_req[q.q_start + i] = r;
      if (cfg.rope_theta > 0.f) {
        const int p_i = b->positions ? b->positions[q.q_start + i] : pos;
        if (p_i < 0) return PIE_ERR_INVALID;
        plan->positions[q.q_start + i] = p_i;
      }
    }
  }

  // ---- output Embeds for the last out_len tokens only (Section 4.2: a call fills output Embeds and / or
  // output KvPages): from here on a request is its attention view - the query tokens that produce an
  // output.  They keep their positions and mask rows (kv_len is unchanged, so the inferred causal limit
  // kv_len - q_len + i of view token i is the one of the original token); a request with out_len 0 is
  // stored and not attended at all.
  bool all_rows_out = true;
  if (b->out_len) {
    for (int r = 0; r < R; ++r) {
      PieReq& q = plan->reqs[r];
      const int skip = q.q_len - b->out_len[r];
      if (skip == 0) continue;
      all_rows_out = false;
      q.q_start += skip;
      q.mask_word_off += (int64_t)skip * q.mask_row_words;
      q.q_len = b->out_len[r];
    }
  }

  // ---- route requests to kernels and partition the work
  // (head groups above 16 - multi-query models - do not fit the split-KV kernel's 16 rows per warp: every request
  //  of such a context has more than 16 rows and runs on the row-tile kernel)
  const bool tiles_ok = (pie_split_supported(ctx) || (pie_tc_supported(ctx) && G > 16)) && !(b->flags & PIE_PLAN_FORCE_SIMPLE);
  std::vector<Unit> split_units, tile_units;
  plan->simple_rows.clear();
  // (8-token pages: the mma.sync row-tile kernel behind PIE_PLAN_NO_TENSOR_TILES has no instantiation, the flag is ignored)
  plan->tile_tc = pie_tc_supported(ctx) && (!(b->flags & PIE_PLAN_NO_TENSOR_TILES) || P == 8);
  const int TILE_ROWS = plan->tile_tc ? 256 : 64;   // two 128-row tcgen05 tiles, or four 16-row warps

  // Shared-prefix cascade: consecutive requests whose page lists start with the same physical
  // pages - parallel samples, beams, branches of one prompt - have their rows gathered and
  // attended to that prefix ONCE, as row tiles of a virtual request on the row-tile kernel; every
  // request then attends only its private pages, and the merge combines the two partials.
  //  * Decode-shaped requests (at most 16 rows): private pages on the split-KV kernel.  The prefix
  //    is read from HBM once per group instead of once per request.
  //  * Requests with more rows that still fill at most half a row tile (a token tree of 32 nodes
  //    under 4 grouped heads: 128 rows): private pages as row-tile items of their own.  Here the
  //    gain is the tile: a lone request would leave half of the 256-row item, and one of the two
  //    softmax warpgroups, without work over the whole prefix.
  // (Requests that fill a row tile on their own, e.g. token trees of 64 nodes, find the shared
  //  pages in L2: gathering them would only add partials.)
  struct Cascade { int32_t first, n, L, vreq; bool big; };
  std::vector<Cascade> cascades;
  std::vector<int32_t> casc_of(R, -1);
  if (tiles_ok && !(b->flags & PIE_PLAN_NO_CASCADE) && all_rows_out) {   // (the gathered rows of a group must be consecutive query tokens)
    const bool always = (b->flags & PIE_PLAN_CASCADE_ALWAYS) != 0;
    const int min_n = always ? 2 : 4, min_L = always ? 1 : 16;
    auto clean_prefix = [&](const PieReq& q) {  // leading kept pages that are fully visible and in place
      int c = 0;
      while (c < q.kept_count - 1 && plan->kept[2 * (size_t)(q.kept_start + c) + 1] == c) ++c;  // (flag bit clear, logical == index)
      return c;
    };
    int64_t saved = 0;
    for (int r = 0; r < R;) {
      const PieReq& q0 = plan->reqs[r];
      const int rows = q0.q_len * G;
      const bool big = rows > 16;
      if (rows == 0 || (big && 2 * rows > TILE_ROWS) || TILE_ROWS % rows != 0 || q0.kept_count < 2 || r + 1 >= R || plan->reqs[r + 1].kept_count < 2 ||
          plan->kept[2 * (size_t)plan->reqs[r + 1].kept_start] != plan->kept[2 * (size_t)q0.kept_start]) {  // (no neighbour with the same first page: no run starts here)
        ++r;
        continue;
      }
      int L = clean_prefix(q0), e = r + 1;
      for (; e < R && L >= min_L; ++e) {
        const PieReq& q = plan->reqs[e];
        if (q.q_len != q0.q_len || q.kept_count < 2) break;
        int c = 0;
        const int cmax = std::min(L, clean_prefix(q));
        while (c < cmax && plan->kept[2 * (size_t)(q.kept_start + c)] == plan->kept[2 * (size_t)(q0.kept_start + c)]) ++c;
        if (c < min_L) break;
        L = c;
      }
      // (a group of larger requests must fill at least one row tile and share at least 1,024 tokens: below that
      //  the partials and the merge cost more than the filled tile gains)
      const bool accept = !big ? (e - r >= min_n && L >= min_L)
                               : (e - r >= 2 && L >= min_L && (always || ((e - r) * rows >= TILE_ROWS && (int64_t)L * P >= 1024)));
      if (accept) {
        cascades.push_back(Cascade{r, e - r, L, 0, big});
        if (!big) saved += (int64_t)(e - r - 1) * L * cfg.num_kv_heads;
        r = e;
      } else {
        ++r;
      }
    }
    // decode-shaped groups are worth a second launch and a merge only when enough page reads disappear
    if (!always && saved < 2048)
      cascades.erase(std::remove_if(cascades.begin(), cascades.end(), [](const Cascade& c) { return !c.big; }), cascades.end());
    for (size_t c = 0; c < cascades.size(); ++c) {
      Cascade& cs = cascades[c];
      const PieReq& q0 = plan->reqs[cs.first];
      PieReq v{};   // the virtual request: all rows of the group, the shared pages, everything visible
      v.q_start = q0.q_start;
      v.q_len = q0.q_len * cs.n;
      v.kv_len = v.q_len + cs.L * P;
      v.kept_start = q0.kept_start;
      v.kept_count = cs.L;
      v.mask_row_words = 0;
      v.mask_word_off = 0;
      v.last_logical = cs.L - 1;
      v.last_page_len = P;
      cs.vreq = (int32_t)plan->reqs.size();
      plan->reqs.push_back(v);
      for (int k = 0; k < cs.n; ++k) casc_of[cs.first + k] = (int32_t)c;
    }
  }
  // Decode units of two adjacent kv heads: the two heads' blocks of a page are neighbours in the pool, so
  // one copy of twice the size brings both, and blocks of 2 - 4 KB are fetched at a visibly lower rate than
  // blocks of 8 KB.  Possible when the rows of both heads fit the 16 rows of a warp for every decode-shaped
  // request of the batch (cascaded requests keep one head per unit: their shared partials are per kv head).
  int hp = 1;
  if (tiles_ok && pie_split_pair_supported(ctx) && cascades.empty() && !(ctx->options[PIE_OPT_NO_FUSION] & 4)) {
    bool any = false, fits = true;
    for (int r = 0; r < R; ++r) {
      const PieReq& q = plan->reqs[r];
      const int rows = q.q_len * G;
      if (rows == 0 || q.kept_count == 0 || rows > 16) continue;
      any = true;
      fits = fits && 2 * rows <= 16;
    }
    if (any && fits) hp = 2;
  }
  std::vector<int32_t> casc_unit0(cascades.size(), 0);  // first tile unit of every cascade
  for (int r = 0; r < R; ++r) {
    const PieReq& q = plan->reqs[r];
    const int rows = q.q_len * G;
    if (rows == 0) continue;               // (stored only: no output row)
    if (!tiles_ok || q.kept_count == 0) {  // (a request with no attendable page only needs zeros / -inf written)
      for (int i = 0; i < q.q_len; ++i)
        for (int h = 0; h < cfg.num_q_heads; ++h) plan->simple_rows.push_back((q.q_start + i) * cfg.num_q_heads + h);
    } else if (rows <= 16) {
      if (casc_of[r] < 0)
        for (int g = 0; g < cfg.num_kv_heads / hp; ++g)   // (hp = 2: g is the pair of kv heads 2g, 2g + 1; rows of the first head, then of the second)
          split_units.push_back(Unit{r, g, 0, rows * hp, q.kept_start, q.kept_start + q.kept_count});
      // (requests of a cascade get their split units below, once the cascade's slots are known)
    } else {
      // (a request of a cascade attends only the pages behind the shared prefix here and writes a partial; the
      //  cascade's slots are added to its merge group once the partition has assigned them)
      const int skip = casc_of[r] >= 0 ? cascades[casc_of[r]].L : 0;
      for (int g = 0; g < cfg.num_kv_heads; ++g)
        for (int row0 = 0; row0 < rows; row0 += TILE_ROWS) {
          int nrows = std::min(TILE_ROWS, rows - row0);
          int end = q.kept_count;
          if (q.mask_row_words == 0) {  // causal: pages beyond the tile's last token are invisible
            int i1 = (row0 + nrows - 1) / G;
            int lim = q.kv_len - q.q_len + i1;
            end = std::min(end, lim / P + 1);
          }
          Unit u{r, g, row0, nrows, q.kept_start + skip, q.kept_start + std::max(end, skip)};
          u.force_partial = skip > 0;
          tile_units.push_back(u);
        }
    }
  }
  for (size_t c = 0; c < cascades.size(); ++c) {
    const Cascade& cs = cascades[c];
    const PieReq& v = plan->reqs[cs.vreq];
    const int vrows = v.q_len * G;
    casc_unit0[c] = (int32_t)tile_units.size();
    for (int g = 0; g < cfg.num_kv_heads; ++g)
      for (int row0 = 0; row0 < vrows; row0 += TILE_ROWS) {
        Unit u{cs.vreq, g, row0, std::min(TILE_ROWS, vrows - row0), v.kept_start, v.kept_start + cs.L};
        u.cascade = true;
        tile_units.push_back(u);
      }
  }
  // SM budget of the two tile kernels.  On request (PIE_OPT_OVERLAP) a mixed batch runs them side
  // by side: the decode kernel is HBM bound and saturates the memory system from roughly 60 % of
  // the SMs, so it keeps at least that many and otherwise a share proportional to its estimated
  // time; the rest go to the tensor-bound prefill / tree kernel.
  int split_sms = ctx->options[PIE_OPT_SPLIT_SMS] > 0 ? std::min(ctx->options[PIE_OPT_SPLIT_SMS], ctx->n_sms) : ctx->n_sms;
  int tile_sms = ctx->options[PIE_OPT_TILE_SMS] > 0 ? std::min(ctx->options[PIE_OPT_TILE_SMS], ctx->n_sms) : ctx->n_sms;
  plan->overlap = false;
  if ((!split_units.empty() || !cascades.empty()) && !tile_units.empty() && plan->tile_tc && ctx->options[PIE_OPT_OVERLAP] != 2 &&
      ctx->n_sms >= 16) {
    if (ctx->options[PIE_OPT_SPLIT_SMS] > 0 && ctx->options[PIE_OPT_TILE_SMS] > 0) {
      plan->overlap = ctx->options[PIE_OPT_OVERLAP] == 1 && split_sms + tile_sms <= ctx->n_sms;   // explicit budgets, on request
    } else {
      // Model: the decode kernel moves `split_bytes` at the chip's copy rate as long as it has about
      // 60 % of the SMs, and proportionally slower below that; the row-tile kernel's time scales with
      // 1 / SMs.  Take the budget that minimises the later finish, and run side by side only if that
      // beats one kernel after the other.
      double split_bytes = 0, tile_flops = 0;
      for (const Unit& u : split_units) split_bytes += (double)(u.page_end - u.page_begin) * hp * 2.0 * P * cfg.head_dim * 2.0;
      for (const Cascade& cs : cascades)   // the private pages of cascaded decode-shaped requests (their split units are made below)
        for (int k = 0; k < (cs.big ? 0 : cs.n); ++k)
          split_bytes += (double)(plan->reqs[cs.first + k].kept_count - cs.L) * cfg.num_kv_heads * 2.0 * P * cfg.head_dim * 2.0;
      for (const Unit& u : tile_units) tile_flops += (double)(u.page_end - u.page_begin) * P * 4.0 * cfg.head_dim * u.nrows;
      const double t_split = split_bytes / 6.4e12, t_tile = tile_flops / 0.76e15;  // whole-chip estimates, seconds (rates measured on the mixed workload: its decode requests alone, its prefill chunks alone)
      const double sat = 0.6 * ctx->n_sms;                                         // SMs that saturate the memory system
      int best_nt = 0;
      double best_t = 1e30;
      // (on its own the planner only takes budgets that leave the decode kernel its saturating share: below it
      //  the model's rates are too rough - one 4,096-token prefill next to 64 decodes ran 8 % slower side by side)
      const int nt_max = ctx->options[PIE_OPT_OVERLAP] == 1 ? ctx->n_sms - 16 : ctx->n_sms - (int)(sat + 0.5);
      for (int nt = 8; nt <= nt_max; nt += 2) {
        const int ns = ctx->n_sms - nt;
        const double ts = t_split * std::max(1.0, sat / ns), tt = t_tile * ctx->n_sms / nt;
        const double t = std::max(ts, tt);
        if (t < best_t) {
          best_t = t;
          best_nt = nt;
        }
      }
      // (automatic only for plain mixed batches: a cascade's row tiles are short gathered-decode items that
      //  the model does not describe - measured 0.133 -> 0.127 ms at best, 0.19 ms with the model's budget)
      if (best_nt > 0 && (ctx->options[PIE_OPT_OVERLAP] == 1 ||
                          (cascades.empty() && best_t < 0.90 * (t_split + t_tile) && t_split + t_tile > 150e-6))) {
        tile_sms = best_nt;
        split_sms = ctx->n_sms - best_nt;
        plan->overlap = true;
      }
    }
  }
  // row tiles first: the cascade pieces get their partial slots, which the split units of the
  // cascaded requests then name as further sources of their merge groups
  UnitSlots tile_slots;
  partition(tile_units, tile_sms, plan->tile_tc ? 32 : 8, TILE_ROWS, true, plan->tile, &tile_slots);
  // merge groups of the larger cascaded requests (row-tile items over their private pages): add the slots of
  // the cascade pieces that hold the same rows
  for (PieMerge& m : plan->tile.merges) {
    if (m.req >= R || casc_of[m.req] < 0) continue;
    const Cascade& cs = cascades[casc_of[m.req]];
    const PieReq& v = plan->reqs[cs.vreq];
    const int tiles_per_head = (v.q_len * G + TILE_ROWS - 1) / TILE_ROWS;
    const int vr0 = (plan->reqs[m.req].q_start - v.q_start) * G + m.row0;   // first virtual row of the group's rows
    const auto& sl = tile_slots[(size_t)casc_unit0[casc_of[m.req]] + (size_t)m.kv_head * tiles_per_head + vr0 / TILE_ROWS];
    m.x_slot0 = sl.first;
    m.x_nslots = sl.second;
    m.x_row0 = vr0 % TILE_ROWS;
  }
  for (size_t c = 0; c < cascades.size(); ++c) {
    const Cascade& cs = cascades[c];
    if (cs.big) continue;
    const PieReq& v = plan->reqs[cs.vreq];
    const int tiles_per_head = (v.q_len * G + TILE_ROWS - 1) / TILE_ROWS;
    for (int k = 0; k < cs.n; ++k) {
      const int r = cs.first + k;
      const PieReq& q = plan->reqs[r];
      const int rows = q.q_len * G, vr0 = (q.q_start - v.q_start) * G;   // first virtual row of the request
      for (int g = 0; g < cfg.num_kv_heads; ++g) {
        Unit u{r, g, 0, rows, q.kept_start + cs.L, q.kept_start + q.kept_count};
        const auto& sl = tile_slots[(size_t)casc_unit0[c] + (size_t)g * tiles_per_head + vr0 / TILE_ROWS];
        u.x_slot0 = sl.first;
        u.x_nslots = sl.second;
        u.x_row0 = vr0 % TILE_ROWS;
        u.force_partial = true;
        split_units.push_back(u);
      }
    }
  }
  // split-KV decode.  Long launches: chunks taken dynamically by the warps of the grid (evens out
  // SMs that get different shares of the memory bandwidth: 5-10 % of the launch).  Shorter ones: fixed
  // shares - whole units per thread block with the merge inside the block when that balances, else one
  // equal share per warp and the merge launch.  The dynamic list always needs the merge launch
  // (10-20 us with its partials), so it pays from about 270 us on: 1.2 GB of K/V in 209 us against 192 us with
  // whole units per block, 2.3 GB in 335 us against 353 us.
  {
    const int n_warps = split_sms * pie_split_warps_per_block(ctx);
    int64_t W = 0;
    int max_rows = 1;
    for (const Unit& u : split_units) {
      W += u.page_end - u.page_begin;
      max_rows = std::max(max_rows, u.nrows);
    }
    plan->split.heads_per_unit = hp;
    plan->split.grid_merge = false;
    const double kv_bytes = (double)W * hp * 2.0 * P * cfg.head_dim * (cfg.dtype == PIE_DTYPE_BF16 ? 2.0 : 4.0);
    const bool long_launch = kv_bytes * ctx->n_sms >= 1.6e9 * split_sms;   // (fewer SMs: the same bytes take longer)
    bool plain_units = true;
    for (const Unit& u : split_units) plain_units = plain_units && !u.force_partial;
    if (long_launch || (W >= (int64_t)200 * n_warps && !plain_units)) {
      chunk_units(split_units, n_warps, plan->split);
    } else {
      // fixed equal shares, nothing left to the counter (a dynamic tail of small chunks was measured:
      // the extra partials cost more in the merge than the better balance gains on a 50 us launch)
      bool plain = true;   // cascade pieces bring partials of another launch: those groups need the merge kernel
      for (const Unit& u : split_units) plain = plain && !u.force_partial;
      bool local = plain && !(ctx->options[PIE_OPT_NO_FUSION] & 2);
      if (local) {
        // the same units as in the previous batch (a decode loop between two page boundaries): take its list
        pie_ctx::LocalListCache& lc = ctx->local_cache;
        const int nw = pie_split_warps_per_block(ctx);
        std::vector<int32_t>& key = plan->local_key;
        key.resize(6 * split_units.size());
        for (size_t k = 0; k < split_units.size(); ++k) {
          const Unit& u = split_units[k];
          int32_t* d = key.data() + 6 * k;
          d[0] = u.req, d[1] = u.kv_head, d[2] = u.row0, d[3] = u.nrows, d[4] = u.page_begin, d[5] = u.page_end;
        }
        if (lc.valid && lc.sms == split_sms && lc.warps == nw && lc.slot_rows == max_rows && lc.key == key) {
          local = lc.balanced;
          if (local) {
            PieLaunchList& ll = plan->split;
            ll.items = lc.items;
            ll.cta_ptr = lc.cta_ptr;
            ll.merges.clear();
            ll.grid = lc.grid;
            ll.n_slots = lc.n_slots;
            ll.slot_rows = max_rows;
            ll.n_static = 0;
          }
        } else {
          local = partition_local(split_units, split_sms, nw, 4, max_rows, plan->split);
          if (local && !(ctx->options[PIE_OPT_NO_FUSION] & 8)) mark_smem_groups(plan->split);
          lc.valid = true;
          lc.balanced = local;
          lc.sms = split_sms, lc.warps = nw, lc.slot_rows = max_rows;
          lc.key.swap(key);
          if (local) {
            lc.items = plan->split.items;
            lc.cta_ptr = plan->split.cta_ptr;
            lc.grid = plan->split.grid;
            lc.n_slots = plan->split.n_slots;
          }
        }
      }
      if (!local && W >= (int64_t)200 * n_warps) {
        chunk_units(split_units, n_warps, plan->split);   // (many visits per warp and no balanced deal of whole units)
      } else {
        if (!local) {
          partition(split_units, n_warps, 4, max_rows, false, plan->split);
          // Units cut across thread blocks are merged inside the kernel too, in two levels: the pieces that lie
          // in one block by that block (as above: shared-memory counter, the warp with the block's first piece
          // combines them), the resulting one partial per block by whichever block writes its partial last (a
          // device-wide fence and one atomic per block and unit, no waiting).  Measured against the merge launch on
          // 4 / 8 / 16 / 24 / 32 single-token requests of 512 - 4,096 tokens (4 - 16 page visits per warp): 17.3 / 21.3 /
          // 24.2 / 31.2 / 39.0 us against 22.9 / 25.9 / 27.0 / 32.8 / 39.8 us; 8 requests of 8 - 16 k tokens 41.9
          // against 47.3 us (attention alone: 11.6 / 14.3 / 18.6 us for 4 / 8 / 16 requests).
          PieLaunchList& ll = plan->split;
          bool two_level = plain && !(ctx->options[PIE_OPT_NO_FUSION] & 2) && !ll.merges.empty();   // (8-token pages come two per visit)
          if (two_level) {
            const int nw = pie_split_warps_per_block(ctx);
            std::vector<int32_t>& scr = plan->slot_group;   // [n_slots] item of a slot, then [items] warp of an item, then [items] new flags
            const size_t ni = ll.items.size(), ns = (size_t)ll.n_slots;
            scr.assign(ns + 2 * ni, 0);
            int32_t* slot_item = scr.data();
            int32_t* item_warp = scr.data() + ns;
            int32_t* new_flags = scr.data() + ns + ni;
            for (int w = 0; w + 1 < (int)ll.cta_ptr.size(); ++w)
              for (int32_t k = ll.cta_ptr[w]; k < ll.cta_ptr[w + 1]; ++k) item_warp[k] = w;
            for (size_t k = 0; k < ni; ++k)
              if (ll.items[k].partial_slot >= 0) slot_item[ll.items[k].partial_slot] = (int32_t)k;
            int cur_block = -1, gids = 0;   // counters used so far in the block the walk is in (groups come in warp order)
            for (const PieMerge& m : ll.merges) {
              // runs of pieces that share a block
              int nb = 0, n0 = 0;
              for (int a = 0; a < m.nslots;) {
                const int blk = item_warp[slot_item[m.slot0 + a]] / nw;
                int b = a + 1;
                while (b < m.nslots && item_warp[slot_item[m.slot0 + b]] / nw == blk) ++b;
                if (nb == 0) n0 = b - a;
                else if (b < m.nslots && b - a != nw) two_level = false;   // (cannot happen with contiguous shares: a block inside a unit has one piece per warp)
                ++nb;
                a = b;
              }
              if (nb > 255 || n0 > 15) two_level = false;
              if (!two_level) break;
              int kb = 0;
              for (int a = 0; a < m.nslots; ++kb) {
                const int blk = item_warp[slot_item[m.slot0 + a]] / nw;
                int b = a + 1;
                while (b < m.nslots && item_warp[slot_item[m.slot0 + b]] / nw == blk) ++b;
                if (blk != cur_block) cur_block = blk, gids = 0;
                uint32_t f = nb > 1 ? (PIE_ITEM_GRID_PIECE | PIE_ITEM_GRID_BITS(nb, kb, n0)) : 0u;
                if (b - a > 1) {
                  if (gids >= PIE_MAX_LOCAL_GROUPS) two_level = false;
                  f |= PIE_ITEM_LOCAL_PIECE | PIE_ITEM_LOCAL_BITS(gids, b - a);
                  ++gids;
                }
                for (int k = a; k < b; ++k)   // (only the block's first piece carries the unit-level fields)
                  new_flags[slot_item[m.slot0 + k]] = (int32_t)(k == a ? (f | (b - a > 1 ? PIE_ITEM_LOCAL_MERGER : 0u)) : (f & ~(PIE_ITEM_GRID_PIECE | PIE_ITEM_GRID_BITS(255, 255, 15))));
                a = b;
              }
              if (!two_level) break;
            }
            if (two_level) {
              for (size_t k = 0; k < ni; ++k) ll.items[k].flags |= (uint32_t)new_flags[k];
              ll.merges.clear();
              ll.grid_merge = true;
              if (!(ctx->options[PIE_OPT_NO_FUSION] & 8)) mark_smem_groups(ll);
            }
          }
        }
        plan->split.n_static = (int32_t)plan->split.items.size();
      }
    }
  }

  // ---- fused append of the decode path (PIE_OPT_NO_FUSION switches it off): when every request brings exactly one new token, all of them run on the split-KV
  // kernel, their last page is in the kept list and no request lists a page another one appends
  // to, the warp that attends a request's last page also writes the new K/V row (into the pool
  // and into its staged copy), and the append launch is dropped.
  const int no_fusion = ctx->options[PIE_OPT_NO_FUSION];
  plan->append_fused = false;
  if (!(no_fusion & 1) && all_rows_out && ctx->cfg.rope_theta <= 0.f && !cross_read && !plan->split.items.empty() &&
      plan->tile.items.empty() && plan->simple_rows.empty()) {
    bool ok = true;
    for (int r = 0; r < R && ok; ++r) {
      const PieReq& q = plan->reqs[r];
      ok = q.q_len == 1 && q.kept_count > 0 &&
           (int)((uint32_t)plan->kept[2 * (size_t)(q.kept_start + q.kept_count - 1) + 1] & ~PIE_KEPT_NEEDS_MASK) == q.last_logical;
    }
    plan->append_fused = ok;
  }
  for (PieLaunchList* ll : {&plan->split, &plan->tile})
    for (PieItem& it : ll->items) {
      const PieReq& q = plan->reqs[it.req];
      if (ll == &plan->split && plan->append_fused && it.page_end == q.kept_start + q.kept_count) it.flags |= PIE_ITEM_APPEND;
      if (ll == &plan->tile) {
        // leading pages of the item that every row of the tile sees in full: the kernel evaluates no
        // mask there.  Inferred causal masks: the pages below the first row's limit; explicit masks:
        // the kept pages before the first one that some row sees only in part.
        int64_t clean_end;   // in the request's kept list
        if (q.mask_row_words == 0) clean_end = ((int64_t)q.kv_len - q.q_len + it.row0 / G + 1) / P;
        else clean_end = it.req < R ? plan->clean_kept[it.req] : q.kept_count;
        const int64_t clean = std::min<int64_t>(std::max<int64_t>(clean_end - (it.page_begin - q.kept_start), 0), it.page_end - it.page_begin);
        it.flags = (uint32_t)clean << PIE_ITEM_CLEAN_SHIFT;
      }
      it.q_start = q.q_start;
      it.q_len = q.q_len;
      it.kv_len = q.kv_len;
      it.mask_row_words = q.mask_row_words;
      it.last_logical = q.last_logical;
      it.last_page_len = q.last_page_len;
      it.mask_word_off = q.mask_word_off;
    }
  pie_plan_info& info = plan->info;
  info = pie_plan_info{};
  info.num_requests = R;
  info.num_query_tokens = T;
  info.num_split_items = (int32_t)plan->split.items.size();
  info.num_tile_items = (int32_t)plan->tile.items.size();
  info.num_simple_rows = (int32_t)plan->simple_rows.size();
  info.num_merge_groups = (int32_t)(plan->split.merges.size() + plan->tile.merges.size());
  info.kept_pages = (int64_t)plan->kept.size() / 2;
  info.mask_words = (int64_t)plan->mask_words.size();
  info.workspace_bytes = ((int64_t)plan->split.n_slots * plan->split.slot_rows +
                          (int64_t)plan->tile.n_slots * plan->tile.slot_rows) * (cfg.head_dim + 1) * 4;
  info.side_by_side_sms = plan->overlap ? plan->tile.grid : 0;
  info.split_unit_kv_heads = plan->split.items.empty() ? 1 : plan->split.heads_per_unit;
  info.reserved0 = 0;
  info.launches = (plan->pre_copies.empty() ? 0 : 1) + (plan->append_fused ? 0 : 1) + (info.num_simple_rows ? 1 : 0) + (info.num_split_items ? 1 : 0) +
                  (info.num_tile_items ? 1 : 0) + (plan->split.merges.empty() ? 0 : 1) +
                  (plan->tile.merges.empty() ? 0 : 1);
  return PIE_OK;
}
