// Host threads of the planner: a job pool and a merge sort.  Results never depend on the
// number of threads; large inputs only get there faster.
#pragma once

#include <algorithm>
#include <atomic>
#include <cstddef>
#include <cstdlib>
#include <thread>
#include <vector>

namespace bcp {

// Host threads for large work lists.  The result never depends on the count.
inline unsigned plan_threads(size_t n_units) {
  if (n_units < 32768) return 1;
  unsigned n = 0;
  if (const char* e = getenv("BCP_PLAN_THREADS")) n = unsigned(strtoul(e, nullptr, 10));
  if (!n) n = std::min(8u, std::thread::hardware_concurrency());
  return std::max(1u, std::min(n, 64u));
}

// job(0) .. job(n_jobs - 1), handed out by a counter to the caller and up to threads - 1 helpers.
// Jobs must not throw; if helpers cannot be started the caller does all the work.
template <class F>
void parallel_jobs(size_t n_jobs, unsigned threads, F&& job) {
  std::atomic<size_t> next{0};
  auto worker = [&] {
    for (size_t j; (j = next.fetch_add(1)) < n_jobs;) job(j);
  };
  std::vector<std::thread> pool;
  if (threads > 1 && n_jobs > 1) {
    try {
      pool.reserve(threads - 1);
      for (unsigned t = 1; t < threads && t < n_jobs; ++t) pool.emplace_back(worker);
    } catch (...) {
    }
  }
  worker();
  for (std::thread& t : pool) t.join();
}

// Merge sort over `threads` chunks; returns whichever of the two arrays holds the result.
// Every merge of two runs is itself split into parts (cut one run evenly, find the matching
// cut of the other by binary search), so that all rounds keep every thread busy.
template <class T, class Less>
T* parallel_sort(T* k, T* tmp, size_t n, unsigned threads, Less less) {
  const size_t chunks = std::max<size_t>(1, std::min<size_t>(threads, n / 8192));
  auto bound = [&](size_t i) { return n * std::min(i, chunks) / chunks; };
  parallel_jobs(chunks, threads, [&](size_t c) { std::sort(k + bound(c), k + bound(c + 1), less); });
  T *from = k, *to = tmp;
  for (size_t w = 1; w < chunks; w *= 2) {
    const size_t pairs = (chunks + 2 * w - 1) / (2 * w);
    const size_t parts = std::max<size_t>(1, (threads + pairs - 1) / pairs);
    parallel_jobs(pairs * parts, threads, [&](size_t job) {
      const size_t j = job / parts, part = job % parts;
      const size_t lo = bound(2 * j * w), mid = bound(2 * j * w + w), hi = bound(2 * j * w + 2 * w);
      const T *a = from + lo, *b = from + mid;
      const size_t na = mid - lo, nb = hi - mid;
      auto cut_b = [&](size_t ia) { return ia >= na ? nb : size_t(std::lower_bound(b, b + nb, a[ia], less) - b); };
      const size_t a0 = na * part / parts, a1 = na * (part + 1) / parts;
      const size_t b0 = part == 0 ? 0 : cut_b(a0), b1 = part + 1 == parts ? nb : cut_b(a1);
      std::merge(a + a0, a + a1, b + b0, b + b1, to + lo + a0 + b0, less);
    });
    std::swap(from, to);
  }
  return from;
}

}  // namespace bcp
