// tracegen_host.cpp — host build of the synthetic trace generator (threads over streams).
#include "tracegen.h"

#include <math.h>

#include <atomic>
#include <thread>
#include <vector>

namespace {

uint64_t closed_form_len(const tg_params& p, uint32_t s) {
  const uint32_t W = tg_warps_per_cta(p.kind), warp = s % W;
  switch (p.kind) {
    case TG_TINY: return p.iters;
    case TG_GEMM: return (uint64_t)p.iters * (warp < 2 ? 36u : 16u);
    case TG_ATTENTION:
      if (warp >= 14) return (uint64_t)p.iters * 8u;
      return (uint64_t)p.iters * (2u + (uint64_t)p.inner * (warp < 2 ? 10u : 6u));
    default: return (uint64_t)p.iters * (2u + (uint64_t)p.inner * 92u);
  }
}

template <class F>
void parallel_streams(uint32_t lo, uint32_t hi, int nthreads, F f) {
  if (nthreads < 1) nthreads = 1;
  std::atomic<uint32_t> next(lo);
  std::vector<std::thread> pool;
  auto worker = [&]() {
    for (;;) {
      const uint32_t s = next.fetch_add(1);
      if (s >= hi) return;
      f(s);
    }
  };
  for (int i = 1; i < nthreads; ++i) pool.emplace_back(worker);
  worker();
  for (auto& t : pool) t.join();
}

}  // namespace

extern "C" {

uint32_t tg_num_streams(const tg_params* p) { return p->num_ctas * tg_warps_per_cta(p->kind); }
uint32_t tg_regions(const tg_params* p) { return tg_num_regions(*p); }
uint32_t tg_warps(const tg_params* p) { return tg_warps_per_cta(p->kind); }

// Writes the length of every stream (after defects and truncation) to lens[S].
int tg_lengths(const tg_params* p, uint64_t* lens, int nthreads) {
  const uint32_t S = tg_num_streams(p);
  const bool fixed = p->thr_dup_begin == 0 && p->thr_drop_end == 0;
  parallel_streams(0, S, nthreads, [&](uint32_t s) {
    const uint64_t full = fixed ? closed_form_len(*p, s) : tg_run_stream(*p, s, nullptr, 0);
    lens[s] = tg_truncated_len(*p, s, full);
  });
  return 0;
}

// Writes streams [s_lo, s_hi) to out, where stream s starts at out[stream_offsets[s] - stream_offsets[s_lo]].
int tg_fill(const tg_params* p, const uint64_t* stream_offsets, uint32_t s_lo, uint32_t s_hi, tg_event* out,
            int nthreads) {
  const uint32_t S = tg_num_streams(p);
  if (s_lo > s_hi || s_hi > S) return 1;
  parallel_streams(s_lo, s_hi, nthreads, [&](uint32_t s) {
    const uint64_t n = stream_offsets[s + 1] - stream_offsets[s];
    if (n) tg_run_stream(*p, s, out + (stream_offsets[s] - stream_offsets[s_lo]), n);
  });
  return 0;
}
}
