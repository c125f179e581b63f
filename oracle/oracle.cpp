// oracle.cpp — single-threaded CPU oracle (test infrastructure; see oracle.h).
//
// Written from the sequential definition, not from the CUDA path: an explicit std::vector
// stack per stream, std::map aggregates, sort + two-pointer sweep for overlap. No blocking,
// no fusion, no reordering beyond what the definition states.
#include "oracle.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <tuple>
#include <utility>
#include <vector>

namespace {

constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr size_t kMaxDepth = 64;
enum { OK = 0, ERR_INVALID = 1, ERR_CAPACITY = 4, ERR_DEPTH = 5, ERR_BAD_REGION = 6, ERR_BAD_OFFSETS = 7 };
enum { FLAG_CTX = 1, FLAG_REV = 2, FLAG_CLAMP = 4 };
enum { AMB_END = 1, AMB_MISNESTED = 2, AMB_EOS = 3 };

struct Frame {
  uint32_t region, ctx;
  uint64_t ts;
  uint32_t idx;
  uint32_t depth;
  uint32_t parent;
  uint64_t child;  // sum of inclusive time of matched intervals directly below this frame
};

void fail(OStatus* st, uint32_t code, uint32_t stream, uint64_t ev) {
  if (st->code == OK) { st->code = code; st->bad_stream = stream; st->bad_event = ev; }
}

}  // namespace

extern "C" int oracle_pair(const OEvent* events, const uint64_t* stream_offsets, uint32_t num_streams,
                           uint32_t num_regions, OInterval* intervals, uint64_t interval_cap,
                           uint64_t* interval_offsets, OAmbig* ambig, uint64_t ambig_cap,
                           uint64_t* ambig_offsets, OStatus* st) {
  if (!stream_offsets || !interval_offsets || !ambig_offsets || !st) return ERR_INVALID;
  if (num_regions == 0 || num_regions > 65536) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  uint64_t n_int = 0, n_amb = 0;
  interval_offsets[0] = 0;
  ambig_offsets[0] = 0;
  for (uint32_t s = 0; s < num_streams; ++s) {
    const uint64_t lo = stream_offsets[s], hi = stream_offsets[s + 1];
    if (hi < lo) { fail(st, ERR_BAD_OFFSETS, s, 0); return OK; }
    const uint64_t n = hi - lo;
    std::vector<Frame> stack;
    std::vector<OAmbig> amb;  // this stream's records, sorted by event index at the end
    auto note = [&](uint32_t kind, uint64_t ts, uint32_t tag, uint32_t ctx, uint32_t idx, uint32_t depth) {
      amb.push_back(OAmbig{ts, tag, ctx, s, idx, kind, depth});
    };
    for (uint64_t i = 0; i < n; ++i) {
      const OEvent& e = events[lo + i];
      const uint32_t region = e.tag >> 1;
      const bool is_end = (e.tag & 1u) != 0;
      if (region >= num_regions) { fail(st, ERR_BAD_REGION, s, i); return OK; }
      if (!is_end) {
        if (stack.size() == kMaxDepth) { fail(st, ERR_DEPTH, s, i); return OK; }
        Frame f;
        f.region = region; f.ctx = e.ctx; f.ts = e.ts; f.idx = static_cast<uint32_t>(i);
        f.depth = static_cast<uint32_t>(stack.size());
        f.parent = stack.empty() ? kNone : stack.back().region;
        f.child = 0;
        stack.push_back(f);
        continue;
      }
      // end marker: innermost open frame of the same region, searching down from the top
      long k = static_cast<long>(stack.size()) - 1;
      while (k >= 0 && stack[static_cast<size_t>(k)].region != region) --k;
      if (k < 0) {
        note(AMB_END, e.ts, e.tag, e.ctx, static_cast<uint32_t>(i), static_cast<uint32_t>(stack.size()));
        continue;
      }
      while (static_cast<long>(stack.size()) - 1 > k) {  // force-close mis-nested frames
        Frame f = stack.back();
        stack.pop_back();
        note(AMB_MISNESTED, f.ts, f.region << 1, f.ctx, f.idx, f.depth);
        stack.back().child += f.child;  // grandchildren time moves up
      }
      Frame f = stack.back();
      stack.pop_back();
      uint16_t flags = 0;
      uint64_t incl, excl;
      if (e.ctx != f.ctx) { flags |= FLAG_CTX; st->n_ctx_mismatch++; }
      if (e.ts < f.ts) { incl = 0; flags |= FLAG_REV; st->n_time_reversed++; } else { incl = e.ts - f.ts; }
      if (f.child > incl) { excl = 0; flags |= FLAG_CLAMP; st->n_child_clamped++; } else { excl = incl - f.child; }
      if (n_int < interval_cap && intervals) {
        OInterval& o = intervals[n_int];
        o.t_begin = f.ts; o.inclusive = incl; o.exclusive = excl;
        o.region = f.region; o.ctx = f.ctx; o.stream = s; o.parent_region = f.parent;
        o.begin_idx = f.idx; o.depth = static_cast<uint16_t>(f.depth); o.flags = flags;
      }
      ++n_int;
      if (!stack.empty()) stack.back().child += incl;
    }
    for (const Frame& f : stack) note(AMB_EOS, f.ts, f.region << 1, f.ctx, f.idx, f.depth);
    std::sort(amb.begin(), amb.end(), [](const OAmbig& a, const OAmbig& b) { return a.event_idx < b.event_idx; });
    for (const OAmbig& a : amb) {
      if (n_amb < ambig_cap && ambig) ambig[n_amb] = a;
      ++n_amb;
    }
    interval_offsets[s + 1] = n_int;
    ambig_offsets[s + 1] = n_amb;
  }
  st->intervals_required = n_int;
  st->ambig_required = n_amb;
  if (n_int > interval_cap) fail(st, ERR_CAPACITY, 0, n_int);
  else if (n_amb > ambig_cap) fail(st, ERR_CAPACITY, 0, n_amb);
  return OK;
}

namespace {

int bin_of(uint64_t d) {  // floor(log2 d), with d in {0, 1} -> 0
  int b = 0;
  while (d > 1) { d >>= 1; ++b; }
  return b;
}

struct Cell {
  OAgg a;
  Cell() { std::memset(&a, 0, sizeof(a)); a.min_incl = ~0ull; }
};

using Key = std::tuple<int, uint32_t, uint32_t>;  // (level, scope key, region)

void materialise(const std::map<Key, Cell>& m, int level, uint32_t nkeys, uint32_t R, OAgg* tab) {
  if (!tab) return;
  Cell empty;
  for (uint64_t i = 0; i < static_cast<uint64_t>(nkeys) * R; ++i) tab[i] = empty.a;
  for (const auto& kv : m) {
    if (std::get<0>(kv.first) != level) continue;
    tab[static_cast<uint64_t>(std::get<1>(kv.first)) * R + std::get<2>(kv.first)] = kv.second.a;
  }
}

}  // namespace

extern "C" int oracle_aggregate(const OInterval* intervals, const uint64_t* interval_offsets,
                                const OAmbig* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                                uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                                uint32_t num_regions, OAgg* warp_tab, OAgg* cta_tab, OAgg* sm_tab,
                                OAgg* kernel_tab, OStatus* st) {
  if (!interval_offsets || !st || warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ERR_INVALID;
  if (num_regions == 0 || num_regions > 65536) return ERR_INVALID;
  if ((sm_tab != nullptr) && (!cta_sm || num_sms == 0)) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  const uint32_t num_ctas = num_streams / warps_per_cta;
  std::map<Key, Cell> m;
  auto keys_of = [&](uint32_t s, uint32_t keys[4]) {
    keys[0] = s;
    keys[1] = s / warps_per_cta;
    keys[2] = cta_sm ? cta_sm[s / warps_per_cta] : 0;
    keys[3] = 0;
  };
  for (uint32_t s = 0; s < num_streams; ++s) {
    uint32_t keys[4];
    keys_of(s, keys);
    if (cta_sm && keys[2] >= num_sms && sm_tab) return ERR_INVALID;
    for (uint64_t i = interval_offsets[s]; i < interval_offsets[s + 1]; ++i) {
      const OInterval& v = intervals[i];
      if (v.region >= num_regions) { fail(st, ERR_BAD_REGION, s, i); return OK; }
      for (int level = 0; level < 4; ++level) {
        OAgg& a = m[Key(level, keys[level], v.region)].a;
        a.count++;
        a.sum_incl += v.inclusive;
        a.min_incl = std::min(a.min_incl, v.inclusive);
        a.max_incl = std::max(a.max_incl, v.inclusive);
        a.sum_excl += v.exclusive;
        a.n_flagged += (v.flags != 0);
        a.hist[bin_of(v.inclusive)]++;
      }
    }
    if (ambig && ambig_offsets) {
      for (uint64_t i = ambig_offsets[s]; i < ambig_offsets[s + 1]; ++i) {
        const OAmbig& r = ambig[i];
        const uint32_t region = r.tag >> 1;
        if (region >= num_regions) { fail(st, ERR_BAD_REGION, s, i); return OK; }
        for (int level = 0; level < 4; ++level) {
          OAgg& a = m[Key(level, keys[level], region)].a;
          if (r.kind == AMB_END) a.n_unmatched_end++; else a.n_unmatched_begin++;
        }
      }
    }
  }
  materialise(m, 0, num_streams, num_regions, warp_tab);
  materialise(m, 1, num_ctas, num_regions, cta_tab);
  materialise(m, 2, num_sms, num_regions, sm_tab);
  materialise(m, 3, 1, num_regions, kernel_tab);
  return OK;
}

namespace {

using Span = std::pair<uint64_t, uint64_t>;  // half-open [first, second)

std::vector<Span> merged_union(std::vector<Span> v) {
  std::sort(v.begin(), v.end());
  std::vector<Span> u;
  for (const Span& s : v) {
    if (!u.empty() && s.first <= u.back().second) u.back().second = std::max(u.back().second, s.second);
    else u.push_back(s);
  }
  return u;
}

uint64_t measure(const std::vector<Span>& u) {
  uint64_t t = 0;
  for (const Span& s : u) t += s.second - s.first;
  return t;
}

}  // namespace

extern "C" int oracle_overlap(const OInterval* intervals, const uint64_t* interval_offsets,
                              uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm,
                              uint32_t num_sms, const uint32_t* pairs, uint32_t num_pairs, OOverlap* out,
                              OStatus* st) {
  if (!interval_offsets || !cta_sm || !st || warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ERR_INVALID;
  if (num_pairs && (!pairs || !out)) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  std::vector<std::vector<uint32_t>> streams_of_sm(num_sms);  // which streams ran on each SM
  for (uint32_t s = 0; s < num_streams; ++s) {
    const uint32_t m = cta_sm[s / warps_per_cta];
    if (m >= num_sms) return ERR_INVALID;
    streams_of_sm[m].push_back(s);
  }
  for (uint32_t k = 0; k < num_pairs; ++k) {
    const uint32_t P = pairs[2 * k], Cn = pairs[2 * k + 1];
    for (uint32_t m = 0; m < num_sms; ++m) {
      std::vector<Span> p, c;
      for (uint32_t s : streams_of_sm[m]) {
        for (uint64_t i = interval_offsets[s]; i < interval_offsets[s + 1]; ++i) {
          const OInterval& v = intervals[i];
          if (v.inclusive == 0) continue;  // empty span
          const Span sp(v.t_begin, v.t_begin + v.inclusive);
          if (v.region == P) p.push_back(sp);
          if (v.region == Cn) c.push_back(sp);
        }
      }
      const std::vector<Span> up = merged_union(p), uc = merged_union(c);
      uint64_t both = 0;
      size_t a = 0, b = 0;
      while (a < up.size() && b < uc.size()) {  // two-pointer sweep over disjoint sorted spans
        const uint64_t lo = std::max(up[a].first, uc[b].first);
        const uint64_t hi = std::min(up[a].second, uc[b].second);
        if (hi > lo) both += hi - lo;
        if (up[a].second < uc[b].second) ++a; else ++b;
      }
      OOverlap& o = out[static_cast<uint64_t>(k) * num_sms + m];
      o.producer_ns = measure(up);
      o.consumer_ns = measure(uc);
      o.overlap_ns = both;
      o.either_ns = o.producer_ns + o.consumer_ns - both;
    }
  }
  return OK;
}

// ---------------------------------------------------------------------------------------------
// Scope selection (Section 1, the observe(region, signals, scope) query; Section 3.2 "Region and
// scope"). The four tests of membership, written out once; everything else repeats the plain
// definitions above on the selected records.
// ---------------------------------------------------------------------------------------------
namespace {

bool bit_set(const uint32_t* mask, uint32_t i) { return mask == nullptr || ((mask[i / 32] >> (i % 32)) & 1u) != 0; }

bool in_scope(const OScope* sc, uint32_t stream, uint32_t ctx, uint32_t region, uint32_t warps_per_cta,
              const uint32_t* cta_sm) {
  if (sc == nullptr) return true;
  if (ctx < sc->ctx_lo || ctx > sc->ctx_hi) return false;                       // iteration window
  const uint32_t w = stream % warps_per_cta;                                      // warp role
  if (sc->warp_mask != ~0ull && (w >= 64 || ((sc->warp_mask >> w) & 1ull) == 0)) return false;
  if (sc->sm_mask != nullptr && cta_sm != nullptr && !bit_set(sc->sm_mask, cta_sm[stream / warps_per_cta])) return false;
  return bit_set(sc->region_mask, region);                                        // region set
}

}  // namespace

extern "C" int oracle_aggregate_scoped(const OInterval* intervals, const uint64_t* interval_offsets,
                                       const OAmbig* ambig, const uint64_t* ambig_offsets, uint32_t num_streams,
                                       uint32_t warps_per_cta, const uint32_t* cta_sm, uint32_t num_sms,
                                       uint32_t num_regions, const OScope* scope, OAgg* warp_tab, OAgg* cta_tab,
                                       OAgg* sm_tab, OAgg* kernel_tab, OAgg* role_tab, OAgg* iter_tab, OStatus* st) {
  if (!interval_offsets || !st || warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ERR_INVALID;
  if (num_regions == 0 || num_regions > 65536) return ERR_INVALID;
  if ((sm_tab != nullptr || (scope && scope->sm_mask)) && (!cta_sm || num_sms == 0)) return ERR_INVALID;
  if (scope && scope->ctx_hi < scope->ctx_lo) return ERR_INVALID;
  if (iter_tab && (!scope || scope->ctx_hi - scope->ctx_lo >= 65536u)) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  const uint32_t num_ctas = num_streams / warps_per_cta;
  const uint32_t num_iters = iter_tab ? scope->ctx_hi - scope->ctx_lo + 1 : 0;
  std::map<Key, Cell> m;  // levels 0..3 as in oracle_aggregate, 4 = warp role, 5 = iteration
  for (uint32_t s = 0; s < num_streams; ++s) {
    uint32_t keys[6];
    keys[0] = s;
    keys[1] = s / warps_per_cta;
    keys[2] = cta_sm ? cta_sm[s / warps_per_cta] : 0;
    keys[3] = 0;
    keys[4] = s % warps_per_cta;
    if (cta_sm && keys[2] >= num_sms && (sm_tab || (scope && scope->sm_mask))) return ERR_INVALID;
    for (uint64_t i = interval_offsets[s]; i < interval_offsets[s + 1]; ++i) {
      const OInterval& v = intervals[i];
      if (v.region >= num_regions) { fail(st, ERR_BAD_REGION, s, i); return OK; }
      if (!in_scope(scope, s, v.ctx, v.region, warps_per_cta, cta_sm)) continue;
      keys[5] = scope ? v.ctx - scope->ctx_lo : 0;
      for (int level = 0; level < 6; ++level) {
        if (level == 5 && !iter_tab) continue;
        OAgg& a = m[Key(level, keys[level], v.region)].a;
        a.count++;
        a.sum_incl += v.inclusive;
        a.min_incl = std::min(a.min_incl, v.inclusive);
        a.max_incl = std::max(a.max_incl, v.inclusive);
        a.sum_excl += v.exclusive;
        a.n_flagged += (v.flags != 0);
        a.hist[bin_of(v.inclusive)]++;
      }
    }
    if (ambig && ambig_offsets) {
      for (uint64_t i = ambig_offsets[s]; i < ambig_offsets[s + 1]; ++i) {
        const OAmbig& r = ambig[i];
        const uint32_t region = r.tag >> 1;
        if (region >= num_regions) { fail(st, ERR_BAD_REGION, s, i); return OK; }
        if (!in_scope(scope, s, r.ctx, region, warps_per_cta, cta_sm)) continue;
        keys[5] = scope ? r.ctx - scope->ctx_lo : 0;
        for (int level = 0; level < 6; ++level) {
          if (level == 5 && !iter_tab) continue;
          OAgg& a = m[Key(level, keys[level], region)].a;
          if (r.kind == AMB_END) a.n_unmatched_end++; else a.n_unmatched_begin++;
        }
      }
    }
  }
  materialise(m, 0, num_streams, num_regions, warp_tab);
  materialise(m, 1, num_ctas, num_regions, cta_tab);
  materialise(m, 2, num_sms, num_regions, sm_tab);
  materialise(m, 3, 1, num_regions, kernel_tab);
  materialise(m, 4, warps_per_cta, num_regions, role_tab);
  materialise(m, 5, num_iters, num_regions, iter_tab);
  return OK;
}

extern "C" int oracle_overlap_scoped(const OInterval* intervals, const uint64_t* interval_offsets,
                                     uint32_t num_streams, uint32_t warps_per_cta, const uint32_t* cta_sm,
                                     uint32_t num_sms, const uint32_t* pairs, uint32_t num_pairs,
                                     const OScope* scope, OOverlap* out, OStatus* st) {
  if (!interval_offsets || !cta_sm || !st || warps_per_cta == 0 || num_streams % warps_per_cta != 0) return ERR_INVALID;
  if (num_pairs && (!pairs || !out)) return ERR_INVALID;
  if (scope && scope->ctx_hi < scope->ctx_lo) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  for (uint32_t s = 0; s < num_streams; ++s)
    if (cta_sm[s / warps_per_cta] >= num_sms) return ERR_INVALID;
  for (uint32_t k = 0; k < num_pairs; ++k) {
    const uint32_t P = pairs[2 * k], Cn = pairs[2 * k + 1];
    for (uint32_t sm = 0; sm < num_sms; ++sm) {
      std::vector<Span> p, c;
      for (uint32_t s = 0; s < num_streams; ++s) {
        if (cta_sm[s / warps_per_cta] != sm) continue;
        for (uint64_t i = interval_offsets[s]; i < interval_offsets[s + 1]; ++i) {
          const OInterval& v = intervals[i];
          if (v.inclusive == 0) continue;  // empty span
          if (!in_scope(scope, s, v.ctx, v.region, warps_per_cta, cta_sm)) continue;
          const Span sp(v.t_begin, v.t_begin + v.inclusive);
          if (v.region == P) p.push_back(sp);
          if (v.region == Cn) c.push_back(sp);
        }
      }
      const std::vector<Span> up = merged_union(p), uc = merged_union(c);
      uint64_t both = 0;
      for (const Span& x : up)        // every producer piece against every consumer piece
        for (const Span& y : uc) {
          const uint64_t lo = std::max(x.first, y.first), hi = std::min(x.second, y.second);
          if (hi > lo) both += hi - lo;
        }
      OOverlap& o = out[static_cast<uint64_t>(k) * num_sms + sm];
      o.producer_ns = measure(up);
      o.consumer_ns = measure(uc);
      o.overlap_ns = both;
      o.either_ns = o.producer_ns + o.consumer_ns - both;
    }
  }
  return OK;
}

// ---------------------------------------------------------------------------------------------
// PC-to-region mapping (Section 3.2) and ambiguity-aware attribution (Section 3.5).
// ---------------------------------------------------------------------------------------------
extern "C" int oracle_map_pc_counts(const OMapEvent* events, const uint64_t* stream_offsets, uint32_t num_streams,
                                    uint32_t num_regions, uint32_t num_pcs, uint64_t* counts, OStatus* st) {
  if (!stream_offsets || !counts || !st || num_regions == 0 || num_pcs == 0) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  std::memset(counts, 0, sizeof(uint64_t) * (static_cast<size_t>(num_regions) + 1) * num_pcs);
  for (uint32_t s = 0; s < num_streams; ++s) {
    std::vector<uint32_t> stack;  // region ids of the open frames, innermost last
    for (uint64_t i = stream_offsets[s]; i < stream_offsets[s + 1]; ++i) {
      const OMapEvent& e = events[i];
      if (e.kind == 2) {  // exec: the innermost active region receives the execution count
        if (e.id >= num_pcs) return ERR_INVALID;
        if (stack.size() == kMaxDepth) { fail(st, ERR_DEPTH, s, i - stream_offsets[s]); return OK; }
        const uint32_t owner = stack.empty() ? num_regions : stack.back();
        counts[static_cast<size_t>(owner) * num_pcs + e.id] += e.count;
      } else if (e.kind == 0) {
        if (e.id >= num_regions) { fail(st, ERR_BAD_REGION, s, i - stream_offsets[s]); return OK; }
        if (stack.size() == kMaxDepth) { fail(st, ERR_DEPTH, s, i - stream_offsets[s]); return OK; }
        stack.push_back(e.id);
      } else {
        if (e.id >= num_regions) { fail(st, ERR_BAD_REGION, s, i - stream_offsets[s]); return OK; }
        size_t k = stack.size();
        while (k > 0 && stack[k - 1] != e.id) --k;   // innermost open frame of this region
        if (k > 0) stack.resize(k - 1);              // it closes, and so does everything above it
      }
    }
  }
  return OK;
}

extern "C" int oracle_attribute(const uint64_t* counts, uint32_t num_rows, uint32_t num_pcs, const double* metric,
                                double* mhat, double* entropy, double* alpha) {
  if (!counts || !metric || !mhat || !entropy || num_rows == 0 || num_pcs == 0) return ERR_INVALID;
  for (uint32_t r = 0; r < num_rows; ++r) mhat[r] = 0.0;
  for (uint32_t p = 0; p < num_pcs; ++p) {
    uint64_t total = 0;
    for (uint32_t r = 0; r < num_rows; ++r) total += counts[static_cast<size_t>(r) * num_pcs + p];
    double h = 0.0;
    for (uint32_t r = 0; r < num_rows; ++r) {
      const uint64_t n = counts[static_cast<size_t>(r) * num_pcs + p];
      const double a = (total == 0 || n == 0) ? 0.0 : static_cast<double>(n) / static_cast<double>(total);
      if (alpha) alpha[static_cast<size_t>(r) * num_pcs + p] = a;
      if (a > 0.0) {
        mhat[r] += a * metric[p];
        h -= a * std::log(a);
      }
    }
    entropy[p] = h;
  }
  return OK;
}

// ---------------------------------------------------------------------------------------------
// Cross-run join with distribution statistics (Sections 3.3 and 3.5; appendix percentiles).
// ---------------------------------------------------------------------------------------------
extern "C" int oracle_join_samples(const OInterval* reference, uint64_t num_reference, const uint64_t* ref_index,
                                   uint32_t num_queries, const OInterval* samples, uint64_t num_samples, OJoin* out,
                                   OStatus* st) {
  if (!st || (num_queries && (!reference || !ref_index || !out)) || (num_samples && !samples)) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  for (uint32_t q = 0; q < num_queries; ++q) {
    if (ref_index[q] >= num_reference) return ERR_INVALID;
    const OInterval& ref = reference[ref_index[q]];
    std::vector<uint64_t> values;
    for (uint64_t i = 0; i < num_samples; ++i) {
      const OInterval& x = samples[i];
      if (x.stream == ref.stream && x.region == ref.region && x.ctx == ref.ctx) values.push_back(x.inclusive);
    }
    std::sort(values.begin(), values.end());
    OJoin& o = out[q];
    std::memset(&o, 0, sizeof(o));
    o.count = values.size();
    for (uint64_t v : values) o.sum += v;
    if (!values.empty()) {
      for (int j = 0; j < 5; ++j) o.pct[j] = values[(static_cast<size_t>(j) * values.size()) / 5];
      o.max = values.back();
    }
    if (values.size() > 4096 && st->code == 0) fail(st, ERR_CAPACITY, ref.stream, ref_index[q]);
  }
  return OK;
}

// ---------------------------------------------------------------------------------------------
// Ring-buffer container -> packed CSR (input handling only; no paper arithmetic involved).
// ---------------------------------------------------------------------------------------------
extern "C" int oracle_ring_linearise(const OEvent* ring, uint32_t slot_capacity, const uint64_t* written,
                                     uint32_t num_streams, OEvent* events, uint64_t event_capacity,
                                     uint64_t* stream_offsets, uint64_t* dropped, OStatus* st) {
  if (!st || !stream_offsets || slot_capacity == 0 || (num_streams && (!ring || !written))) return ERR_INVALID;
  std::memset(st, 0, sizeof(*st));
  uint64_t total = 0;
  for (uint32_t s = 0; s < num_streams; ++s) {
    stream_offsets[s] = total;
    total += std::min<uint64_t>(written[s], slot_capacity);
    if (dropped) dropped[s] = written[s] > slot_capacity ? written[s] - slot_capacity : 0;
  }
  stream_offsets[num_streams] = total;
  st->intervals_required = total;
  if (total > event_capacity) { fail(st, ERR_CAPACITY, 0, total); return OK; }
  for (uint32_t s = 0; s < num_streams; ++s) {
    const uint64_t kept = std::min<uint64_t>(written[s], slot_capacity);
    const uint64_t first = written[s] - kept;  // index of the oldest surviving record
    for (uint64_t i = 0; i < kept; ++i)
      events[stream_offsets[s] + i] = ring[static_cast<uint64_t>(s) * slot_capacity + (first + i) % slot_capacity];
  }
  return OK;
}
