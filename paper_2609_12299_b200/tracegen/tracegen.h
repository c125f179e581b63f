// tracegen.h — seeded synthetic region-marker traces (input generator only).
//
// This module holds none of the method's arithmetic: it only writes begin/end marker
// events {u64 ts_ns, u32 tag = region << 1 | is_end, u32 ctx}. The same source is compiled
// for the host (g++, threads over streams) and for the device (nvcc, one thread per stream)
// and both produce bit-identical traces: every floating-point step uses only IEEE-exact
// operations (+ - * / sqrt, no fused multiply-add, hand-written log/exp/cos series), so the
// CPU oracle and the CUDA library can each be fed the same trace without copying it.
//
// Trace kinds stand in for the workloads the paper profiles (Section 4): a warp-specialised
// persistent GEMM, attention kernels and a persistent decode megakernel; plus a tiny random
// well-formed trace. Defects (dropped ends, duplicated begins, truncated streams) are applied
// on top by probability thresholds.
#ifndef ARGUS_TRACEGEN_H_
#define ARGUS_TRACEGEN_H_
#include <math.h>
#include <stdint.h>

#if defined(__CUDACC__)
#define TG_HD __host__ __device__ inline
#else
#define TG_HD inline
#endif

struct tg_event { uint64_t ts; uint32_t tag; uint32_t ctx; };

enum { TG_TINY = 1, TG_GEMM = 2, TG_ATTENTION = 3, TG_DECODE = 4 };

struct tg_params {
  uint32_t kind;      // TG_*
  uint32_t num_ctas;  // C
  uint32_t iters;     // TINY: events per stream (even); GEMM: tile iterations; ATTENTION: tiles; DECODE: tokens
  uint32_t inner;     // ATTENTION: KV iterations per tile; DECODE: layers; else unused
  uint64_t seed;
  uint64_t thr_dup_begin;  // a begin is written twice when a 64-bit draw is below this
  uint64_t thr_drop_end;   // an end is dropped when a 64-bit draw is below this
  uint64_t thr_trunc;      // a stream is truncated when a 64-bit draw is below this
};

TG_HD uint32_t tg_warps_per_cta(uint32_t kind) {
  return kind == TG_TINY ? 4u : kind == TG_GEMM ? 12u : 16u;
}
TG_HD uint32_t tg_num_regions(const tg_params& p) {
  return p.kind == TG_TINY ? 8u : p.kind == TG_GEMM ? 5u : p.kind == TG_ATTENTION ? 9u : 4u + 9u * p.inner;
}

// ---- counter-based generator: splitmix64 keyed by (seed, stream, lane) -------------------
struct tg_rng {
  uint64_t s;
  TG_HD uint64_t next() {
    s += 0x9E3779B97F4A7C15ull;
    uint64_t z = s;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  }
};
TG_HD tg_rng tg_make_rng(uint64_t seed, uint32_t stream, uint32_t lane) {
  tg_rng r;
  r.s = seed * 0xD1342543DE82EF95ull + ((uint64_t)stream << 8) + lane;
  r.next();
  r.s ^= r.next();
  return r;
}

// ---- IEEE-exact elementary functions (identical on host and device) ----------------------
TG_HD double tg_u01(uint64_t x) { return (double)(x >> 11) * (1.0 / 9007199254740992.0); }

union tg_bits { double d; uint64_t u; };

TG_HD double tg_log(double x) {  // x > 0, normal
  tg_bits b; b.d = x;
  long long e = (long long)((b.u >> 52) & 0x7ffull) - 1023;
  b.u = (b.u & 0x000fffffffffffffull) | 0x3ff0000000000000ull;
  double m = b.d;
  if (m > 1.4142135623730951) { m = m * 0.5; e += 1; }
  const double s = (m - 1.0) / (m + 1.0);
  const double s2 = s * s;
  double p = 1.0 / 21.0;
  p = p * s2 + 1.0 / 19.0;
  p = p * s2 + 1.0 / 17.0;
  p = p * s2 + 1.0 / 15.0;
  p = p * s2 + 1.0 / 13.0;
  p = p * s2 + 1.0 / 11.0;
  p = p * s2 + 1.0 / 9.0;
  p = p * s2 + 1.0 / 7.0;
  p = p * s2 + 1.0 / 5.0;
  p = p * s2 + 1.0 / 3.0;
  p = p * s2 + 1.0;
  return (double)e * 0.6931471805599453 + 2.0 * s * p;
}

TG_HD double tg_exp(double y) {  // |y| < 700
  const double t = y * 1.4426950408889634 + 0.5;
  long long k = (long long)t;
  if ((double)k > t) k -= 1;
  const double r = (y - (double)k * 0.693147180369123816490e+00) - (double)k * 1.90821492927058770002e-10;
  double p = 1.0 / 6227020800.0;
  p = p * r + 1.0 / 479001600.0;
  p = p * r + 1.0 / 39916800.0;
  p = p * r + 1.0 / 3628800.0;
  p = p * r + 1.0 / 362880.0;
  p = p * r + 1.0 / 40320.0;
  p = p * r + 1.0 / 5040.0;
  p = p * r + 1.0 / 720.0;
  p = p * r + 1.0 / 120.0;
  p = p * r + 1.0 / 24.0;
  p = p * r + 1.0 / 6.0;
  p = p * r + 0.5;
  p = p * r + 1.0;
  p = p * r + 1.0;
  tg_bits b; b.u = (uint64_t)(k + 1023) << 52;
  return p * b.d;
}

TG_HD double tg_cos2pi(double u) {  // cos(2*pi*u), u in [0, 1)
  const double t = u * 4.0;
  const int q = (int)t;
  const double a = (t - (double)q) * 1.5707963267948966;
  const double a2 = a * a;
  double c = 1.0 / 620448401733239439360000.0;  // 1/24!
  c = 1.0 / 1124000727777607680000.0 - c * a2;  // 1/22!
  c = 1.0 / 2432902008176640000.0 - c * a2;     // 1/20!
  c = 1.0 / 6402373705728000.0 - c * a2;        // 1/18!
  c = 1.0 / 20922789888000.0 - c * a2;          // 1/16!
  c = 1.0 / 87178291200.0 - c * a2;             // 1/14!
  c = 1.0 / 479001600.0 - c * a2;               // 1/12!
  c = 1.0 / 3628800.0 - c * a2;                 // 1/10!
  c = 1.0 / 40320.0 - c * a2;                   // 1/8!
  c = 1.0 / 720.0 - c * a2;                     // 1/6!
  c = 1.0 / 24.0 - c * a2;                      // 1/4!
  c = 0.5 - c * a2;
  c = 1.0 - c * a2;
  double s = 1.0 / 15511210043330985984000000.0;  // 1/25!
  s = 1.0 / 25852016738884976640000.0 - s * a2;   // 1/23!
  s = 1.0 / 51090942171709440000.0 - s * a2;      // 1/21!
  s = 1.0 / 121645100408832000.0 - s * a2;        // 1/19!
  s = 1.0 / 355687428096000.0 - s * a2;           // 1/17!
  s = 1.0 / 1307674368000.0 - s * a2;             // 1/15!
  s = 1.0 / 6227020800.0 - s * a2;                // 1/13!
  s = 1.0 / 39916800.0 - s * a2;                  // 1/11!
  s = 1.0 / 362880.0 - s * a2;                    // 1/9!
  s = 1.0 / 5040.0 - s * a2;                      // 1/7!
  s = 1.0 / 120.0 - s * a2;                       // 1/5!
  s = 1.0 / 6.0 - s * a2;                         // 1/3!
  s = (1.0 - s * a2) * a;
  return q == 0 ? c : q == 1 ? -s : q == 2 ? -c : s;
}

// ---- distributions ----------------------------------------------------------------------
TG_HD uint64_t tg_geom005(tg_rng& r) {  // support {0, 1, ...}, p = 0.05
  const double u = tg_u01(r.next());
  return (uint64_t)(tg_log(1.0 - u) / -0.05129329438755058);
}
TG_HD uint64_t tg_lognormal(tg_rng& r, double mu, double sigma) {  // Box-Muller, one variate
  const double u1 = tg_u01(r.next());
  const double u2 = tg_u01(r.next());
  const double z = sqrt(-2.0 * tg_log(1.0 - u1)) * tg_cos2pi(u2);
  return (uint64_t)tg_exp(mu + sigma * z);
}
TG_HD uint64_t tg_pareto15(tg_rng& r, double xm) {  // alpha = 1.5, capped so ns fit easily
  const double u = tg_u01(r.next());
  double e = -0.6666666666666666 * tg_log(1.0 - u);
  if (e > 20.0) e = 20.0;
  return (uint64_t)(xm * tg_exp(e));
}

// ---- emitter: applies defects, counts, writes, truncates --------------------------------
struct tg_emitter {
  tg_event* out;   // null = count only
  uint64_t n;      // events produced so far
  uint64_t limit;  // stop writing at this many events (truncation)
  tg_rng drng;     // defect decisions, separate from the program's draws
  uint64_t thr_dup, thr_drop;
  TG_HD void put(uint64_t ts, uint32_t tag, uint32_t ctx) {
    if (n < limit && out) { out[n].ts = ts; out[n].tag = tag; out[n].ctx = ctx; }
    n += 1;
  }
  TG_HD void marker(uint64_t ts, uint32_t region, uint32_t is_end, uint32_t ctx) {
    const uint64_t x = drng.next();
    const uint32_t tag = (region << 1) | is_end;
    if (is_end) {
      if (x < thr_drop) return;
      put(ts, tag, ctx);
    } else {
      put(ts, tag, ctx);
      if (x < thr_dup) put(ts, tag, ctx);
    }
  }
};

// ---- per-stream programs ----------------------------------------------------------------
struct tg_clock {
  uint64_t t;
  tg_rng r;
  tg_emitter* em;
  TG_HD void begin(uint32_t region, uint32_t ctx) { t += tg_geom005(r); em->marker(t, region, 0, ctx); }
  TG_HD void end(uint32_t region, uint32_t ctx) { t += tg_geom005(r); em->marker(t, region, 1, ctx); }
  TG_HD void leaf(uint32_t region, uint32_t ctx, uint64_t dur) {  // begin, dur ns, end (no extra gap)
    t += tg_geom005(r);
    em->marker(t, region, 0, ctx);
    t += dur;
    em->marker(t, region, 1, ctx);
  }
  TG_HD uint64_t work() { return tg_lognormal(r, 6.0, 0.8); }
};

#define TG_T_BASE 1700000000000000000ull

TG_HD void tg_prog_tiny(const tg_params& p, tg_clock& c) {
  // random well-formed program of exactly p.iters events, height <= 3, self-nesting allowed
  uint32_t stack[3];
  uint32_t h = 0, ctx = 0;
  for (uint32_t rem = p.iters; rem > 0; --rem) {
    const uint64_t x = c.r.next();
    const bool can_begin = h < 3 && h + 2 <= rem;  // leave room to close everything
    bool do_begin;
    if (h == 0) do_begin = true;
    else if (!can_begin) do_begin = false;
    else do_begin = (x >> 63) != 0;
    c.t += tg_geom005(c.r);
    if (do_begin) {
      const uint32_t region = (uint32_t)((x >> 8) & 7u);
      if (h == 0) ctx = (uint32_t)((x >> 16) & 15u);
      stack[h++] = region;
      c.em->marker(c.t, region, 0, ctx);
    } else {
      c.em->marker(c.t, stack[--h], 1, ctx);
    }
  }
}

TG_HD void tg_prog_gemm(const tg_params& p, uint32_t warp, tg_clock& c) {
  enum { TILE_LOOP = 0, TMA_LOAD = 1, MMA = 2, EPILOGUE = 3, BARRIER_WAIT = 4 };
  for (uint32_t it = 0; it < p.iters; ++it) {
    c.begin(TILE_LOOP, it);
    if (warp < 2) {
      const uint32_t op = warp == 0 ? TMA_LOAD : MMA;
      for (int k = 0; k < 8; ++k) {
        c.begin(op, it);
        c.leaf(BARRIER_WAIT, it, c.work());
        c.end(op, it);
      }
      c.leaf(BARRIER_WAIT, it, c.work());
    } else {
      c.leaf(BARRIER_WAIT, it, c.work());
      c.begin(EPILOGUE, it);
      for (int k = 0; k < 5; ++k) c.leaf(BARRIER_WAIT, it, c.work());
      c.end(EPILOGUE, it);
    }
    c.end(TILE_LOOP, it);
  }
}

TG_HD void tg_prog_attention(const tg_params& p, uint32_t cta, uint32_t warp, tg_clock& c) {
  enum { ATTN_TILE = 0, KV_ITER = 1, LOAD_KV = 2, QK_MMA = 3, SOFTMAX = 4, PV_MMA = 5, CORRECTION = 6, STORE_O = 7, WAIT = 8 };
  const uint64_t t0 = TG_T_BASE + 64ull * cta;
  for (uint32_t tile = 0; tile < p.iters; ++tile) {
    c.begin(ATTN_TILE, tile * p.inner);
    if (warp >= 14) {
      const uint32_t ctx = tile * p.inner;
      c.leaf(WAIT, ctx, c.work());
      c.begin(STORE_O, ctx);
      c.leaf(WAIT, ctx, c.work());
      c.end(STORE_O, ctx);
    } else {
      for (uint32_t kv = 0; kv < p.inner; ++kv) {
        const uint32_t ctx = tile * p.inner + kv;
        // warps of a CTA re-align at each KV iteration so producer/consumer spans overlap
        c.t += tg_geom005(c.r);
        const uint64_t aligned = t0 + 2048ull * ctx;
        if (c.t < aligned) c.t = aligned;
        c.em->marker(c.t, KV_ITER, 0, ctx);
        if (warp < 2) {
          const uint32_t a = warp == 0 ? LOAD_KV : QK_MMA;
          const uint32_t b = warp == 0 ? LOAD_KV : PV_MMA;
          c.begin(a, ctx); c.leaf(WAIT, ctx, c.work()); c.end(a, ctx);
          c.begin(b, ctx); c.leaf(WAIT, ctx, c.work()); c.end(b, ctx);
        } else {
          c.leaf(WAIT, ctx, c.work());
          c.leaf(warp < 10 ? SOFTMAX : CORRECTION, ctx, c.work());
        }
        c.end(KV_ITER, ctx);
      }
    }
    c.end(ATTN_TILE, tile * p.inner);
  }
}

TG_HD void tg_prog_decode(const tg_params& p, tg_clock& c) {
  enum { TOKEN_STEP = 0, LAYER = 1, TILE_WORK = 2, SYNC_WAIT = 3, OP_BASE = 4 };
  for (uint32_t tok = 0; tok < p.iters; ++tok) {
    c.begin(TOKEN_STEP, tok);
    for (uint32_t layer = 0; layer < p.inner; ++layer) {
      c.begin(LAYER, tok);
      for (uint32_t op = 0; op < 8; ++op) {
        const uint32_t region = OP_BASE + 9 * layer + op;
        c.begin(region, tok);
        for (int k = 0; k < 2; ++k) {
          c.begin(TILE_WORK, tok);
          c.t += c.work();
          c.leaf(SYNC_WAIT, tok, tg_pareto15(c.r, 100.0));
          c.end(TILE_WORK, tok);
        }
        c.end(region, tok);
      }
      const uint32_t allsync = OP_BASE + 9 * layer + 8;
      c.begin(allsync, tok);
      for (int k = 0; k < 4; ++k) c.leaf(SYNC_WAIT, tok, tg_pareto15(c.r, 100.0));
      c.end(allsync, tok);
      c.end(LAYER, tok);
    }
    c.end(TOKEN_STEP, tok);
  }
}

// Runs stream `s` into `out` (null = count only), writing at most `limit` events.
// Returns the number of events the un-truncated stream has.
TG_HD uint64_t tg_run_stream(const tg_params& p, uint32_t s, tg_event* out, uint64_t limit) {
  const uint32_t W = tg_warps_per_cta(p.kind);
  const uint32_t cta = s / W, warp = s % W;
  tg_emitter em;
  em.out = out; em.n = 0; em.limit = limit;
  em.drng = tg_make_rng(p.seed, s, 1);
  em.thr_dup = p.thr_dup_begin; em.thr_drop = p.thr_drop_end;
  tg_clock c;
  c.r = tg_make_rng(p.seed, s, 0);
  c.em = &em;
  c.t = TG_T_BASE + 64ull * cta + tg_geom005(c.r);
  if (p.kind == TG_TINY) tg_prog_tiny(p, c);
  else if (p.kind == TG_GEMM) tg_prog_gemm(p, warp, c);
  else if (p.kind == TG_ATTENTION) tg_prog_attention(p, cta, warp, c);
  else tg_prog_decode(p, c);
  return em.n;
}

// Length of stream `s` after truncation, given its un-truncated length.
TG_HD uint64_t tg_truncated_len(const tg_params& p, uint32_t s, uint64_t full) {
  tg_rng r = tg_make_rng(p.seed, s, 2);
  const uint64_t pick = r.next();
  const double u = tg_u01(r.next());
  if (pick < p.thr_trunc) return (uint64_t)(u * (double)full);
  return full;
}

#endif  // ARGUS_TRACEGEN_H_
