/*
 * Seeded synthetic router output: top-k expert ids per token.
 *
 * This file only draws inputs.  It holds none of the planning method's
 * arithmetic and is the one piece of code that both the CPU oracle's tests and
 * the CUDA path's tests/bench consume (they read the buffer it fills).
 *
 * Each token draws k DISTINCT experts one after another from a per-plan
 * categorical distribution given as a 63-bit integer CDF (sequential sampling
 * without replacement: a draw that repeats an earlier expert of the same token
 * is thrown away and redrawn).  Random bits come from a counter-based hash of
 * (seed, plan, rank, token, draw, attempt), so the output does not depend on
 * the number of threads or on the order tokens are generated in.
 */
#include <stdint.h>
#include <stddef.h>

static inline uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

/* Exposed so the Python side can derive permutations / parameters from the same stream. */
uint64_t wl_hash(uint64_t seed, uint64_t a, uint64_t b, uint64_t c) {
  uint64_t h = mix64(seed);
  h = mix64(h ^ a);
  h = mix64(h ^ b);
  h = mix64(h ^ c);
  return h;
}

/* First index i with u < cdf[i]; cdf is non-decreasing and cdf[n-1] = 2^63. */
static inline int upper_bound63(const uint64_t* cdf, int n, uint64_t u) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (u < cdf[mid]) hi = mid; else lo = mid + 1;
  }
  return lo;
}

/*
 * out[B][R][T][k] int32.  cdf[B][E] uint64.  plan_base is added to the plan
 * index inside the hash so a batch can be generated in pieces.
 * Returns 0, or -1 if k > E or k > 64.
 */
int wl_gen_topk(uint64_t seed, int64_t plan_base, int B, int R, int T, int k, int E,
                const uint64_t* cdf, int32_t* out) {
  if (k > E || k > 64 || k < 1) return -1;
  const int64_t rows = (int64_t)B * R;
#pragma omp parallel for schedule(static)
  for (int64_t row = 0; row < rows; ++row) {
    const int b = (int)(row / R), s = (int)(row % R);
    const uint64_t* c = cdf + (size_t)b * E;
    const uint64_t hrow = wl_hash(seed, (uint64_t)(plan_base + b), (uint64_t)s, 0x746f6b656e73ull);
    int32_t* o = out + (size_t)row * T * k;
    for (int t = 0; t < T; ++t) {
      const uint64_t htok = mix64(hrow ^ (uint64_t)t);
      int32_t chosen[64];
      for (int j = 0; j < k; ++j) {
        for (uint64_t attempt = 0;; ++attempt) {
          const uint64_t u = mix64(htok ^ ((uint64_t)j << 40) ^ attempt) >> 1;
          const int e = upper_bound63(c, E, u);
          int dup = 0;
          for (int i = 0; i < j; ++i) dup |= (chosen[i] == e);
          if (!dup) { chosen[j] = e; break; }
        }
        o[(size_t)t * k + j] = chosen[j];
      }
    }
  }
  return 0;
}
