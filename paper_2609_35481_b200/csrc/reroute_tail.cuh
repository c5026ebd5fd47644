// Ranking tail of the per-token assignment, shared by the reroute kernel and by the per-token
// kernel of the three-kernel chain: the split assignments of a tile are ranked (stable, by flat
// index) with per-lane packed counters and dealt to the instances along their quota lists.
#pragma once

#include "topoep_internal.cuh"

namespace topoep {

namespace {

// Sum of the eight 4-bit fields of x (each field <= 4 here).
__device__ __forceinline__ int nibble_sum(unsigned x) {
  const unsigned y = (x & 0x0f0f0f0fu) + ((x >> 4) & 0x0f0f0f0fu);
  return (int)((y * 0x01010101u) >> 24);
}

// A work item is the position of a split assignment in the tile; its expert and the number of
// equal ids before it in its group of four are read back from the id array when it is processed.

// Everything the ranking of the split items needs.
struct SplitCtx {
  uint4* cnt4; unsigned* cntw; int* base; const int* route; int* seg; int* cum; int* inst;
  int* tbase; const unsigned short* work; const int32_t* rec; const int32_t* g_tp;
  const int32_t* ids; int32_t* out; SplitRec rl; int rows, n_split, n_list, n_work;
  uint32_t* status;
  bool lists_local;   // seg, cum and inst are complete in shared memory already (nothing to fetch)
};

// Rank the split items of the tile and patch their outputs (whole CTA).
__device__ __forceinline__ void rank_and_patch(const SplitCtx& c, int tid, int nt, int warp,
                                               int nwarps) {
  const int lane = tid & 31, rows = c.rows;
  auto sync = [] { __syncthreads(); };
  const bool fetch = !c.lists_local && (c.n_split > kSplitCap || c.n_list > kFastLists);
  if (fetch) {   // rare: fetch the rest of the record
#pragma unroll 1
    for (int i = tid; i <= c.n_split; i += nt) c.seg[i] = c.rec[c.rl.seg + i];
#pragma unroll 1
    for (int i = tid; i < c.n_list; i += nt) {
      c.cum[i] = c.rec[c.rl.cum + i];
      c.inst[i] = c.rec[c.rl.inst + i];
    }
  }
  bool broken = false;
#pragma unroll 1
  for (int p0 = 0; p0 < c.n_split; p0 += kSplitCap) {
    const int n_here = min(kSplitCap, c.n_split - p0);
    if (p0 > 0) {   // later passes: fresh counters and tile bases (the first set came up front)
#pragma unroll 1
      for (int i = tid; i < n_here * rows; i += nt) c.cnt4[i] = make_uint4(0u, 0u, 0u, 0u);
      if (tid < n_here) c.tbase[tid] = c.g_tp[p0 + tid];
    }
    if (p0 > 0 || fetch) sync();
    // every item bumps the 4-bit counter of its (split expert, row, lane)
#pragma unroll 1
    for (int w = tid; w < c.n_work; w += nt) {
      const int pos = CK(c.status, c.work[w], rows * 128);
      const int i = -2 - c.route[__ldg(c.ids + pos)] - p0;
      if (i < 0 || i >= n_here) continue;
      const int vec = pos >> 2;                            // int4 index inside the tile
      const int rr = vec >> 5, ln = vec & 31;              // row, lane inside the row
      atomicAdd(&c.cntw[(i * rows + rr) * 4 + (ln >> 3)], 1u << (4 * (ln & 7)));
    }
    sync();
    // base[i][rr] = tile base + ids of split expert i in rows before rr
#pragma unroll 1
    for (int i = warp; i < n_here; i += nwarps) {
      int carry = c.tbase[i];
#pragma unroll 1
      for (int r0 = 0; r0 < rows; r0 += 32) {
        const int rr = r0 + lane;
        int tot = 0;
        if (rr < rows) {
          const uint4 q = c.cnt4[i * rows + rr];
          tot = nibble_sum(q.x) + nibble_sum(q.y) + nibble_sum(q.z) + nibble_sum(q.w);
        }
        int all;
        const int ex = warp_exclusive_scan(tot, lane, &all);
        if (rr < rows) c.base[i * rows + rr] = carry + ex;
        carry += all;
      }
    }
    sync();
#pragma unroll 1
    for (int w = tid; w < c.n_work; w += nt) {
      const int pos = CK(c.status, c.work[w], rows * 128), vec = pos >> 2;
      const int e = __ldg(c.ids + pos);
      const int i = -2 - c.route[e] - p0;
      if (i < 0 || i >= n_here) continue;
      int prev = 0;   // equal ids earlier in the same group of four
#pragma unroll 1
      for (int u = pos & ~3; u < pos; ++u) prev += __ldg(c.ids + u) == e ? 1 : 0;
      const int rr = vec >> 5, ln = vec & 31, word = ln >> 3, shift = 4 * (ln & 7);
      const uint4 q = c.cnt4[i * rows + rr];
      const unsigned cw[4] = {q.x, q.y, q.z, q.w};
      int rho = c.base[i * rows + rr] + prev;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (u < word) rho += nibble_sum(cw[u]);
        else if (u == word) rho += nibble_sum(cw[u] & ((1u << shift) - 1u));
      }
      int at = c.seg[p0 + i];
      const int end = c.seg[p0 + i + 1] - 1;
      while (at < end && rho >= c.cum[at]) ++at;
      at = CK(c.status, at, c.n_list);
      broken |= rho >= c.cum[at];
      c.out[pos] = c.inst[at];
    }
    if (p0 + kSplitCap < c.n_split) sync();
  }
  if (broken) atomicOr(c.status, TOPOEP_FLAG_INTERNAL);
}

}  // namespace

}  // namespace topoep
