// Body of the placement / routing solver, shared by the solver kernel and by the combined
// solver + per-token kernel of the two-kernel chain for small calls.  See solve.cu for the method.
#pragma once

#include <limits.h>

#include "topoep_internal.cuh"

namespace topoep {

namespace {

constexpr int kRankCap = 128;   // stage 1 ranks up to this many candidates of a domain all-pairs

struct SolveLayout {
  size_t cand, col_main, col_rep, stat, mrank, mlocal, host_lo, host_hi, col_expert, col_cr, hostcol,
      sdom, col_rank, D, qd, U, L, used, cnt, win_e, win_v, est, nwin, total;
};

// The static block: everything that depends only on the handle and the domain, laid out in the
// workspace exactly as in shared memory so that one contiguous copy brings it in.
//   ints:   mrank[E] mlocal[E] host_lo[E] host_hi[E] col_expert[C] col_cr[C]
//   shorts: hostcol[G*E] sdom[R] col_rank[C]
__host__ __device__ inline size_t solve_static_ints(const Dims& d) {
  const size_t ints = 4 * (size_t)d.E + 2 * (size_t)d.C;
  const size_t shorts = (size_t)d.G * d.E + d.R + d.C;
  return (ints + (shorts + 1) / 2 + 3) & ~(size_t)3;
}

__host__ __device__ inline SolveLayout solve_layout(const Dims& d) {
  auto pad4 = [](size_t ints) { return (ints + 3) & ~(size_t)3; };
  SolveLayout o;
  size_t at = 0;
  o.col_main = at;   at += sizeof(int) * pad4((size_t)d.G * d.e_loc * d.R);   // [G*e_loc][R]
  o.col_rep = at;    at += sizeof(int) * pad4((size_t)d.G * d.N * d.R);       // [G*N][R]
  o.stat = at;
  o.mrank = at;      at += sizeof(int) * (size_t)d.E;
  o.mlocal = at;     at += sizeof(int) * (size_t)d.E;
  o.host_lo = at;    at += sizeof(int) * (size_t)d.E;
  o.host_hi = at;    at += sizeof(int) * (size_t)d.E;
  o.col_expert = at; at += sizeof(int) * (size_t)d.C;
  o.col_cr = at;     at += sizeof(int) * (size_t)d.C;
  o.hostcol = at;    at += sizeof(short) * (size_t)d.G * d.E;
  o.sdom = at;       at += sizeof(short) * (size_t)d.R;
  o.col_rank = at;   at += sizeof(short) * (size_t)d.C;
  at = o.stat + sizeof(int) * solve_static_ints(d);
  o.D = at;          at += sizeof(int) * pad4((size_t)d.M * d.E);
  // the candidate lists of inter-node placement (one per warp) are dead before the first q is
  // written: they share the q block's bytes, so that at 128 ranks two blocks still fit an SM
  o.qd = at;
  o.cand = at;
  {
    const size_t q_bytes = sizeof(int) * (size_t)d.R * d.qstride;
    const size_t cand_bytes = sizeof(unsigned long long) * (size_t)kRankCap * (kSolveThreads / 32);
    at += ((q_bytes > cand_bytes ? q_bytes : cand_bytes) + 15) & ~(size_t)15;
  }
  o.U = at;          at += sizeof(int) * (size_t)d.C;
  o.L = at;          at += sizeof(int) * (size_t)d.G;
  o.used = at;       at += sizeof(int) * (size_t)d.G;
  o.cnt = at;        at += sizeof(int) * (size_t)d.R * d.G;
  o.win_e = at;      at += sizeof(int) * (size_t)d.G * d.N;   // LPT policy: stage-1 winners in order
  o.win_v = at;      at += sizeof(int) * (size_t)d.G * d.N;   //             and their demand
  at = (at + 7) & ~(size_t)7;
  o.est = at;        at += sizeof(long long) * (size_t)d.G;   //             estimated rank loads
  o.nwin = at;       at += sizeof(int) * (size_t)d.M;         // replicas inter-node placement made, per domain
  o.total = (at + 15) & ~(size_t)15;
  return o;
}

// n ints global -> shared, 16 bytes at a time when both sides allow it.
__device__ __forceinline__ void copy_async(int* dst, const int32_t* src, int n, int tid, int nt) {
  if ((n & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
#pragma unroll 1
    for (int i = tid; i < n / 4; i += nt) cp_async16(dst + 4 * i, src + 4 * i);
  } else {
#pragma unroll 1
    for (int i = tid; i < n; i += nt) cp_async4(dst + i, src + i);
  }
}

// Policy variant of inter-node placement (kept out of line: it is rarely on, and the solver's
// straight-line code is fetch-bound): the winners, in candidate order, each to the rank with a
// free slot and the smallest estimated load (demand on its main instances + demand of the
// replicas it already took); ties to the lowest rank.  Sequential by nature: one lane deals.
__device__ __noinline__ void lpt_deal(const int* col_main, long long* est, const int* win_e,
                                      const int* win_v, int* used, int* col_expert, int* col_cr,
                                      short* hostcol, int n_win, int G, int R, int E, int e_loc,
                                      int s_phys, int stage1_slots, int cost_rank_inter, int lane) {
  const unsigned full = 0xffffffffu;
  __syncwarp();
  for (int g = 0; g < G; ++g) {   // main-instance demand of rank g: its columns, all sources
    long long sum = 0;
#pragma unroll 1
    for (int l = 0; l < e_loc; ++l) {
      if (col_expert[g * s_phys + l] < 0) continue;   // a rank with fewer mains: no such column
#pragma unroll 1
      for (int i = lane; i < R; i += 32) sum += col_main[((size_t)g * e_loc + l) * R + i];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(full, sum, o);
    if (lane == 0) est[g] = sum;
  }
  __syncwarp();
  if (lane == 0) {
#pragma unroll 1
    for (int k = 0; k < n_win; ++k) {
      int bg = -1;
#pragma unroll 1
      for (int g = 0; g < G; ++g)
        if (used[g] < stage1_slots && (bg < 0 || est[g] < est[bg])) bg = g;
      const int e = win_e[k], col = bg * s_phys + e_loc + used[bg];   // n_win <= G * slots
      col_expert[col] = e;
      col_cr[col] = cost_rank_inter;
      hostcol[bg * E + e] = (short)col;
      used[bg] += 1;
      est[bg] += win_v[k];
    }
  }
  __syncwarp();
}

// LPT: the least-loaded-rank policy of inter-node placement is compiled in (a separate
// instantiation: the default kernel is fetch-bound and carries no code it never runs).
template <bool LPT>
__device__ __forceinline__ void solve_body(const SolveParams& p, unsigned char* smem, int dm, int b) {
  const Dims d = p.d;
  const int M = d.M, G = d.G, R = d.R, E = d.E, N = d.N, C = d.C, QS = d.qstride;
  const int s_phys = d.s_phys, e_loc = d.e_loc;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const unsigned full = 0xffffffffu;
  if (p.pdl == 2) pdl_trigger();

  const SolveLayout lay = solve_layout(d);
  unsigned long long* cand_all = reinterpret_cast<unsigned long long*>(smem + lay.cand);
  int* col_main = reinterpret_cast<int*>(smem + lay.col_main);
  int* col_rep = reinterpret_cast<int*>(smem + lay.col_rep);
  int* mrank = reinterpret_cast<int*>(smem + lay.mrank);
  int* mlocal = reinterpret_cast<int*>(smem + lay.mlocal);
  int* D = reinterpret_cast<int*>(smem + lay.D);
  int* qd = reinterpret_cast<int*>(smem + lay.qd);
  unsigned* host_lo = reinterpret_cast<unsigned*>(smem + lay.host_lo);   // hosting domains 0..31
  unsigned* host_hi = reinterpret_cast<unsigned*>(smem + lay.host_hi);   // hosting domains 32..63
  int* col_expert = reinterpret_cast<int*>(smem + lay.col_expert);
  int* col_cr = reinterpret_cast<int*>(smem + lay.col_cr);
  int* U = reinterpret_cast<int*>(smem + lay.U);
  int* L = reinterpret_cast<int*>(smem + lay.L);
  int* used = reinterpret_cast<int*>(smem + lay.used);
  int* cnt = reinterpret_cast<int*>(smem + lay.cnt);
  int* win_e = reinterpret_cast<int*>(smem + lay.win_e);
  int* win_v = reinterpret_cast<int*>(smem + lay.win_v);
  long long* est = reinterpret_cast<long long*>(smem + lay.est);
  int* nwin = reinterpret_cast<int*>(smem + lay.nwin);
  short* hostcol = reinterpret_cast<short*>(smem + lay.hostcol);
  const short* sdom = reinterpret_cast<const short*>(smem + lay.sdom);
  const short* col_rank = reinterpret_cast<const short*>(smem + lay.col_rank);   // rank of a column

  const int32_t* om_m = p.ws.omega_m + (size_t)b * R * e_loc * R;   // rows = main instances
  // In the combined kernel the placement blocks publish inter-node placement: this block reads
  // the records instead of loading the demand of every domain and ranking every domain's
  // candidates again (the least-loaded-rank policy needs the demand values: it keeps doing so).
  // The records are staged where the demand would have been.
  const int GNw = G * N;
  // Worth the wait for the records only where the demand is large (many domains, many experts):
  // a small one is loaded and ranked sooner than the placement blocks' result arrives.
  const bool from_records = p.fused && !LPT && GNw + 1 <= E && M > 1 && p.stage1_slots > 0 && M * E >= 4096;

  // ---- first batch of asynchronous copies: the static block of this domain first (main-rank tables,
  // hosting masks and column tables as they are before any replica exists), then -- once the
  // omega kernel is done -- the demand and this domain's main columns
  copy_async(reinterpret_cast<int*>(smem + lay.stat),
             p.ws.solve_static + (size_t)dm * solve_static_ints(d), (int)solve_static_ints(d), tid, nt);
  if (tid < G) used[tid] = 0;
  if (tid < M) nwin[tid] = 0;
#pragma unroll 1
  for (int i = tid; i < R * G; i += nt) cnt[i] = 0;
  if (!p.acc) {
    pdl_wait();
    if (!from_records) copy_async(D, p.ws.demand + (size_t)b * M * E, M * E, tid, nt);
    copy_async(col_main, om_m + (size_t)dm * G * e_loc * R, G * e_loc * R, tid, nt);
    cp_async_wait_all();
    __syncthreads();
  } else {
    // Two-kernel chain: the histogram kernel summed the routing matrix and the demand into the
    // accumulators (one pair holds the sums, the other zeros: add them).  The static block must
    // be in first, it names the experts of the columns.
    cp_async_wait_all();
    __syncthreads();
    pdl_wait();
    const int32_t* dA = p.ws.acc_demand[0] + (size_t)b * M * E;
    const int32_t* dB = p.ws.acc_demand[1] + (size_t)b * M * E;
    if (!from_records) {
#pragma unroll 4
      for (int i = tid; i < M * E; i += nt) D[i] = __ldcg(dA + i) + __ldcg(dB + i);
    }
    // main columns: a warp step covers 8 columns x 4 sources (blocked main maps: one sector each)
    const int32_t* oA = p.ws.acc_omega[0] + (size_t)b * R * E;
    const int32_t* oB = p.ws.acc_omega[1] + (size_t)b * R * E;
    const int ncols = G * e_loc, nc8 = (ncols + 7) / 8, ns4 = (R + 3) / 4;
#pragma unroll 2
    for (int task = warp; task < nc8 * ns4; task += nwarps) {
      const int cb = task % nc8, sb = task / nc8;
      const int c = cb * 8 + (lane & 7), s = sb * 4 + (lane >> 3);
      if (c < ncols && s < R) {
        const int g = c / e_loc, l = c - g * e_loc;
        const int e = col_expert[g * s_phys + l];
        col_main[c * R + s] = e < 0 ? 0 : __ldcg(oA + (size_t)s * E + e) + __ldcg(oB + (size_t)s * E + e);
      }
    }
    __syncthreads();
    if (p.ws.demand && !from_records) {   // kept for inspection (debug tensor); row dm by this CTA
#pragma unroll 1
      for (int e = tid; e < E; e += nt) p.ws.demand[((size_t)b * M + dm) * E + e] = D[dm * E + e];
    }
  }

  // ---- inter-node placement, every domain, one warp each ------------------------------------
  // Candidates in descending (b, then ascending e) order == descending (D, ascending e) for a
  // uniform ||W|| and S_tok; the i-th goes to rank i mod G, slot i / G (fewest used slots first,
  // ties to the lower rank).
  if (from_records) {
    const unsigned serial = __ldcg(p.ws.epoch + 4);
    const unsigned long long* rec = p.ws.place_rec + (size_t)b * M * (GNw + 1);
    int* recs = D;   // [M][GN + 1]: count, winners in rank order
    bool all = false;
#pragma unroll 1
    for (unsigned it = 0; it < kFlagWaitLimit && !all; ++it) {
      bool ok = true;
#pragma unroll 1
      for (int i = tid; i < M * (GNw + 1); i += nt) {
        const unsigned long long w = __ldcg(rec + i);
        ok = ok && (unsigned)(w >> 32) == serial;
        recs[i] = (int)(unsigned)w;
      }
      all = __syncthreads_and(ok);
    }
    if (!all && tid == 0) atomicOr(p.ws.status, TOPOEP_FLAG_INTERNAL);
    // hosting masks of every domain's winners; this domain's winners into its columns: the i-th
    // to rank i mod G, slot i / G
#pragma unroll 1
    for (int i = tid; i < M * GNw; i += nt) {
      const int dd = i / GNw, k = i - dd * GNw;
      const int n = all ? min(max(recs[dd * (GNw + 1)], 0), GNw) : 0;
      if (k == 0) nwin[dd] = n;
      if (k >= n) continue;
      const int e = CK(p.ws.status, recs[dd * (GNw + 1) + 1 + k], E);
      if (dd < 32) atomicOr(&host_lo[e], 1u << dd); else atomicOr(&host_hi[e], 1u << (dd - 32));
      if (dd == dm) {
        const int g = k % G, j = k / G, col = g * s_phys + e_loc + j;
        col_expert[col] = e;
        col_cr[col] = p.cost_rank_inter;   // its main lies in another domain
        hostcol[g * E + e] = (short)col;
        atomicMax(&used[g], j + 1);
      }
    }
  } else if (M > 1 && p.stage1_slots > 0) {
    const int slots = G * p.stage1_slots;   // all N per rank unless some are reserved
#pragma unroll 1
    for (int dd = warp; dd < M; dd += nwarps) {
      int* Dd = D + dd * E;
      // compact the candidates (D > 0) of this domain into cand[]: key = (D, -e)
      unsigned long long* cand = cand_all + (size_t)warp * kRankCap;
      int n_c = 0;
#pragma unroll 1
      for (int e0 = 0; e0 < E; e0 += 32) {
        const int e = e0 + lane;
        int v = 0;
        if (e < E) {
          // a candidate has positive benefit (D above the threshold) and its main elsewhere; bit dd
          // of the mask is still the main-domain bit here: only this warp ever sets it, below
          const unsigned hosted = dd < 32 ? host_lo[e] >> dd : host_hi[e] >> (dd - 32);
          v = (hosted & 1u) ? 0 : Dd[e];
          v = v > p.cand_thr ? v : 0;
        }
        const unsigned m = __ballot_sync(full, v > 0);
        const int at = n_c + __popc(m & lanemask_lt());
        if (v > 0 && at < kRankCap)
          cand[at] = ((unsigned long long)(unsigned)v << 32) | (unsigned)~(unsigned)e;
        n_c += __popc(m);
      }
      __syncwarp();
      int n_win = 0;   // candidates that get a slot
      if (n_c <= kRankCap) {
        n_win = min(n_c, slots);
        // few candidates: every candidate counts the keys above its own; rank < slots wins
#pragma unroll 1
        for (int c0 = 0; c0 < n_c; c0 += 32) {
          const int c = c0 + lane;
          const unsigned long long mine = c < n_c ? cand[c] : 0ull;
          int rank = 0;
          for (int o = 0; o < n_c; ++o) rank += cand[o] > mine ? 1 : 0;
          if (c < n_c && rank < slots) {
            const int e = (int)~(unsigned)mine;
            if (dd < 32) atomicOr(&host_lo[e], 1u << dd); else atomicOr(&host_hi[e], 1u << (dd - 32));
            if (LPT && dd == dm) {
              win_e[rank] = e;                   // placed below, in order, by estimated load
              win_v[rank] = (int)(mine >> 32);
            } else if (dd == dm) {
              const int g = rank % G, j = rank / G, col = g * s_phys + e_loc + j;
              col_expert[col] = e;
              col_cr[col] = p.cost_rank_inter;   // its main lies in another domain
              hostcol[g * E + e] = (short)col;
              atomicMax(&used[g], j + 1);
            }
          }
        }
      } else {
        // many candidates: pick the maximum slot by slot (non-candidates are zeroed first)
#pragma unroll 1
        for (int e = lane; e < E; e += 32) {
          const unsigned hosted = dd < 32 ? host_lo[e] >> dd : host_hi[e] >> (dd - 32);
          if ((hosted & 1u) || Dd[e] <= p.cand_thr) Dd[e] = 0;
        }
        __syncwarp();
#pragma unroll 1
        for (int i = 0; i < slots; ++i) {
          int bestD = 0, bestE = INT_MAX;
#pragma unroll 1
          for (int e = lane; e < E; e += 32) {
            const int x = Dd[e];
            if (x > bestD) { bestD = x; bestE = e; }   // ascending e: first hit is smallest
          }
          const int maxD = __reduce_max_sync(full, bestD);
          if (maxD <= 0) break;
          n_win = i + 1;
          const int e = __reduce_min_sync(full, bestD == maxD ? bestE : INT_MAX);
          if (lane == 0) {
            Dd[e] = 0;   // taken
            if (dd < 32) atomicOr(&host_lo[e], 1u << dd); else atomicOr(&host_hi[e], 1u << (dd - 32));
            if (LPT && dd == dm) {
              win_e[i] = e;
              win_v[i] = maxD;
            } else if (dd == dm) {
              const int g = i % G, j = i / G, col = g * s_phys + e_loc + j;
              col_expert[col] = e;
              col_cr[col] = p.cost_rank_inter;
              hostcol[g * E + e] = (short)col;
              used[g] = j + 1;
            }
          }
          __syncwarp();
        }
      }
      if (LPT && dd == dm)
        lpt_deal(col_main, est, win_e, win_v, used, col_expert, col_cr, hostcol, n_win, G, R, E, e_loc,
                 s_phys, p.stage1_slots, p.cost_rank_inter, lane);
      if (lane == 0) nwin[dd] = n_win;
    }
  }
  __syncthreads();
  // Two-kernel chain: when inter-node placement used every slot of every domain, the refinement
  // cannot act (a move needs a target with a free slot) and the whole plan follows in closed form
  // from the routing matrix and this placement.  The rank blocks of the grid produce it then,
  // spread over R blocks instead of M, and this block has nothing left to do.
  if (p.fused && !LPT) {
    bool closed = true;
    if (N > 0) {
      if (M == 1 || p.stage1_slots != N) closed = false;
#pragma unroll 1
      for (int dd = 0; dd < M; ++dd) closed = closed && nwin[dd] == G * N;
    }
    if (closed) return;
  }

  TL_MAX(p.ws, 20);   // inter-node placement known
  // ---- second batch of asynchronous copies: the routing-matrix columns of this domain's replicas ----
#pragma unroll 1
  for (int i = warp; i < G * N; i += nwarps) {
    const int e = col_expert[(i / N) * s_phys + e_loc + i % N];
    if (e < 0) continue;
    if (p.acc) {
      const int32_t* oA = p.ws.acc_omega[0] + (size_t)b * R * E + e;
      const int32_t* oB = p.ws.acc_omega[1] + (size_t)b * R * E + e;
#pragma unroll 1
      for (int s = lane; s < R; s += 32)
        col_rep[i * R + s] = __ldcg(oA + (size_t)s * E) + __ldcg(oB + (size_t)s * E);
      continue;
    }
    const int32_t* src = om_m + (size_t)(mrank[e] * e_loc + mlocal[e]) * R;
    copy_async(col_rep + i * R, src, R, lane, 32);
  }

  // ---- routing construction for the columns of this domain ----------------------------------
  // After stage 1 an expert has at most one instance per domain.  A source keeps everything in
  // its own domain when an instance is there; otherwise it splits over all instances (ascending
  // rank == ascending hosting domain), remainder to `rem` instances starting at (s+e) mod n.
  // A warp takes a column, its lanes the sources; main columns first, replica columns once their
  // copies have landed.
#pragma unroll 1
  for (int pass = 0; pass < 2; ++pass) {
    if (pass == 1) {
      cp_async_wait_all();
      __syncthreads();
    }
    const int ncols = pass == 0 ? G * e_loc : G * N;
    const int per = pass == 0 ? e_loc : N;
    const int* w_base = pass == 0 ? col_main : col_rep;
    // four columns of a warp at a time, so that their dependent shared-memory reads overlap
    constexpr int kCols = 4;
#pragma unroll 1
    for (int i0 = warp; i0 < ncols; i0 += kCols * nwarps) {
      int c[kCols], e[kCols], n[kCols], idx[kCols], usum[kCols];
      unsigned long long hm[kCols];
#pragma unroll
      for (int u = 0; u < kCols; ++u) {
        const int i = i0 + u * nwarps;
        const int g = i / per, l = i - g * per;
        c[u] = g * s_phys + (pass == 0 ? l : e_loc + l);
        e[u] = i < ncols ? col_expert[c[u]] : -2;   // -1: empty slot, -2: no such column
        usum[u] = 0;
      }
#pragma unroll
      for (int u = 0; u < kCols; ++u) {
        hm[u] = 0;
        n[u] = 1;
        idx[u] = 0;
        if (e[u] >= 0) {
          hm[u] = ((unsigned long long)host_hi[e[u]] << 32) | host_lo[e[u]];
          n[u] = __popcll(hm[u]);
          idx[u] = __popcll(hm[u] & ((1ull << dm) - 1ull));
        }
      }
#pragma unroll 1
      for (int s0 = 0; s0 < R; s0 += 32) {
        const int s = s0 + lane;
        const int ds = s < R ? sdom[s] : 0;
#pragma unroll
        for (int u = 0; u < kCols; ++u) {
          int v = 0;
          if (s < R && e[u] >= 0) {
            const int w = w_base[(i0 + u * nwarps) * R + s];
            if (ds == dm || n[u] == 1) {   // own domain, or the only instance anywhere
              v = w;
            } else if (!((hm[u] >> ds) & 1ull)) {
              const int base = w / n[u], rem = w - base * n[u];
              int sh = idx[u] - (s + e[u]) % n[u];
              if (sh < 0) sh += n[u];
              v = base + (sh < rem ? 1 : 0);
            }
          }
          if (s < R && e[u] >= -1) qd[s * QS + c[u]] = v;
          usum[u] += v;
        }
      }
#pragma unroll
      for (int u = 0; u < kCols; ++u) {
        const int tot = __reduce_add_sync(full, usum[u]);
        if (lane == 0 && e[u] >= -1) U[c[u]] = tot;
      }
    }
  }
  __syncthreads();
  if (tid < G) {
    int sum = 0;
#pragma unroll 1
    for (int l = 0; l < s_phys; ++l) sum += U[tid * s_phys + l];
    L[tid] = sum;
  }
  __syncthreads();

  TL_MAX(p.ws, 21);   // routing constructed, loads known
  // ---- intra-node refinement: warp 0, one commit per iteration ------------------------------
  if (warp == 0) {
    int it = 0;
    const int chunk = (R + 31) / 32;
    // lane -> (target rank gt, start slot k0): lanes gt, gt+G, ... share a target and stride the
    // instance slots of the busiest rank
    const int gt = lane % G, k0 = lane / G, kstep = max(32 / G, 1);
    const bool lane_on = lane < G * kstep;
    // Inter-node placement leaves an expert at most one instance per domain, so a move needs a
    // target with a free slot; when every slot of the domain is taken there is nothing to do.
    // lane g keeps L_g and the used-slot count of rank g in registers for the whole loop
    int Lreg = lane < G ? L[lane] : -1;
    int usedreg = lane < G ? used[lane] : N;
    const bool any_free = __any_sync(full, usedreg < N);
    for (; any_free;) {
      const int Lb = __reduce_max_sync(full, Lreg);
      const int gb = __ffs(__ballot_sync(full, Lreg == Lb)) - 1;   // busiest, lowest id on ties
      const int Lt = __shfl_sync(full, Lreg, gt);
      const bool has_slot = __shfl_sync(full, usedreg, gt) < N;
      int bd = 0;
      unsigned bk = 0xffffffffu;
      const int half = (Lb - Lt) >> 1;                           // half-gap bound
      const bool on = lane_on && gt != gb && half >= p.min_delta;
      // Selects instead of branches: one warp runs this loop alone, so a taken branch costs more
      // than the handful of wasted table reads of a lane that has no candidate.
#pragma unroll 1
      for (int l = k0; l < s_phys; l += 2 * kstep) {
        const int cb0 = gb * s_phys + l;
        const bool two = l + kstep < s_phys;
        const int cb1 = two ? cb0 + kstep : cb0;
        const int e0 = col_expert[cb0], e1 = col_expert[cb1];
        const int u0 = U[cb0], u1 = U[cb1];
        const unsigned cr0 = (unsigned)col_cr[cb0], cr1 = (unsigned)col_cr[cb1];
        const int hc0 = hostcol[gt * E + max(e0, 0)];
        const int hc1 = hostcol[gt * E + max(e1, 0)];
        const int d0 = min(u0, half), d1 = min(u1, half);
        const bool ok0 = on && e0 >= 0 && u0 > 0 && (hc0 >= 0 || has_slot) && d0 >= p.min_delta;
        const bool ok1 = on && two && e1 >= 0 && u1 > 0 && (hc1 >= 0 || has_slot) && d1 >= p.min_delta;
        const unsigned key0 = ((hc0 >= 0 ? 0u : cr0) << 28) | ((unsigned)e0 << 5) | (unsigned)gt;
        const unsigned key1 = ((hc1 >= 0 ? 0u : cr1) << 28) | ((unsigned)e1 << 5) | (unsigned)gt;
        const bool b0 = ok0 && (d0 > bd || (d0 == bd && key0 < bk));
        bd = b0 ? d0 : bd;
        bk = b0 ? key0 : bk;
        const bool b1 = ok1 && (d1 > bd || (d1 == bd && key1 < bk));
        bd = b1 ? d1 : bd;
        bk = b1 ? key1 : bk;
      }
      const int bl = on ? Lt : INT_MAX;
      const int md = __reduce_max_sync(full, bd);
      if (md <= 0) break;
      const int ml = __reduce_min_sync(full, bd == md ? bl : INT_MAX);
      const unsigned mk = __reduce_min_sync(full, (bd == md && bl == ml) ? bk : 0xffffffffu);
      if (it >= p.max_iters) {
        if (lane == 0) atomicOr(p.ws.status, TOPOEP_FLAG_REFINE_CAP);
        break;
      }
      const int e = CK(p.ws.status, (int)((mk >> 5) & 0x7fffffu), E), wt = (int)(mk & 31u);
      const int cb = CK(p.ws.status, hostcol[gb * E + e], C);
      int ct = hostcol[wt * E + e];
      if (ct < 0) {   // create the replica in the target's next free slot
        ct = CK(p.ws.status, wt * s_phys + e_loc + __shfl_sync(full, usedreg, wt), C);
        if (lane == 0) {
          col_expert[ct] = e;
          col_cr[ct] = col_cr[cb];
          hostcol[wt * E + e] = (short)ct;
        }
        if (lane == wt) usedreg += 1;
      }
      // Move md units of q from column cb to ct; sources in the order: the target rank itself,
      // then the others ascending, the busiest rank last.  The lanes walk the sources in natural
      // order (a plain scan) and correct for the two that are out of place: in the required
      // order a source s other than those two is preceded by rt and by the lower sources except
      // rt and rb; rb is preceded by everything else.
      const int rb = dm * G + gb, rt = dm * G + wt;
      const int qrt = qd[rt * QS + cb], qrb = qd[rb * QS + cb];
      const int i0 = min(R, lane * chunk), i1 = min(R, i0 + chunk);
      if (chunk <= 4) {
        // up to 128 ranks: a lane's sources fit in registers, so both columns are read with
        // independent loads before the scan instead of one dependent load per source after it
        int v[4], w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int s = i0 + j;
          v[j] = s < i1 ? qd[s * QS + cb] : 0;
          w[j] = s < i1 ? qd[s * QS + ct] : 0;
        }
        int total;
        int pre = warp_exclusive_scan(v[0] + v[1] + v[2] + v[3], lane, &total);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int s = i0 + j;
          int before = qrt + pre - (rt < s ? qrt : 0) - (rb < s ? qrb : 0);
          before = s == rt ? 0 : before;
          before = s == rb ? total - qrb : before;
          const int take = min(max(md - before, 0), v[j]);
          if (s < i1 && take > 0) {
            qd[s * QS + cb] = v[j] - take;
            qd[s * QS + ct] = w[j] + take;
          }
          pre += v[j];
        }
      } else {
        int sum = 0;
#pragma unroll 1
        for (int s = i0; s < i1; ++s) sum += qd[s * QS + cb];
        int total;
        int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
        for (int s = i0; s < i1; ++s) {
          const int v = qd[s * QS + cb];
          int before = qrt + pre - (rt < s ? qrt : 0) - (rb < s ? qrb : 0);
          if (s == rt) before = 0;
          if (s == rb) before = total - qrb;
          const int take = min(max(md - before, 0), v);
          if (take > 0) {
            qd[s * QS + cb] = v - take;
            qd[s * QS + ct] += take;
          }
          pre += v;
        }
      }
      if (lane == 0) { U[cb] -= md; U[ct] += md; }
      if (lane == gb) Lreg -= md;
      if (lane == wt) Lreg += md;
      __syncwarp();
      ++it;
    }
    if (lane < G) { L[lane] = Lreg; used[lane] = usedreg; }
    if (lane == 0) p.ws.refine_iters[(size_t)b * M + dm] = it;
  }
  __syncthreads();

  TL_MAX(p.ws, 22);   // refinement done
  // ---- results of this domain ----------------------------------------------------------------
#pragma unroll 1
  for (int idx = tid; idx < G * N; idx += nt) {
    const int g = idx / N, j = idx - g * N;
    const int e = col_expert[g * s_phys + e_loc + j];
    const size_t at = ((size_t)b * R + dm * G + g) * N + j;
    p.ws.replica_map[at] = e;
    if (p.out_replica_map) p.out_replica_map[at] = e;
  }
#pragma unroll 1
  for (int c = tid; c < C; c += nt) {
    const int u = col_expert[c] >= 0 ? U[c] : 0;
    const size_t at = (size_t)b * d.P + (size_t)dm * C + c;
    p.ws.inst_counts[at] = u;
    if (p.out_inst_counts) p.out_inst_counts[at] = u;
  }
  if (tid < G) p.ws.rank_load[(size_t)b * R + dm * G + tid] = L[tid];
  // q rows of this domain's columns; counts[s][r] accumulated per (source, rank) on the way
#pragma unroll 1
  for (int s = warp; s < R; s += nwarps) {
    int32_t* qrow = p.ws.q + ((size_t)b * R + s) * d.P + (size_t)dm * C;
#pragma unroll 1
    for (int c = lane; c < C; c += 32) {
      const int v = qd[s * QS + c];
      qrow[c] = v;
      if (v != 0) atomicAdd(&cnt[s * G + col_rank[c]], v);
    }
  }
  __syncthreads();
#pragma unroll 1
  for (int i = tid; i < R * G; i += nt) {
    const int s = i / G, g = i - s * G;
    const size_t at = ((size_t)b * R + s) * R + dm * G + g;
    p.ws.counts[at] = cnt[i];
    p.out_counts[at] = cnt[i];
  }
  // receive offsets of rank r: exclusive scan over the sources, one warp per rank
#pragma unroll 1
  for (int g = warp; g < G; g += nwarps) {
    int32_t* recv = p.out_offsets + (((size_t)b * 2 + 1) * R + dm * G + g) * (R + 1);
    const int ch = (R + 31) / 32;
    const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
    int sum = 0;
#pragma unroll 1
    for (int s = i0; s < i1; ++s) sum += cnt[s * G + g];
    int total;
    int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
    for (int s = i0; s < i1; ++s) { recv[s] = pre; pre += cnt[s * G + g]; }
    if (lane == 0) recv[R] = total;
  }
  // Two-kernel chain: tell the per-token blocks of this grid that wait for the refinement that
  // this domain's results are in memory (the serial number of the call is the flag value, so the
  // flags never need clearing).
  if (p.fused) {
    __threadfence();
    __syncthreads();
    TL_MAX(p.ws, 16);
    if (tid == 0) {
      const unsigned serial = __ldcg(p.ws.epoch + 4);
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.ws.done_flags + (size_t)b * M + dm),
                   "r"(serial)
                   : "memory");
    }
  }
}

}  // namespace

}  // namespace topoep
