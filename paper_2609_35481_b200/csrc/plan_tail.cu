// Second kernel of the two-kernel chain for small calls (paper, "Planning on the Critical Path":
// one (layer, microbatch) plan at a time sits in front of every MoE layer, so its latency, not
// its throughput, is what counts).
//
// Chain: accumulating histogram -> this kernel.  One grid, four kinds of blocks:
//
//   placement blocks (plan, domain)        inter-node placement of one domain, published;
//   solver blocks    (plan, domain)        the body of the solver kernel;
//   rank blocks      (plan, rank)          the plan in closed form, one rank's share of it;
//   per-token blocks (plan, source, tile)  the per-token assignment of one tile.
//
// A placement block ranks the candidates of its domain with all its warps and publishes the
// winners as a short record of 64-bit words, each tagged with the serial number of the call, so
// a reader knows a word is this call's without any other handshake.  Rank and per-token blocks
// poll the records of their plan (with a limit).  Code that runs once per block costs about 15
// cycles per instruction on this machine, so a block does as little of it as possible: what M
// blocks can compute once is not recomputed by hundreds.
// If the placement used every replica slot, intra-node refinement cannot act: a move needs a
// target with a free slot, because an expert has at most one instance per domain after
// inter-node placement.  Then the plan is a closed form of the routing matrix and the placement
// (paper, "Inter-node placement": routing construction, loads), and
//   * a per-token block derives the routing table of its source from row s of the routing matrix
//     and streams its tile without waiting for anybody: histogram -> per-token assignment is
//     the critical path;
//   * a rank block writes what belongs to rank r: row r of q, of the dispatch counts and of the
//     send offsets, its instance loads U, its rank load L, its receive offsets, its replica slots;
//   * the solver blocks return at once.
// Otherwise (some slot is free) the rank blocks return at once, the solver blocks run placement,
// routing and refinement as in the solver kernel and publish a flag each, and a per-token block
// waits for the flags of its plan (polled with a limit) and reads row s of q and the replica
// map.  The solver blocks have the lowest block indices, so they are scheduled first, and they
// wait for nobody: the wait cannot starve them.
//
// From the routing table on, a per-token block does what the reroute kernel does: tile prefixes,
// resolved tiles, stream, ranking tail.
#include <limits.h>

#include <algorithm>

#include "topoep_internal.cuh"
#include "reroute_tail.cuh"
#include "solve_body.cuh"

namespace topoep {

namespace {

constexpr int kP2RankCap = 128;                  // candidates of a domain ranked all-pairs
constexpr int kP2Warps = kSolveThreads / 32;     // every block of this kernel has this shape

__device__ __forceinline__ void cp_async16_cg(void* smem_dst, const void* gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}

// Exclusive scan of (flag[e], flag[e] * nz[e]) with flag = nz >= 2 over e < n by the whole CTA;
// results in out_a / out_b (entry n = totals).  Each thread owns a contiguous chunk.
__device__ __forceinline__ void tail_scan2(const int* nz, int n, int* out_a, int* out_b,
                                           int* warp_tot, int tid, int nt) {
  const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  const int chunk = (n + nt - 1) / nt;
  const int i0 = min(n, tid * chunk), i1 = min(n, i0 + chunk);
  int a = 0, b = 0;
#pragma unroll 1
  for (int i = i0; i < i1; ++i) {
    const int f = nz[i] >= 2;
    a += f;
    b += f ? nz[i] : 0;
  }
  int ta, tb;
  int ea = warp_exclusive_scan(a, lane, &ta);
  int eb = warp_exclusive_scan(b, lane, &tb);
  if (lane == 0) { warp_tot[warp] = ta; warp_tot[nw + warp] = tb; }
  __syncthreads();
  int ba = 0, bb = 0;
#pragma unroll 1
  for (int w = 0; w < warp; ++w) { ba += warp_tot[w]; bb += warp_tot[nw + w]; }
  ea += ba;
  eb += bb;
#pragma unroll 1
  for (int i = i0; i < i1; ++i) {
    const int f = nz[i] >= 2;
    out_a[i] = ea;
    out_b[i] = eb;
    ea += f;
    eb += f ? nz[i] : 0;
  }
  if (tid == nt - 1) { out_a[n] = ea; out_b[n] = eb; }
  __syncthreads();
}

// ---- placement blocks ----------------------------------------------------------------------------
// (Paper, "Inter-node placement": the candidates of a domain -- main instance elsewhere, positive
// benefit, i.e. demand above the threshold -- in descending order (D, then ascending e); the i-th
// winner goes to rank i mod G, slot i / G.)  Record of (plan, domain): GN + 1 words,
//   word 0     = serial << 32 | number of winners
//   word 1 + i = serial << 32 | i-th winner (0xffffffff: none)
struct PlaceLayout { size_t cand, D, mdom, chunk, winl, total; };

__host__ __device__ inline PlaceLayout place_layout(const Dims& d) {
  auto pad4 = [](size_t ints) { return (ints + 3) & ~(size_t)3; };
  PlaceLayout o;
  size_t at = 0;
  o.cand = at;  at += sizeof(unsigned long long) * (size_t)kP2RankCap;
  o.D = at;     at += sizeof(int) * pad4(d.E);
  o.mdom = at;  at += sizeof(int) * pad4(d.E);
  o.chunk = at; at += sizeof(int) * pad4((size_t)(d.E + 31) / 32 + 1);
  o.winl = at;  at += sizeof(int) * pad4((size_t)d.G * d.N + 1);
  o.total = at;
  return o;
}

__device__ __forceinline__ void place_body(const SolveParams& p, unsigned char* smem, int dm, int b) {
  const Dims d = p.d;
  const int M = d.M, G = d.G, E = d.E, GN = d.G * d.N, slots = G * p.stage1_slots;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const unsigned full = 0xffffffffu;
  const PlaceLayout lay = place_layout(d);
  unsigned long long* cand = reinterpret_cast<unsigned long long*>(smem + lay.cand);
  int* Dd = reinterpret_cast<int*>(smem + lay.D);
  int* mdom = reinterpret_cast<int*>(smem + lay.mdom);       // 1: main instance in this domain
  int* chunk = reinterpret_cast<int*>(smem + lay.chunk);     // candidates per 32 experts
  int* winl = reinterpret_cast<int*>(smem + lay.winl);
  const int nchunks = (E + 31) / 32;
  TL_MIN(p.ws, 2);
#pragma unroll 1
  for (int e = tid; e < E; e += nt) mdom[e] = __ldg(p.ws.main_rank + e) / G == dm ? 1 : 0;
  for (int i = tid; i <= GN; i += nt) winl[i] = -1;
  pdl_wait();
  TL_MIN(p.ws, 3);
  const unsigned serial = __ldcg(p.ws.epoch + 4);
  const size_t drow = ((size_t)b * M + dm) * E;
  if (p.acc) {   // one accumulator pair holds the sums, the other zeros
    const int32_t* dA = p.ws.acc_demand[0] + drow;
    const int32_t* dB = p.ws.acc_demand[1] + drow;
#pragma unroll 1
    for (int e = tid; e < E; e += nt) {
      const int v = __ldcg(dA + e) + __ldcg(dB + e);
      Dd[e] = v;
      p.ws.demand[drow + e] = v;   // kept for inspection
    }
  } else {       // the omega kernel left the demand in the workspace
#pragma unroll 1
    for (int e = tid; e < E; e += nt) Dd[e] = __ldcg(p.ws.demand + drow + e);
  }
  __syncthreads();
  TL_MAX(p.ws, 4);
  int n_win = 0;
  if (M > 1 && slots > 0) {
    // candidates per chunk of 32 experts, then their places in the compacted list
#pragma unroll 1
    for (int c = warp; c < nchunks; c += nwarps) {
      const int e = c * 32 + lane;
      const bool is = e < E && !mdom[e] && Dd[e] > p.cand_thr;
      const unsigned m = __ballot_sync(full, is);
      if (lane == 0) chunk[c] = __popc(m);
    }
    __syncthreads();
    int total = 0;
#pragma unroll 1
    for (int c = lane; c < nchunks; c += 32) total += chunk[c];
    total = __reduce_add_sync(full, total);
    if (total <= kP2RankCap) {
#pragma unroll 1
      for (int c = warp; c < nchunks; c += nwarps) {
        int before = 0;
#pragma unroll 1
        for (int u = lane; u < c; u += 32) before += chunk[u];
        before = __reduce_add_sync(full, before);
        const int e = c * 32 + lane;
        const bool is = e < E && !mdom[e] && Dd[e] > p.cand_thr;
        const unsigned m = __ballot_sync(full, is);
        if (is)
          cand[CK(p.ws.status, before + __popc(m & lanemask_lt()), kP2RankCap)] =
              ((unsigned long long)(unsigned)Dd[e] << 32) | (unsigned)~(unsigned)e;
      }
      __syncthreads();
      // a warp takes a candidate, its lanes the others: rank = keys above its own
      n_win = min(total, slots);
#pragma unroll 1
      for (int c = warp; c < total; c += nwarps) {
        const unsigned long long mine = cand[c];
        int rank = 0;
#pragma unroll 1
        for (int o0 = 0; o0 < total; o0 += 32)
          rank += __popc(__ballot_sync(full, o0 + lane < total && cand[o0 + lane] > mine));
        if (lane == 0 && rank < slots) winl[CK(p.ws.status, rank, GN)] = (int)~(unsigned)mine;
      }
    } else if (warp == 0) {
      // many candidates: pick the maximum slot by slot (non-candidates are zeroed first)
#pragma unroll 1
      for (int e = lane; e < E; e += 32)
        if (mdom[e] || Dd[e] <= p.cand_thr) Dd[e] = 0;
      __syncwarp();
#pragma unroll 1
      for (int i = 0; i < slots; ++i) {
        int bestD = 0, bestE = INT_MAX;
#pragma unroll 1
        for (int e = lane; e < E; e += 32) {
          const int v = Dd[e];
          if (v > bestD) { bestD = v; bestE = e; }   // ascending e: first hit is smallest
        }
        const int maxD = __reduce_max_sync(full, bestD);
        if (maxD <= 0) break;
        n_win = i + 1;
        const int e = __reduce_min_sync(full, bestD == maxD ? bestE : INT_MAX);
        if (lane == 0) { Dd[CK(p.ws.status, e, E)] = 0; winl[CK(p.ws.status, i, GN)] = e; }
        __syncwarp();
      }
      if (lane == 0) winl[GN] = n_win;   // hand the count to the publishing threads
    }
    __syncthreads();
    if (total > kP2RankCap) n_win = winl[GN];
  }
  unsigned long long* rec = p.ws.place_rec + ((size_t)b * M + dm) * (GN + 1);
  for (int i = tid; i <= GN; i += nt) {
    const unsigned v = i == 0 ? (unsigned)n_win : (unsigned)winl[i - 1];
    __stcg(rec + i, ((unsigned long long)serial << 32) | v);
  }
  TL_MAX(p.ws, 5);
}

// Readers of the placement records of plan b: poll until every word carries this call's serial
// number (bounded), then win[dd * GN + i], nwin[dd] and the winners' bits in the hosting masks
// (which hold the main-domain bits already).  False if the records did not arrive.
// slot_dd[i] = domain of winner entry i (a table, set up before the wait: no divisions here).
__device__ __forceinline__ bool fetch_placement(const Workspace& ws, int ws_experts, int b,
                                                unsigned serial, int M, int GN, int* win,
                                                int* nwin, const int* slot_dd,
                                                unsigned* hm_lo, unsigned* hm_hi, int tid, int nt) {
  const unsigned long long* rec = ws.place_rec + (size_t)b * M * (GN + 1);
  bool all = false;
#pragma unroll 1
  for (unsigned it = 0; it < kFlagWaitLimit && !all; ++it) {
    bool ok = true;
#pragma unroll 1
    for (int i = tid; i < M * GN; i += nt) {   // winner i of domain dd is word dd + 1 + i
      const unsigned long long w = __ldcg(rec + slot_dd[i] + 1 + i);
      ok = ok && (unsigned)(w >> 32) == serial;
      win[i] = (int)(unsigned)w;
    }
#pragma unroll 1
    for (int dd = tid; dd < M; dd += nt) {     // the count of domain dd is word dd * (GN + 1)
      const unsigned long long w = __ldcg(rec + (size_t)dd * (GN + 1));
      ok = ok && (unsigned)(w >> 32) == serial;
      nwin[dd] = (int)(unsigned)w;
    }
    all = __syncthreads_and(ok);
  }
  if (!all) {
    if (tid == 0) atomicOr(ws.status, TOPOEP_FLAG_INTERNAL);
    return false;
  }
#pragma unroll 1
  for (int i = tid; i < M * GN; i += nt) {
    const int dd = CK(ws.status, slot_dd[i], M), k = i - dd * GN;
    const int e = win[i] < 0 ? -1 : CK(ws.status, win[i], ws_experts);
    if (k < nwin[dd] && e >= 0) {
      if (dd < 32) atomicOr(&hm_lo[e], 1u << dd); else atomicOr(&hm_hi[e], 1u << (dd - 32));
    }
  }
  __syncthreads();
  return true;
}

// Can the refinement act at all?  Only a target with a free slot can take a move.
__device__ __forceinline__ bool plan_is_closed_form(const int* nwin, int M, int GN, int N,
                                                    int stage1_slots, int lpt) {
  bool closed = lpt == 0;
  if (N > 0) {
    if (M == 1 || stage1_slots != N) closed = false;
#pragma unroll 1
    for (int dd = 0; dd < M; ++dd) closed = closed && nwin[dd] == GN;
  }
  return closed;
}

// q(s, instance of e in domain dd) after inter-node placement (paper, "Inter-node placement",
// routing construction): a source keeps everything in its own domain when an instance is there;
// otherwise omega(s,e) = w is split over all n instances (ascending hosting domain), remainder to
// `rem` instances starting at (s+e) mod n.
__device__ __forceinline__ int closed_q(int w, unsigned long long hm, int dd, int ds, int s, int e) {
  const int n = __popcll(hm);
  if (ds == dd || n == 1) return w;   // own domain, or the only instance anywhere
  if ((hm >> ds) & 1ull) return 0;    // the source's own domain hosts e: nothing leaves it
  const int bs = w / n, rem = w - bs * n;
  int sh = __popcll(hm & ((1ull << dd) - 1ull)) - (s + e) % n;
  if (sh < 0) sh += n;
  return bs + (sh < rem ? 1 : 0);
}

// Instance of the replica of e that inter-node placement put into domain dd.  slot_p[dd * GN + i]
// is the instance of the i-th winner's slot (rank i mod G, slot i / G of the domain): a table,
// because integer division costs dozens of instructions on the critical path.
__device__ __forceinline__ int replica_instance(const int* win, const int* nwin, const int* slot_p,
                                                int dd, int e, int GN) {
  const int* w = win + dd * GN;
  const int n = nwin[dd];
  int i = 0;
#pragma unroll 1
  while (i < n - 1 && w[i] != e) ++i;
  return slot_p[dd * GN + (i < 0 ? 0 : i)];
}

// ---- per-token blocks -------------------------------------------------------------------------
struct TailLayout {
  size_t cnt, base, work;      // the ranking tail's counters, bases and work list
  size_t route, hdr, seg, cum, inst, tbase, tpre;
  size_t rm, qrow, mr, ml, orow, hm_lo, hm_hi, win, nwin, nz, single, sidx, seg_e, crow,
      split_e, warp_tot, mdom, slot_p, slot_dd, chunk_ns, chunk_nl, tc;
  size_t total;
};

__host__ __device__ inline TailLayout tail_layout(const Dims& d, int tiles) {
  auto pad4 = [](size_t ints) { return (ints + 3) & ~(size_t)3; };
  const int rows = 4 * kP2Warps;
  const size_t RN = (size_t)d.R * d.N, GN = (size_t)d.G * d.N;
  TailLayout o;
  size_t at = 0;
  o.cnt = at;   at += sizeof(uint4) * (size_t)kSplitCap * rows;
  o.base = at;  at += sizeof(int) * (size_t)kSplitCap * rows;
  o.work = at;  at += (sizeof(unsigned short) * (size_t)kPlan2TileIds + 15) & ~(size_t)15;
  auto ints = [&](size_t n) { const size_t r = at; at += sizeof(int) * pad4(n); return r; };
  o.route = ints(d.E + 1);
  o.hdr = ints(4);
  o.seg = ints(d.E + 1);
  o.cum = ints(d.P);
  o.inst = ints(d.P);
  o.tbase = ints(kSplitCap);
  o.tpre = ints(d.E);
  o.rm = ints(RN + 1);
  o.qrow = ints(d.P);
  o.mr = ints(d.E);
  o.ml = ints(d.E);
  o.orow = ints(d.E);
  o.hm_lo = ints(d.E);
  o.hm_hi = ints(d.E);
  o.win = ints((size_t)d.M * GN + 1);
  o.nwin = ints(d.M);
  o.nz = ints(d.E);
  o.single = ints(d.E);
  o.sidx = ints(d.E + 1);
  o.seg_e = ints(d.E + 1);
  o.crow = ints(d.R);
  o.split_e = ints(d.E);
  o.warp_tot = ints(2 * kP2Warps);
  o.mdom = ints(d.E);
  o.slot_p = ints(RN + 1);
  o.slot_dd = ints(RN + 1);
  o.chunk_ns = ints(RN / 32 + 2);
  o.chunk_nl = ints(RN / 32 + 2);
  o.tc = at;   // per-tile counts of the row, 16 bits each: [tiles][E]
  at += (sizeof(unsigned short) * (size_t)tiles * d.E + 15) & ~(size_t)15;
  o.total = at;
  return o;
}

// Shared-memory tables of a per-token block.
struct TailSm {
  int *route, *hdr, *seg, *cum, *inst, *rm, *qrow, *mr, *ml, *nz, *single, *sidx, *seg_e, *crow,
      *split_e, *warp_tot;
};

// The refinement decides q (some replica slot was free after inter-node placement): wait for the
// solver blocks of this plan (bounded polls), read row s of q and the replica map, and build the
// routing table the way the route kernel does.
__device__ __forceinline__ void slow_route(const TailParams& p, const TailSm& t, int tile, int s, int b,
                                        unsigned serial) {
  const Dims& d = p.d;
  const int M = d.M, R = d.R, E = d.E, N = d.N, P = d.P, s_phys = d.s_phys, e_loc = d.e_loc;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const unsigned full = 0xffffffffu;
  const int RN = R * N;
  const size_t row = (size_t)b * R + s;
  int *route = t.route, *hdr = t.hdr, *seg = t.seg, *cum = t.cum, *inst = t.inst, *rm = t.rm,
      *qrow = t.qrow, *mr = t.mr, *ml = t.ml, *nz = t.nz, *single = t.single, *sidx = t.sidx,
      *seg_e = t.seg_e, *crow = t.crow, *split_e = t.split_e, *warp_tot = t.warp_tot;
  int n_split, n_list;
  // ---- the refinement decides q: wait for the solver blocks of this plan (bounded polls),
  // then row s of q and the replica map come from memory.  Warp 1 polls: warp 0 would share its
  // scheduler with the refinement warp of a solver block on the same SM.
  if (warp == 1) {
    const unsigned* flags = p.ws.done_flags + (size_t)b * M;
    bool done = false;
#pragma unroll 1
    for (unsigned it = 0; it < kFlagWaitLimit && !done; ++it) {
      bool mine = true;
#pragma unroll 1
      for (int dd = lane; dd < M; dd += 32) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flags + dd) : "memory");
        mine = mine && v == serial;
      }
      done = __all_sync(full, mine);
      // the waiting warp shares its scheduler with the solver block's refinement warp when the
      // two blocks sit on one SM: poll at intervals, not back to back
      if (!done) __nanosleep(500);
    }
    if (!done && lane == 0) atomicOr(p.ws.status, TOPOEP_FLAG_INTERNAL);
  }
  __syncthreads();
#pragma unroll 1
  for (int i = tid; i < RN; i += nt) rm[i] = __ldcg(p.ws.replica_map + (size_t)b * RN + i);
#pragma unroll 1
  for (int i = tid; i < P; i += nt) qrow[i] = __ldcg(p.ws.q + row * P + i);
  __syncthreads();
  // instances with a share, per expert; split experts and their lists
#pragma unroll 1
  for (int e = tid; e < E; e += nt) {
    nz[e] = qrow[ml[e]] > 0 ? 1 : 0;
    single[e] = ml[e];
  }
  __syncthreads();
#pragma unroll 1
  for (int i = tid; i < RN; i += nt) {
    const int e = rm[i];
    if (e >= 0 && qrow[(i / N) * s_phys + e_loc + i % N] > 0) atomicAdd(&nz[e], 1);
  }
  __syncthreads();
#pragma unroll 1
  for (int i = tid; i < RN; i += nt) {   // the one instance with a share, when it is a replica
    const int e = rm[i];
    const int pi = (i / N) * s_phys + e_loc + i % N;
    if (e >= 0 && nz[e] == 1 && qrow[pi] > 0) single[e] = pi;
  }
  tail_scan2(nz, E, sidx, seg_e, warp_tot, tid, nt);
  n_split = sidx[E];
  n_list = seg_e[E];
#pragma unroll 1
  for (int e = tid; e < E; e += nt) {
    const bool split = nz[e] >= 2;
    route[e] = split ? -2 - sidx[e] : single[e];
    if (split) { seg[sidx[e]] = seg_e[e]; split_e[sidx[e]] = e; }
  }
  if (tid == 0) {
    hdr[0] = n_split; hdr[1] = n_list; hdr[2] = 0; hdr[3] = 0;
    seg[n_split] = n_list;
  }
  if (tile == 0) {   // dispatch counts of row s, for the send offsets below
#pragma unroll 1
    for (int r = tid; r < R; r += nt) {
      int sum = 0;
#pragma unroll 1
      for (int l = 0; l < s_phys; ++l) sum += qrow[r * s_phys + l];
      crow[r] = sum;
    }
  }
  __syncthreads();
  // Split lists, one warp per split expert: the instances with a share in ascending rank order
  // (the replica slots are in rank order; the main instance goes in front of the first slot on
  // a higher rank) with cumulative quotas.
#pragma unroll 1
  for (int i = warp; i < n_split; i += nwarps) {
    const int e = split_e[i];
    const int lb = seg_e[e], qm = qrow[ml[e]], rmain = mr[e];
    int carry_pos = 0, carry_cum = 0, main_pos = 0, main_below = 0;
#pragma unroll 1
    for (int i0 = 0; i0 < RN; i0 += 32) {
      const int slot = i0 + lane;
      int v = 0, r = 0, pi = 0;
      if (slot < RN && rm[slot] == e) {
        r = slot / N;
        pi = r * s_phys + e_loc + (slot - r * N);
        v = max(qrow[pi], 0);
      }
      const unsigned m = __ballot_sync(full, v > 0);
      if (m == 0) continue;
      int tot;
      const int ex = warp_exclusive_scan(v, lane, &tot);
      const bool below_main = v > 0 && r < rmain;
      main_pos += __popc(__ballot_sync(full, below_main));
      main_below += __reduce_add_sync(full, below_main ? v : 0);
      if (v > 0) {
        const bool after_main = qm > 0 && rmain < r;
        const int pos = carry_pos + __popc(m & lanemask_lt()) + (after_main ? 1 : 0);
        cum[lb + pos] = carry_cum + ex + v + (after_main ? qm : 0);
        inst[lb + pos] = pi;
      }
      carry_pos += __popc(m);
      carry_cum += tot;
    }
    if (lane == 0 && qm > 0) {
      cum[lb + main_pos] = main_below + qm;
      inst[lb + main_pos] = ml[e];
    }
  }
  __syncthreads();
}

// ROUTE_ONLY: a route block of the four-kernel chain -- one per (plan, source): it builds the
// same routing table, for every tile of the row, and writes it in the form reroute_kernel reads
// (the role of route_kernel); `tile` is the row's last tile then.
template <bool VEC, bool ROUTE_ONLY>
__device__ __forceinline__ void tail_body(const TailParams& p, unsigned char* smem, int tile, int s,
                                          int b) {
  const Dims d = p.d;
  const int M = d.M, G = d.G, R = d.R, E = d.E, N = d.N, P = d.P, s_phys = d.s_phys, e_loc = d.e_loc;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const int rows = 4 * nwarps;   // 128-id rows of the tile, in flat order
  const unsigned full = 0xffffffffu;
  const TailLayout lay = tail_layout(d, p.tiles);
  uint4* cnt4 = reinterpret_cast<uint4*>(smem + lay.cnt);
  unsigned* cntw = reinterpret_cast<unsigned*>(smem + lay.cnt);
  int* base = reinterpret_cast<int*>(smem + lay.base);
  unsigned short* work = reinterpret_cast<unsigned short*>(smem + lay.work);
  int* route = reinterpret_cast<int*>(smem + lay.route);
  int* hdr = reinterpret_cast<int*>(smem + lay.hdr);
  int* seg = reinterpret_cast<int*>(smem + lay.seg);         // [n_split+1] list start of split i
  int* cum = reinterpret_cast<int*>(smem + lay.cum);
  int* inst = reinterpret_cast<int*>(smem + lay.inst);
  int* tbase = reinterpret_cast<int*>(smem + lay.tbase);
  int* tpre = reinterpret_cast<int*>(smem + lay.tpre);       // [n_split] prefix over earlier tiles
  int* rm = reinterpret_cast<int*>(smem + lay.rm);           // [R*N] expert in replica slot
  int* qrow = reinterpret_cast<int*>(smem + lay.qrow);       // [P]   q(s, instance)
  int* mr = reinterpret_cast<int*>(smem + lay.mr);           // [E]   main rank
  int* ml = reinterpret_cast<int*>(smem + lay.ml);           // [E]   main instance id
  int* orow = reinterpret_cast<int*>(smem + lay.orow);       // [E]   omega[s][.]
  unsigned* hm_lo = reinterpret_cast<unsigned*>(smem + lay.hm_lo);
  unsigned* hm_hi = reinterpret_cast<unsigned*>(smem + lay.hm_hi);
  int* win = reinterpret_cast<int*>(smem + lay.win);         // [M][G*N] stage-1 winners in order
  int* nwin = reinterpret_cast<int*>(smem + lay.nwin);       // [M]
  int* nz = reinterpret_cast<int*>(smem + lay.nz);           // [E]   instances with q > 0
  int* single = reinterpret_cast<int*>(smem + lay.single);   // [E]
  int* sidx = reinterpret_cast<int*>(smem + lay.sidx);       // [E+1] split index of e
  int* seg_e = reinterpret_cast<int*>(smem + lay.seg_e);     // [E+1] list start of e (split only)
  int* crow = reinterpret_cast<int*>(smem + lay.crow);       // [R]   counts[s][.]
  int* split_e = reinterpret_cast<int*>(smem + lay.split_e); // [n_split] expert of split index i
  int* warp_tot = reinterpret_cast<int*>(smem + lay.warp_tot);
  int* mdom = reinterpret_cast<int*>(smem + lay.mdom);       // [E]   main domain
  int* slot_p = reinterpret_cast<int*>(smem + lay.slot_p);   // [M*GN] instance of a winner's slot
  int* slot_dd = reinterpret_cast<int*>(smem + lay.slot_dd); // [M*GN] its domain
  int* chunk_ns = reinterpret_cast<int*>(smem + lay.chunk_ns);   // split experts per 32 winners
  int* chunk_nl = reinterpret_cast<int*>(smem + lay.chunk_nl);   // list entries per 32 winners
  unsigned short* tc = reinterpret_cast<unsigned short*>(smem + lay.tc);   // [tiles][E]

  const TailSm t = {route, hdr, seg, cum, inst, rm, qrow, mr, ml, nz, single, sidx, seg_e, crow,
                    split_e, warp_tot};
  const size_t row = (size_t)b * R + s;
  const int begin = tile * p.tile_ids;
  const int count = min(p.tile_ids, p.n_ids - begin);
  const int32_t* ids = p.ids + row * (size_t)p.n_ids + begin;
  int32_t* out = p.out_token_replica + row * (size_t)p.n_ids + begin;
  const int RN = R * N, GN = G * N, ds = s / G;
  TL_MIN(p.ws, 6);

  // ---- before the histogram kernel is known to be complete: the ids (nobody's output) and the
  // handle's static tables
  int4 x[kIdsPerThread / 4];
  if (!ROUTE_ONLY) {
#pragma unroll
    for (int j = 0; j < kIdsPerThread / 4; ++j) x[j] = load_ids4(ids, j * nt + tid, count, VEC);
  }
#pragma unroll 1
  for (int e = tid; e < E; e += nt) {
    const int md = __ldg(p.ws.main_dom + e), mi = __ldg(p.ws.main_inst + e);
    mr[e] = __ldg(p.ws.main_rank + e);
    ml[e] = mi;
    mdom[e] = md;           // the expert's main domain hosts it from the start
    hm_lo[e] = md < 32 ? 1u << md : 0u;
    hm_hi[e] = md < 32 ? 0u : 1u << (md - 32);
    route[e] = mi;          // most experts have one instance with a share: their main instance
  }
  // tables of the winner slots: entry dd * GN + i sits on rank i mod G of domain dd, slot i / G
#pragma unroll 1
  for (int idx = tid; idx < M * GN; idx += nt) {
    slot_dd[idx] = __ldg(p.ws.slot_dd + idx);
    slot_p[idx] = __ldg(p.ws.slot_p + idx);
  }
  __syncthreads();
  if (tid == 0) {
    route[E] = -1;          // every id outside [0,E) is clamped onto this entry
    hdr[0] = 0; hdr[1] = 0; hdr[2] = 0; hdr[3] = 0;
    seg[0] = 0;
  }
  static_assert(kSplitCap % 8 == 0, "counter words per thread");
#pragma unroll
  for (int u = 0; u < kSplitCap / 8; ++u) cnt4[u * nt + tid] = make_uint4(0u, 0u, 0u, 0u);
  pdl_wait();
  TL_MIN(p.ws, 7);
  // ---- one round of loads of what the histogram kernel wrote (read past L1): the row's tile
  // counts and row s of the routing matrix -- one accumulator pair holds the sums, the other
  // zeros, so the two are added -- and the first poll of the placement records
  const unsigned serial = __ldcg(p.ws.epoch + 4);   // of this call: the histogram kernel advanced it
  {
    const unsigned short* src =
        reinterpret_cast<const unsigned short*>(p.ws.tile_cnt) + row * (size_t)p.max_tiles * E;
    const int n16 = (tile + 1) * E;   // the row's tiles up to and including this one
    if (E % 8 == 0) {
#pragma unroll 1
      for (int i = tid; i < n16 / 8; i += nt) cp_async16_cg(tc + 8 * i, src + 8 * i);
    } else {
#pragma unroll 1
      for (int i = tid; i < n16; i += nt) tc[i] = __ldcg(src + i);
    }
    if (p.acc) {
      const int32_t* oA = p.ws.acc_omega[0] + row * E;
      const int32_t* oB = p.ws.acc_omega[1] + row * E;
#pragma unroll 1
      for (int e = tid; e < E; e += nt) orow[e] = __ldcg(oA + e) + __ldcg(oB + e);
    } else {
#pragma unroll 1
      for (int e = tid; e < E; e += nt) orow[e] = __ldcg(p.ws.omega + row * E + e);
    }
  }
  const bool have_placement =
      fetch_placement(p.ws, E, b, serial, M, GN, win, nwin, slot_dd, hm_lo, hm_hi, tid, nt);
  cp_async_wait_all();
  __syncthreads();
  if (!have_placement) return;   // flagged; nothing sensible can be written
  TL_MAX(p.ws, 8);
  int n_split, n_list;

  const bool closed = plan_is_closed_form(nwin, M, GN, N, p.stage1_slots, p.stage1_lpt);
  if (closed) {
    // ---- the routing table of source s straight from omega[s][.] and the placement.  Every
    // expert that won no replica keeps the entry set up front (its main instance).  Warp 0 walks
    // the winners once: a replica in the source's own domain takes everything; an expert that the
    // source's domain does not host is shared out over its instances, and the entry of its first
    // replica domain stands for it.  Then every warp takes such an entry, a lane per instance.
    int* ent_k = rm;      // [M*GN] list start of the entry's expert (split), or -1: nothing to do
    int* ent_si = qrow;   // [M*GN] its split index, or -1: a single unit, one instance gets it
    // (32 winners per warp step; with more than 32 winners a first pass counts the split experts
    // and list entries of every step, so that all warps can take steps in the second pass)
    const int chunks = (M * GN + 31) >> 5;
#pragma unroll 1
    for (int pass = chunks > 1 ? 0 : 1; pass < 2; ++pass) {
#pragma unroll 1
      for (int c = warp; c < chunks; c += nwarps) {
        const int idx = c * 32 + lane;
        const bool valid = idx < M * GN;
        const int dd = valid ? slot_dd[idx] : 0;
        const int e = valid ? CK(p.ws.status, win[idx], E) : 0;
        const unsigned long long hm = ((unsigned long long)hm_hi[e] << 32) | hm_lo[e];
        const int md = mdom[e], n = __popcll(hm), w = orow[e];
        // first replica domain of e = lowest hosting domain that is not its main's
        const bool first = valid && !((hm >> ds) & 1ull) &&
                           __ffsll((long long)(hm & ~(1ull << md))) - 1 == dd;
        const int nzv = first ? min(w, n) : 0;   // instances with a share: all n once w >= n
        const bool split = nzv >= 2;
        const unsigned sm = __ballot_sync(full, split);
        int ltot;
        const int lpre = warp_exclusive_scan(split ? nzv : 0, lane, &ltot);
        if (pass == 0) {
          if (lane == 0) { chunk_ns[c] = __popc(sm); chunk_nl[c] = ltot; }
          continue;
        }
        int ns = 0, nl = 0;   // split experts and list entries of the earlier steps
        if (chunks > 1) {
#pragma unroll 1
          for (int u = lane; u < c; u += 32) { ns += chunk_ns[u]; nl += chunk_nl[u]; }
          ns = __reduce_add_sync(full, ns);
          nl = __reduce_add_sync(full, nl);
        }
        if (valid) {
          if (dd == ds) route[e] = slot_p[idx];
          const int si = ns + __popc(sm & lanemask_lt());
          ent_k[idx] = nzv >= 1 ? nl + lpre : -1;
          ent_si[idx] = split ? si : -1;
          if (split) {
            route[e] = -2 - si;
            seg[CK(p.ws.status, si, E)] = nl + lpre;
            split_e[CK(p.ws.status, si, E)] = e;
          }
        }
        if (c == chunks - 1 && lane == 0) {
          hdr[0] = ns + __popc(sm);
          hdr[1] = nl + ltot;
          seg[CK(p.ws.status, ns + __popc(sm), E + 1)] = nl + ltot;
        }
      }
      __syncthreads();
    }
    n_split = hdr[0];
    n_list = hdr[1];
#pragma unroll 1
    for (int idx = warp; idx < M * GN; idx += nwarps) {
      const int k0 = ent_k[idx];
      if (k0 < 0) continue;
      const int e = CK(p.ws.status, win[idx], E), si = ent_si[idx];
      const unsigned long long hm = ((unsigned long long)hm_hi[e] << 32) | hm_lo[e];
      const int md = mdom[e], n = __popcll(hm), w = orow[e];
      const int bs = w / n, rem = w - bs * n, start = (s + e) % n;
      int carry_pos = 0, carry_cum = 0;
#pragma unroll 1
      for (int t0 = 0; t0 < n; t0 += 32) {   // lane t: the t-th hosting domain, ascending
        const int t = t0 + lane;
        int v = 0, pi = 0;
        if (t < n) {
          unsigned long long m = hm;
#pragma unroll 1
          for (int u = 0; u < t; ++u) m &= m - 1;
          const int dx = __ffsll((long long)m) - 1;
          int sh = t - start;
          if (sh < 0) sh += n;
          v = bs + (sh < rem ? 1 : 0);
          if (v > 0) pi = dx == md ? ml[e] : replica_instance(win, nwin, slot_p, dx, e, GN);
        }
        const unsigned m2 = __ballot_sync(full, v > 0);
        int tot;
        const int ex = warp_exclusive_scan(v, lane, &tot);
        if (v > 0) {
          if (si >= 0) {
            const int pos = CK(p.ws.status, k0 + carry_pos + __popc(m2 & lanemask_lt()), P);
            cum[pos] = carry_cum + ex + v;
            inst[pos] = pi;
          } else {
            route[e] = pi;   // one unit: it goes to the instance at index (s+e) mod n
          }
        }
        carry_pos += __popc(m2);
        carry_cum += tot;
      }
    }
    __syncthreads();
  } else {
    slow_route(p, t, ROUTE_ONLY ? 0 : tile, s, b, serial);
    n_split = hdr[0];
    n_list = hdr[1];
  }
  TL_MAX(p.ws, 9);
  if (ROUTE_ONLY) {
    // ---- write the tables in the layout reroute_kernel reads: route[e]; the split record (header,
    // list starts, cumulative quotas, instances); per tile and split expert the prefix over the
    // earlier tiles, and for the first kSplitCap split experts also the resolved instance
    const SplitRec rl = split_rec_layout(E, P, p.max_tiles);
    int32_t* rec = p.ws.split_rec + row * (size_t)rl.ints;
    int32_t* g_route = p.ws.route + row * E;
#pragma unroll 1
    for (int e = tid; e < E; e += nt) g_route[e] = route[e];
#pragma unroll 1
    for (int i = tid; i <= n_split; i += nt) rec[rl.seg + i] = seg[i];
#pragma unroll 1
    for (int k = tid; k < n_list; k += nt) {
      rec[rl.cum + k] = cum[k];
      rec[rl.inst + k] = inst[k];
    }
    if (tid == 0) { rec[0] = n_split; rec[1] = n_list; rec[2] = 0; rec[3] = 0; }
    const size_t trow = row * (size_t)p.max_tiles * E;
    const int tiles = p.tiles;
#pragma unroll 1
    for (int i = warp; i < n_split; i += nwarps) {   // a warp per split expert, a lane per tile
      const int e = CK(p.ws.status, split_e[i], E);
      int carry = 0;
#pragma unroll 1
      for (int t0 = 0; t0 < tiles; t0 += 32) {
        const int tl = t0 + lane;
        const int tv = tl < tiles ? tc[(size_t)tl * E + e] : 0;
        int tot;
        const int ex = carry + warp_exclusive_scan(tv, lane, &tot);
        carry += tot;
        if (tl < tiles) {
          p.ws.tile_pref[trow + (size_t)tl * E + i] = ex;
          if (i < kSplitCap) {
            int lo = 0, res = -1;
#pragma unroll 1
            for (int k = seg[i]; k < seg[i + 1]; ++k) {
              const int hi = cum[CK(p.ws.status, k, P)];
              if (ex >= lo && ex + tv <= hi) { res = inst[CK(p.ws.status, k, P)]; break; }
              lo = hi;
            }
            int32_t* t3 = rec + rl.tp + tl * 3 * kSplitCap + i;
            t3[0] = ex;
            t3[kSplitCap] = res;
            t3[2 * kSplitCap] = e;
          }
        }
      }
    }
    if (!closed) {
      // send offsets of source s (the rank block of s writes them when the plan is closed-form)
      if (warp == 0) {
        int32_t* send = p.out_offsets + (((size_t)b * 2 + 0) * R + s) * (R + 1);
        const int ch = (R + 31) / 32;
        const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
        int sum = 0;
#pragma unroll 1
        for (int r = i0; r < i1; ++r) sum += crow[r];
        int total;
        int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
        for (int r = i0; r < i1; ++r) { send[r] = pre; pre += crow[r]; }
        if (lane == 0) send[R] = total;
      }
    }
    return;
  }
  // Cross-tile base of every split expert's stable rank, and the resolved tiles: when the ids of
  // the expert in this tile occupy ranks [ex, ex + tv) inside ONE instance's quota interval, they
  // all go to that instance and the tile ranks nothing for it.
#pragma unroll 1
  for (int i = tid; i < n_split; i += nt) {
    const int e = CK(p.ws.status, split_e[i], E);
    int ex = 0;
#pragma unroll 1
    for (int t = 0; t < tile; ++t) ex += tc[(size_t)t * E + e];
    const int tv = tc[(size_t)tile * E + e];
    int lo = 0, res = -1;
#pragma unroll 1
    for (int k = seg[i]; k < seg[i + 1]; ++k) {
      const int hi = cum[CK(p.ws.status, k, P)];
      if (ex >= lo && ex + tv <= hi) { res = inst[CK(p.ws.status, k, P)]; break; }
      lo = hi;
    }
    tpre[i] = ex;
    if (i < kSplitCap) tbase[i] = ex;
    if (res >= 0) route[e] = res;
  }
  if ((ROUTE_ONLY || tile == 0) && !closed) {
    // (the rank block of s writes these when the plan is closed-form)
    // row s of the routing matrix, kept for inspection and the summaries
#pragma unroll 1
    for (int e = tid; e < E; e += nt) p.ws.omega[row * E + e] = orow[e];
    // send offsets of source s: exclusive scan over the destination ranks, total appended
    if (warp == 0) {
      int32_t* send = p.out_offsets + (((size_t)b * 2 + 0) * R + s) * (R + 1);
      const int ch = (R + 31) / 32;
      const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
      int sum = 0;
#pragma unroll 1
      for (int r = i0; r < i1; ++r) sum += crow[r];
      int total;
      int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
      for (int r = i0; r < i1; ++r) { send[r] = pre; pre += crow[r]; }
      if (lane == 0) send[R] = total;
    }
  }
  __syncthreads();

  TL_MAX(p.ws, 10);
  // ---- stream: look up and store; split ids are remembered, pushed and patched below
  const unsigned uE = (unsigned)E;
  unsigned split_mask = 0;
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) {
    const int vec = j * nt + tid;
    const int t0 = route[min((unsigned)x[j].x, uE)];
    const int t1 = route[min((unsigned)x[j].y, uE)];
    const int t2 = route[min((unsigned)x[j].z, uE)];
    const int t3 = route[min((unsigned)x[j].w, uE)];
    split_mask |= (((unsigned)(t0 + 1) >> 31) | ((unsigned)(t1 + 1) >> 31) << 1 |
                   ((unsigned)(t2 + 1) >> 31) << 2 | ((unsigned)(t3 + 1) >> 31) << 3) << (4 * j);
    const int4 r = make_int4(max(t0, -1), max(t1, -1), max(t2, -1), max(t3, -1));
    if (VEC) {
      if (4 * vec < count) __stcs(reinterpret_cast<int4*>(out) + vec, r);
    } else {
      if (4 * vec + 0 < count) out[4 * vec + 0] = r.x;
      if (4 * vec + 1 < count) out[4 * vec + 1] = r.y;
      if (4 * vec + 2 < count) out[4 * vec + 2] = r.z;
      if (4 * vec + 3 < count) out[4 * vec + 3] = r.w;
    }
  }
  while (split_mask) {
    const int k = __ffs(split_mask) - 1;
    split_mask &= split_mask - 1;
    work[CK(p.ws.status, atomicAdd(hdr + 2, 1), kPlan2TileIds)] =
        (unsigned short)(4 * ((k >> 2) * nt + tid) + (k & 3));
  }
  __syncthreads();   // also orders the stores above before the patches below
  const int n_work = hdr[2];
  TL_MAX(p.ws, 11);
  if (n_work > 0) {
    const SplitRec rl = split_rec_layout(E, P, p.max_tiles);
    const SplitCtx c = {cnt4, cntw, base, route, seg, cum, inst, tbase, work, nullptr, tpre, ids, out,
                        rl, rows, n_split, n_list, n_work, p.ws.status, true};
    rank_and_patch(c, tid, nt, warp, nwarps);
  }
  TL_MAX(p.ws, 12);
  TL_MIN(p.ws, 13);
}

// ---- rank blocks: the plan in closed form, rank r's share ---------------------------------------
struct RankLayout {
  size_t hm_lo, hm_hi, win, nwin, mr, mie, orow, colv, qrow, crow, ccol, U, slot_dd, total;
};

__host__ __device__ inline RankLayout rank_layout(const Dims& d) {
  auto pad4 = [](size_t ints) { return (ints + 3) & ~(size_t)3; };
  RankLayout o;
  size_t at = 0;
  auto ints = [&](size_t n) { const size_t r = at; at += sizeof(int) * pad4(n); return r; };
  o.hm_lo = ints(d.E);
  o.hm_hi = ints(d.E);
  o.win = ints((size_t)d.M * d.G * d.N + 1);
  o.nwin = ints(d.M);
  o.mr = ints(d.E);
  o.mie = ints((size_t)d.R * (d.e_loc > 0 ? d.e_loc : 1));
  o.orow = ints(d.E);
  o.colv = ints((size_t)d.s_phys * d.R);
  o.qrow = ints(d.P);
  o.crow = ints(d.R);
  o.ccol = ints(d.R);
  o.U = ints(d.s_phys);
  o.slot_dd = ints((size_t)d.R * d.N + 1);
  o.total = at;
  return o;
}

__device__ __forceinline__ void rank_body(const SolveParams& p, unsigned char* smem, int r, int b) {
  const Dims d = p.d;
  const int M = d.M, G = d.G, R = d.R, E = d.E, N = d.N, P = d.P, s_phys = d.s_phys, e_loc = d.e_loc;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const RankLayout lay = rank_layout(d);
  unsigned* hm_lo = reinterpret_cast<unsigned*>(smem + lay.hm_lo);
  unsigned* hm_hi = reinterpret_cast<unsigned*>(smem + lay.hm_hi);
  int* win = reinterpret_cast<int*>(smem + lay.win);
  int* nwin = reinterpret_cast<int*>(smem + lay.nwin);
  int* mr = reinterpret_cast<int*>(smem + lay.mr);
  int* mie = reinterpret_cast<int*>(smem + lay.mie);       // [R][e_loc] expert of a main instance
  int* orow = reinterpret_cast<int*>(smem + lay.orow);     // [E]   omega[r][.]  (r as a source)
  int* colv = reinterpret_cast<int*>(smem + lay.colv);     // [s_phys][R] omega[.][e] of my columns
  int* qrow = reinterpret_cast<int*>(smem + lay.qrow);     // [P]   q(r, instance) (r as a source)
  int* crow = reinterpret_cast<int*>(smem + lay.crow);     // [R]   counts[r][.]
  int* ccol = reinterpret_cast<int*>(smem + lay.ccol);     // [R]   counts[.][r]
  int* U = reinterpret_cast<int*>(smem + lay.U);           // [s_phys] loads of my instances
  int* slot_dd = reinterpret_cast<int*>(smem + lay.slot_dd);
  const int GN = G * N, dm = r / G, g = r - dm * G;
  const size_t row = (size_t)b * R + r;

  // static tables first: they name the experts of this rank's main columns
#pragma unroll 1
  for (int e = tid; e < E; e += nt) {
    const int m = __ldg(p.ws.main_rank + e);
    mr[e] = m;
    const int md = m / G;
    hm_lo[e] = md < 32 ? 1u << md : 0u;
    hm_hi[e] = md < 32 ? 0u : 1u << (md - 32);
  }
#pragma unroll 1
  for (int i = tid; i < R * e_loc; i += nt) mie[i] = __ldg(p.ws.main_inst_expert + i);
#pragma unroll 1
  for (int i = tid; i < R; i += nt) ccol[i] = 0;
#pragma unroll 1
  for (int i = tid; i < M * GN; i += nt) slot_dd[i] = i / GN;
  if (tid < s_phys) U[tid] = 0;
  __syncthreads();
  pdl_wait();
  const unsigned serial = __ldcg(p.ws.epoch + 4);
  // the routing matrix of plan b: the sum of the two accumulator pairs (one holds the sums, the
  // other zeros), or the matrix the omega kernel left in the workspace
  const int32_t* oA = (p.acc ? p.ws.acc_omega[0] : p.ws.omega) + (size_t)b * R * E;
  const int32_t* oB = p.ws.acc_omega[1] + (size_t)b * R * E;
  const bool two = p.acc != 0;
  auto om = [&](size_t at) { return two ? __ldcg(oA + at) + __ldcg(oB + at) : __ldcg(oA + at); };
  {
#pragma unroll 1
    for (int e = tid; e < E; e += nt) orow[e] = om((size_t)r * E + e);
    // my main columns: omega[s][e] for every source s
#pragma unroll 1
    for (int i = tid; i < e_loc * R; i += nt) {
      const int l = i / R, s = i - l * R, e = mie[r * e_loc + l];
      colv[i] = e < 0 ? 0 : om((size_t)s * E + e);
    }
  }
  if (!fetch_placement(p.ws, E, b, serial, M, GN, win, nwin, slot_dd, hm_lo, hm_hi, tid, nt)) return;
  TL_MAX(p.ws, 14);
  if (!plan_is_closed_form(nwin, M, GN, N, p.stage1_slots, p.stage1_lpt)) return;   // solver's job

  // my replica columns (every slot is taken): a second, short round of loads
#pragma unroll 1
  for (int i = tid; i < N * R; i += nt) {
    const int j = i / R, s = i - j * R, e = CK(p.ws.status, win[dm * GN + j * G + g], E);
    colv[(e_loc + j) * R + s] = om((size_t)s * E + e);
  }
  // meanwhile: row r of q (r as a source) and of the dispatch counts
#pragma unroll 1
  for (int pi = tid; pi < P; pi += nt) {
    const int rr = pi / s_phys, l = pi - rr * s_phys, dd = rr / G;
    const int e0 = l < e_loc ? mie[rr * e_loc + l] : win[dd * GN + (l - e_loc) * G + (rr - dd * G)];
    const int e = e0 < 0 ? -1 : CK(p.ws.status, e0, E);
    int v = 0;
    if (e >= 0) v = closed_q(orow[e], ((unsigned long long)hm_hi[e] << 32) | hm_lo[e], dd, dm, r, e);
    qrow[pi] = v;
    p.ws.q[row * P + pi] = v;
  }
  __syncthreads();
#pragma unroll 1
  for (int rr = tid; rr < R; rr += nt) {
    int sum = 0;
#pragma unroll 1
    for (int l = 0; l < s_phys; ++l) sum += qrow[rr * s_phys + l];
    crow[rr] = sum;
    p.ws.counts[row * R + rr] = sum;
    p.out_counts[row * R + rr] = sum;
  }
  // row r of the routing matrix, kept for inspection and the summaries
#pragma unroll 1
  for (int e = tid; e < E; e += nt) p.ws.omega[row * E + e] = orow[e];
  // my columns: q(s, my instance l) for every source s; instance loads U and counts[s][r]
#pragma unroll 1
  for (int i = tid; i < s_phys * R; i += nt) {
    const int l = i / R, s = i - l * R;
    const int e0 = l < e_loc ? mie[r * e_loc + l] : win[dm * GN + (l - e_loc) * G + g];
    if (e0 < 0) continue;
    const int e = CK(p.ws.status, e0, E);
    const int v = closed_q(colv[i], ((unsigned long long)hm_hi[e] << 32) | hm_lo[e], dm, s / G, s, e);
    if (v != 0) { atomicAdd(&U[l], v); atomicAdd(&ccol[s], v); }
  }
  __syncthreads();
  if (tid < s_phys) {
    const size_t at = (size_t)b * P + (size_t)r * s_phys + tid;
    p.ws.inst_counts[at] = U[tid];
    if (p.out_inst_counts) p.out_inst_counts[at] = U[tid];
  }
  if (tid < N) {
    const size_t at = ((size_t)b * R + r) * N + tid;
    const int e = win[dm * GN + tid * G + g];
    p.ws.replica_map[at] = e;
    if (p.out_replica_map) p.out_replica_map[at] = e;
  }
  if (tid == 0) {
    int load = 0;
#pragma unroll 1
    for (int l = 0; l < s_phys; ++l) load += U[l];
    p.ws.rank_load[row] = load;
    if (g == 0) p.ws.refine_iters[(size_t)b * M + dm] = 0;
  }
  // send offsets of source r: exclusive scan of its dispatch counts, total appended
  if (warp == 1 % (nt >> 5)) {
    int32_t* send = p.out_offsets + (((size_t)b * 2 + 0) * R + r) * (R + 1);
    const int ch = (R + 31) / 32;
    const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
    int sum = 0;
#pragma unroll 1
    for (int x = i0; x < i1; ++x) sum += crow[x];
    int total;
    int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
    for (int x = i0; x < i1; ++x) { send[x] = pre; pre += crow[x]; }
    if (lane == 0) send[R] = total;
  }
  // receive offsets of rank r: exclusive scan over the sources, total appended
  if (warp == 0) {
    int32_t* recv = p.out_offsets + (((size_t)b * 2 + 1) * R + r) * (R + 1);
    const int ch = (R + 31) / 32;
    const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
    int sum = 0;
#pragma unroll 1
    for (int s = i0; s < i1; ++s) sum += ccol[s];
    int total;
    int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
    for (int s = i0; s < i1; ++s) { recv[s] = pre; pre += ccol[s]; }
    if (lane == 0) recv[R] = total;
  }
  TL_MAX(p.ws, 15);
}

struct Plan2Params {
  SolveParams sp;
  TailParams tp;
  int n_solve;   // blocks [0, n_solve): placement, (plan i / M, domain i % M); the next n_solve
                 // blocks: solver, same numbering
  int n_rank;    // then the per-token blocks (two-kernel chain) or n_rank route blocks (four-kernel
                 // chain); the LAST n_rank blocks: rank blocks, (plan i / R, rank i % R)
};

template <bool LPT, bool VEC, bool ROUTE_ONLY>
__global__ void __launch_bounds__(kSolveThreads, 2) plan2_kernel(const Plan2Params p) {
  extern __shared__ __align__(16) unsigned char smem[];
  int i = blockIdx.x;
  if (i < p.n_solve) {
    place_body(p.sp, smem, i % p.sp.d.M, i / p.sp.d.M);
    return;
  }
  i -= p.n_solve;
  if (i < p.n_solve) {
    solve_body<LPT>(p.sp, smem, i % p.sp.d.M, i / p.sp.d.M);
    return;
  }
  i -= p.n_solve;
  // The blocks on the critical path come next (blocks start in index order, a few dozen per
  // microsecond when they are this large); the rank blocks, which nobody waits for, come last.
  const int n_front = (int)gridDim.x - 2 * p.n_solve - p.n_rank;
  if (i >= n_front) {
    i -= n_front;
    if (!LPT) rank_body(p.sp, smem, i % p.sp.d.R, i / p.sp.d.R);
    return;
  }
  const int tiles = p.tp.tiles, R = p.tp.d.R;
  if (ROUTE_ONLY) tail_body<VEC, true>(p.tp, smem, tiles - 1, i % R, i / R);
  else tail_body<VEC, false>(p.tp, smem, i % tiles, (i / tiles) % R, i / (tiles * R));
}

}  // namespace

size_t plan2_smem_bytes(const Dims& d, int tiles) {
  return std::max(std::max(tail_layout(d, tiles).total, rank_layout(d).total),
                  std::max(solve_smem_bytes(d), place_layout(d).total));
}

size_t plan2_route_smem_bytes(const Dims& d, int tiles) { return plan2_smem_bytes(d, tiles); }

long long plan2_blocks(const Dims& d, int tiles, int batch) {
  return (2ll * d.M + d.R + (long long)tiles * d.R) * batch;
}

cudaError_t launch_plan2(const SolveParams& sp, const TailParams& tp, int batch, bool route_only,
                         cudaStream_t stream) {
  Plan2Params p;
  p.sp = sp;
  p.tp = tp;
  p.n_solve = sp.d.M * batch;
  p.n_rank = sp.d.R * batch;
  const long long blocks = route_only ? (2ll * sp.d.M + 2ll * sp.d.R) * batch
                                      : plan2_blocks(sp.d, tp.tiles, batch);
  const dim3 grid((unsigned)blocks), block(kSolveThreads);
  const size_t smem = plan2_smem_bytes(tp.d, tp.tiles);
  const bool pdl = tp.pdl != 0;
  if (route_only) {   // no ids in these blocks: the VEC variants differ by nothing they run
    return sp.stage1_lpt ? launch_kernel(plan2_kernel<true, false, true>, grid, block, smem, stream, pdl, p)
                         : launch_kernel(plan2_kernel<false, false, true>, grid, block, smem, stream, pdl, p);
  }
  if (sp.stage1_lpt)
    return tp.vec_ok ? launch_kernel(plan2_kernel<true, true, false>, grid, block, smem, stream, pdl, p)
                     : launch_kernel(plan2_kernel<true, false, false>, grid, block, smem, stream, pdl, p);
  return tp.vec_ok ? launch_kernel(plan2_kernel<false, true, false>, grid, block, smem, stream, pdl, p)
                   : launch_kernel(plan2_kernel<false, false, false>, grid, block, smem, stream, pdl, p);
}

cudaError_t configure_plan2(size_t smem) {
  cudaError_t e;
  const int n = (int)smem;
  const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  if ((e = cudaFuncSetAttribute(plan2_kernel<true, true, false>, attr, n)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(plan2_kernel<true, false, false>, attr, n)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(plan2_kernel<false, true, false>, attr, n)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(plan2_kernel<false, false, false>, attr, n)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(plan2_kernel<true, false, true>, attr, n)) != cudaSuccess) return e;
  return cudaFuncSetAttribute(plan2_kernel<false, false, true>, attr, n);
}

}  // namespace topoep
