// Two-stage placement / routing solver and dispatch layout (paper, "Two-Stage GPU-Native
// Solver": inter-node placement with b_{d,e} = 2 D_{d,e} S_tok - ||W||, routing construction,
// loads U and L, intra-node refinement with delta = min(U, floor((L_b - L_t)/2)); constraints
// C1-C5; dispatch counts and offsets derived on the device).
//
// One CTA per (plan, NVLink domain).  The CTA owns the destination side of its domain: the
// columns q[.][p] of the instances p that live on its G ranks, for every source rank, held in
// shared memory together with the placement, U and L.  What it needs from the other domains
// -- which domains host each expert after inter-node placement -- it recomputes itself, one
// warp per domain, so no CTA ever waits for another.  Refinement is the serial part: one warp
// runs the loop, every selection is a warp reduction over a totally ordered key.
// What needs every domain's result (send offsets, per-source routing tables) is left to the
// route kernel that follows.
#include <limits.h>

#include "topoep_internal.cuh"

namespace topoep {

namespace {

struct SolveLayout {
  size_t hostmask, D, qd, col_expert, col_cr, U, L, used, cnt, hostcol, total;
};

__host__ __device__ inline SolveLayout solve_layout(const Dims& d) {
  SolveLayout o;
  size_t at = 0;
  o.hostmask = at;   at += sizeof(unsigned long long) * (size_t)d.E;
  o.D = at;          at += sizeof(int) * (size_t)d.M * d.E;
  o.qd = at;         at += sizeof(int) * (size_t)d.R * d.qstride;
  o.col_expert = at; at += sizeof(int) * (size_t)d.C;
  o.col_cr = at;     at += sizeof(int) * (size_t)d.C;
  o.U = at;          at += sizeof(int) * (size_t)d.C;
  o.L = at;          at += sizeof(int) * (size_t)d.G;
  o.used = at;       at += sizeof(int) * (size_t)d.G;
  o.cnt = at;        at += sizeof(int) * (size_t)d.R * d.G;
  o.hostcol = at;    at += sizeof(short) * (size_t)d.G * d.E;
  o.total = (at + 15) & ~(size_t)15;
  return o;
}

__global__ void __launch_bounds__(kSolveThreads) solve_kernel(const SolveParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const Dims d = p.d;
  const int M = d.M, G = d.G, R = d.R, E = d.E, N = d.N, C = d.C, QS = d.qstride;
  const int s_phys = d.s_phys, e_loc = d.e_loc;
  const int dm = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const unsigned full = 0xffffffffu;

  const SolveLayout lay = solve_layout(d);
  unsigned long long* hostmask = reinterpret_cast<unsigned long long*>(smem + lay.hostmask);
  int* D = reinterpret_cast<int*>(smem + lay.D);
  int* qd = reinterpret_cast<int*>(smem + lay.qd);
  int* col_expert = reinterpret_cast<int*>(smem + lay.col_expert);
  int* col_cr = reinterpret_cast<int*>(smem + lay.col_cr);
  int* U = reinterpret_cast<int*>(smem + lay.U);
  int* L = reinterpret_cast<int*>(smem + lay.L);
  int* used = reinterpret_cast<int*>(smem + lay.used);
  int* cnt = reinterpret_cast<int*>(smem + lay.cnt);
  short* hostcol = reinterpret_cast<short*>(smem + lay.hostcol);

  const int32_t* om = p.omega + (size_t)b * R * E;
  const int32_t* main_rank = p.ws.main_rank;

  // ---- tables of the own domain; candidate demand of every domain -------------------------
  for (int i = tid; i < G * E; i += nt) hostcol[i] = -1;
  for (int c = tid; c < C; c += nt) {
    const int g = c / s_phys, l = c - g * s_phys;
    col_expert[c] = l < e_loc ? p.ws.main_inst_expert[(size_t)(dm * G + g) * e_loc + l] : -1;
    col_cr[c] = p.cost_rank_intra;   // a main instance of this domain: parameters come from inside
    U[c] = 0;
  }
  if (tid < G) used[tid] = 0;
  for (int e = tid; e < E; e += nt) hostmask[e] = 1ull << (main_rank[e] / G);
  // D[dd][e] = sum over the G source ranks of domain dd, kept only where e is a stage-1 candidate
  // of dd (main outside dd and b > 0), else 0.  Loads are issued eight at a time.
  for (int idx0 = tid; idx0 < M * E; idx0 += 4 * nt) {
    int sum[4] = {0, 0, 0, 0};
    for (int g0 = 0; g0 < G; g0 += 8) {
      int v[4][8];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int idx = idx0 + a * nt;
        const int dd = idx / E, e = idx - dd * E;
        const int32_t* col = om + (size_t)dd * G * E + e;
#pragma unroll
        for (int u = 0; u < 8; ++u)
          v[a][u] = (idx < M * E && g0 + u < G) ? __ldg(col + (size_t)(g0 + u) * E) : 0;
      }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int u = 0; u < 8; ++u) sum[a] += v[a][u];
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int idx = idx0 + a * nt;
      if (idx >= M * E) break;
      const int dd = idx / E, e = idx - dd * E;
      const bool cand = dd != main_rank[e] / G &&
                        2 * (long long)sum[a] * p.token_bytes - p.expert_bytes > 0;
      D[idx] = cand ? sum[a] : 0;
    }
  }
  __syncthreads();
  for (int c = tid; c < C; c += nt) {
    const int e = col_expert[c];
    if (e >= 0) hostcol[(c / s_phys) * E + e] = (short)c;
  }

  // ---- inter-node placement, every domain, one warp each ------------------------------------
  // Candidates in descending (b, then ascending e) order == descending (D, ascending e) for a
  // uniform ||W|| and S_tok; the i-th goes to rank i mod G, slot i / G (fewest used slots first,
  // ties to the lower rank).
  if (M > 1 && N > 0) {
    for (int dd = warp; dd < M; dd += nwarps) {
      int* Dd = D + dd * E;
      for (int i = 0; i < G * N; ++i) {
        int bestD = 0;
        unsigned bestK = 0;   // ~e: larger means smaller e
        for (int e = lane; e < E; e += 32) {
          const int v = Dd[e];
          if (v > bestD) { bestD = v; bestK = ~(unsigned)e; }   // ascending e: first hit is smallest
        }
        const int maxD = __reduce_max_sync(full, bestD);
        if (maxD <= 0) break;
        const unsigned k = __reduce_max_sync(full, bestD == maxD ? bestK : 0u);
        const int e = (int)~k;
        if (lane == 0) {
          Dd[e] = 0;   // taken
          atomicOr(&hostmask[e], 1ull << dd);
          if (dd == dm) {
            const int g = i % G, j = i / G, c = g * s_phys + e_loc + j;
            col_expert[c] = e;
            col_cr[c] = p.cost_rank_inter;   // its main lies in another domain
            hostcol[g * E + e] = (short)c;
            used[g] = j + 1;
          }
        }
        __syncwarp();
      }
    }
  }
  __syncthreads();

  // ---- routing construction for the columns of this domain ----------------------------------
  // After stage 1 an expert has at most one instance per domain.  A source keeps everything in
  // its own domain when an instance is there; otherwise it splits over all instances (ascending
  // rank == ascending hosting domain), remainder to `rem` instances starting at (s+e) mod n.
  for (int idx0 = tid; idx0 < R * C; idx0 += 4 * nt) {
    int w[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {   // the four omega loads go out before any is used
      const int idx = idx0 + u * nt;
      w[u] = 0;
      if (idx < R * C) {
        const int s = idx / C, e = col_expert[idx - s * C];
        if (e >= 0) w[u] = __ldg(om + (size_t)s * E + e);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int idx = idx0 + u * nt;
      if (idx >= R * C) break;
      const int s = idx / C, c = idx - s * C;
      const int e = col_expert[c];
      int v = 0;
      if (e >= 0) {
        const int ds = s / G;
        if (ds == dm) {
          v = w[u];
        } else {
          const unsigned long long hm = hostmask[e];
          if (!((hm >> ds) & 1ull)) {
            const int n = __popcll(hm);
            const int i = __popcll(hm & ((1ull << dm) - 1ull));
            const int base = w[u] / n, rem = w[u] - base * n;
            int sh = i - (s + e) % n;
            if (sh < 0) sh += n;
            v = base + (sh < rem ? 1 : 0);
          }
        }
      }
      qd[s * QS + c] = v;
    }
  }
  __syncthreads();
  for (int c = tid; c < C; c += nt) {
    int sum = 0;
    for (int s = 0; s < R; ++s) sum += qd[s * QS + c];
    U[c] = sum;
  }
  __syncthreads();
  if (tid < G) {
    int sum = 0;
    for (int l = 0; l < s_phys; ++l) sum += U[tid * s_phys + l];
    L[tid] = sum;
  }
  __syncthreads();

  // ---- intra-node refinement: warp 0, one commit per iteration ------------------------------
  if (warp == 0) {
    int it = 0;
    const int chunk = (R + 31) / 32;
    for (;;) {
      const int Lg = lane < G ? L[lane] : -1;
      const int Lb = __reduce_max_sync(full, Lg);
      const int gb = __ffs(__ballot_sync(full, Lg == Lb)) - 1;   // busiest, lowest id on ties
      int bd = 0, bl = INT_MAX;
      unsigned bk = 0xffffffffu;
      for (int idx = lane; idx < s_phys * G; idx += 32) {
        const int l = idx / G, gt = idx - l * G;
        const int cb = gb * s_phys + l;
        const int e = col_expert[cb];
        if (gt == gb || e < 0) continue;
        const int u = U[cb];
        if (u <= 0) continue;
        const int hc = hostcol[gt * E + e];
        if (hc < 0 && used[gt] >= N) continue;              // neither hosts e nor has a free slot
        const int Lt = L[gt];
        const int delta = min(u, (Lb - Lt) >> 1);           // half-gap bound
        if (delta < p.min_delta) continue;
        const unsigned cr = hc >= 0 ? 0u : (unsigned)col_cr[cb];
        const unsigned key = (cr << 28) | ((unsigned)e << 5) | (unsigned)gt;
        if (delta > bd || (delta == bd && (Lt < bl || (Lt == bl && key < bk)))) {
          bd = delta; bl = Lt; bk = key;
        }
      }
      const int md = __reduce_max_sync(full, bd);
      if (md <= 0) break;
      const int ml = __reduce_min_sync(full, bd == md ? bl : INT_MAX);
      const unsigned mk = __reduce_min_sync(full, (bd == md && bl == ml) ? bk : 0xffffffffu);
      if (it >= p.max_iters) {
        if (lane == 0) atomicOr(p.ws.status, TOPOEP_FLAG_REFINE_CAP);
        break;
      }
      const int e = (int)((mk >> 5) & 0x7fffffu), gt = (int)(mk & 31u);
      const int cb = hostcol[gb * E + e];
      int ct = hostcol[gt * E + e];
      if (ct < 0) {   // create the replica in the target's next free slot
        ct = gt * s_phys + e_loc + used[gt];
        __syncwarp();
        if (lane == 0) {
          col_expert[ct] = e;
          col_cr[ct] = col_cr[cb];
          hostcol[gt * E + e] = (short)ct;
          used[gt] += 1;
        }
      }
      // Move md units of q from column cb to ct; sources in the order: the target rank itself,
      // then the others ascending, the busiest rank last.
      const int rb = dm * G + gb, rt = dm * G + gt;
      const int lo = min(rb, rt), hi = max(rb, rt);
      const int i0 = min(R, lane * chunk), i1 = min(R, i0 + chunk);
      int sum = 0;
      for (int i = i0; i < i1; ++i) {
        int s = i == 0 ? rt : (i == R - 1 ? rb : i - 1);
        if (i != 0 && i != R - 1) { if (s >= lo) ++s; if (s >= hi) ++s; }
        sum += qd[s * QS + cb];
      }
      int pre = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(full, pre, o);
        if (lane >= o) pre += t;
      }
      pre -= sum;
      for (int i = i0; i < i1; ++i) {
        int s = i == 0 ? rt : (i == R - 1 ? rb : i - 1);
        if (i != 0 && i != R - 1) { if (s >= lo) ++s; if (s >= hi) ++s; }
        const int v = qd[s * QS + cb];
        const int take = min(max(md - pre, 0), v);
        if (take > 0) {
          qd[s * QS + cb] = v - take;
          qd[s * QS + ct] += take;
        }
        pre += v;
      }
      if (lane == 0) {
        U[cb] -= md; U[ct] += md;
        L[gb] -= md; L[gt] += md;
      }
      __syncwarp();
      ++it;
    }
    if (lane == 0) p.ws.refine_iters[(size_t)b * M + dm] = it;
  }
  __syncthreads();

  // ---- results of this domain ----------------------------------------------------------------
  for (int idx = tid; idx < G * N; idx += nt) {
    const int g = idx / N, j = idx - g * N;
    const int e = col_expert[g * s_phys + e_loc + j];
    const size_t at = ((size_t)b * R + dm * G + g) * N + j;
    p.ws.replica_map[at] = e;
    if (p.out_replica_map) p.out_replica_map[at] = e;
  }
  for (int idx = tid; idx < R * C; idx += nt) {
    const int s = idx / C, c = idx - s * C;
    p.ws.q[((size_t)b * R + s) * d.P + (size_t)dm * C + c] = qd[s * QS + c];
  }
  for (int c = tid; c < C; c += nt) {
    const size_t at = (size_t)b * d.P + (size_t)dm * C + c;
    p.ws.inst_counts[at] = U[c];
    if (p.out_inst_counts) p.out_inst_counts[at] = U[c];
  }
  if (tid < G) p.ws.rank_load[(size_t)b * R + dm * G + tid] = L[tid];
  for (int idx = tid; idx < R * G; idx += nt) {
    const int s = idx / G, g = idx - s * G;
    int sum = 0;
    for (int l = 0; l < s_phys; ++l) sum += qd[s * QS + g * s_phys + l];
    cnt[idx] = sum;
    const size_t at = ((size_t)b * R + s) * R + dm * G + g;
    p.ws.counts[at] = sum;
    p.out_counts[at] = sum;
  }
  __syncthreads();
  if (tid < G) {   // receive offsets of rank r: exclusive scan over the sources
    int32_t* recv = p.out_offsets + (((size_t)b * 2 + 1) * R + dm * G + tid) * (R + 1);
    int run = 0;
    for (int s = 0; s < R; ++s) { recv[s] = run; run += cnt[s * G + tid]; }
    recv[R] = run;
  }

}

}  // namespace

size_t solve_smem_bytes(const Dims& d) { return solve_layout(d).total; }

cudaError_t launch_solve(const SolveParams& p, int batch, cudaStream_t stream) {
  const dim3 grid(p.d.M, batch);
  solve_kernel<<<grid, kSolveThreads, solve_smem_bytes(p.d), stream>>>(p);
  return cudaGetLastError();
}

cudaError_t configure_solve(size_t smem) {
  return cudaFuncSetAttribute(solve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace topoep
