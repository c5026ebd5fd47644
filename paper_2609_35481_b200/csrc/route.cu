// Per-source routing tables and send offsets (paper, "System Design": the token-routing
// decisions q drive dispatch; "derives receive counts on the GPU").
//
// One CTA per (plan, source rank s).  For every expert e it looks at the instances that got a
// nonzero share q(s,e,.) of the source's assignments:
//   one (or none) -> route[e] = that instance: every assignment of (s,e) goes there, no ranking;
//   two or more   -> e is a "split" expert of s: route[e] = -2-i, and list i holds the instances in
//                    ascending rank order with their cumulative quotas.
// On the benchmark workloads 2-6% of the assignments belong to split pairs (replicated experts
// seen from a domain that has no instance, or refined inside a domain), so the reroute kernel
// ranks only those.  For the split experts the CTA also turns the row's per-tile counts into
// exclusive prefixes over tiles.  Last, it scans row s of the dispatch counts into send offsets.
//
// The kernel is latency-bound (a few KB per CTA), so every input is fetched in one round of
// independent loads before the first barrier; only the tile counts of the split experts need a
// second round.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

struct RouteLayout { size_t rm, qrow, mr, ml, nz, single, sidx, seg, crow, split_e, warp_tot, total; };

__host__ __device__ inline RouteLayout route_layout(const Dims& d) {
  RouteLayout o;
  size_t at = 0;
  o.rm = at;       at += sizeof(int) * (size_t)(d.R * d.N + 1);
  o.qrow = at;     at += sizeof(int) * (size_t)d.P;
  o.mr = at;       at += sizeof(int) * (size_t)d.E;
  o.ml = at;       at += sizeof(int) * (size_t)d.E;
  o.nz = at;       at += sizeof(int) * (size_t)d.E;
  o.single = at;   at += sizeof(int) * (size_t)d.E;
  o.sidx = at;     at += sizeof(int) * (size_t)(d.E + 1);
  o.seg = at;      at += sizeof(int) * (size_t)(d.E + 1);
  o.crow = at;     at += sizeof(int) * (size_t)d.R;
  o.split_e = at;  at += sizeof(int) * (size_t)d.E;
  o.warp_tot = at; at += sizeof(int) * 2 * (kRouteThreads / 32);
  o.total = at;
  return o;
}

// Exclusive scan of (flag[e], flag[e] * nz[e]) with flag = nz >= 2 over e < n by the whole CTA;
// results in out_a / out_b (entry n = totals).  Each thread owns a contiguous chunk.
__device__ void block_scan2(const int* nz, int n, int* out_a, int* out_b, int* warp_tot, int tid,
                            int nt) {
  const int lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  const int chunk = (n + nt - 1) / nt;
  const int i0 = min(n, tid * chunk), i1 = min(n, i0 + chunk);
  int a = 0, b = 0;
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
  for (int w = 0; w < warp; ++w) { ba += warp_tot[w]; bb += warp_tot[nw + w]; }
  ea += ba;
  eb += bb;
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

__global__ void __launch_bounds__(kRouteThreads) route_kernel(const RouteParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const Dims d = p.d;
  const int R = d.R, E = d.E, N = d.N, P = d.P, s_phys = d.s_phys, e_loc = d.e_loc;
  const int s = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  if (p.pdl == 2) pdl_trigger();
  const RouteLayout lay = route_layout(d);
  int* rm = reinterpret_cast<int*>(smem + lay.rm);         // [R*N] expert in replica slot
  int* qrow = reinterpret_cast<int*>(smem + lay.qrow);     // [P]   q(s, instance)
  int* mr = reinterpret_cast<int*>(smem + lay.mr);         // [E]   main rank
  int* ml = reinterpret_cast<int*>(smem + lay.ml);         // [E]   main instance id
  int* nz = reinterpret_cast<int*>(smem + lay.nz);         // [E]   instances with q > 0
  int* single = reinterpret_cast<int*>(smem + lay.single); // [E]
  int* sidx = reinterpret_cast<int*>(smem + lay.sidx);     // [E+1] split index of e
  int* seg = reinterpret_cast<int*>(smem + lay.seg);       // [E+1] list start of e (split only)
  int* crow = reinterpret_cast<int*>(smem + lay.crow);     // [R]   counts[s][.]
  int* split_e = reinterpret_cast<int*>(smem + lay.split_e); // [E]   expert of split index i
  int* warp_tot = reinterpret_cast<int*>(smem + lay.warp_tot);

  const size_t row = (size_t)b * R + s;
  const int RN = R * N;
  // static tables before the solver is known to be done, its results after
  for (int e = tid; e < E; e += nt) {
    const int r = p.ws.main_rank[e];
    mr[e] = r;
    ml[e] = r * s_phys + p.ws.main_local[e];
  }
  pdl_wait();
  for (int i = tid; i < RN; i += nt) rm[i] = p.ws.replica_map[(size_t)b * RN + i];
  for (int i = tid; i < P; i += nt) qrow[i] = p.ws.q[row * P + i];
  for (int r = tid; r < R; r += nt) crow[r] = p.ws.counts[row * R + r];
  __syncthreads();

  for (int e = tid; e < E; e += nt) {
    nz[e] = qrow[ml[e]] > 0 ? 1 : 0;
    single[e] = ml[e];
  }
  __syncthreads();
  for (int i = tid; i < RN; i += nt) {
    const int e = rm[i];
    if (e >= 0 && qrow[(i / N) * s_phys + e_loc + i % N] > 0) atomicAdd(&nz[e], 1);
  }
  __syncthreads();
  for (int i = tid; i < RN; i += nt) {   // the one instance with a share, when it is a replica
    const int e = rm[i];
    const int pi = (i / N) * s_phys + e_loc + i % N;
    if (e >= 0 && nz[e] == 1 && qrow[pi] > 0) single[e] = pi;
  }
  block_scan2(nz, E, sidx, seg, warp_tot, tid, nt);
  const int n_split = sidx[E], n_list = seg[E];

  // second round of loads: tile counts of the split experts (prefix over tiles below)
  const SplitRec rl = split_rec_layout(E, P, p.max_tiles);
  int32_t* rec = p.ws.split_rec + row * (size_t)rl.ints;
  int32_t* route = p.ws.route + row * E;
  for (int e = tid; e < E; e += nt) {
    const bool split = nz[e] >= 2;
    route[e] = split ? -2 - sidx[e] : single[e];
    if (split) { rec[rl.seg + sidx[e]] = seg[e]; split_e[sidx[e]] = e; }
  }
  if (tid == 0) {   // rec[2] doubles as the reroute kernel's initial (empty) work-list length
    rec[0] = n_split; rec[1] = n_list; rec[2] = 0; rec[3] = 0;
    rec[rl.seg + n_split] = n_list;
  }

  // Split lists: position of an instance = number of nonzero instances of e on lower ranks; its
  // cumulative quota = its own share plus the shares of those.
  for (int e = tid; e < E; e += nt) {
    if (nz[e] < 2 || qrow[ml[e]] <= 0) continue;
    int pos = 0, below = 0;
    const int lim = mr[e] * N;
    for (int i = 0, r = 0, j = 0; i < lim; ++i) {
      const int v = qrow[r * s_phys + e_loc + j];
      if (rm[i] == e && v > 0) { ++pos; below += v; }
      if (++j == N) { j = 0; ++r; }
    }
    rec[rl.cum + seg[e] + pos] = below + qrow[ml[e]];
    rec[rl.inst + seg[e] + pos] = ml[e];
  }
  for (int i = tid; i < RN; i += nt) {
    const int e = rm[i];
    if (e < 0 || nz[e] < 2) continue;
    const int r = i / N, pi = r * s_phys + e_loc + (i - r * N);
    if (qrow[pi] <= 0) continue;
    const int qm = qrow[ml[e]];
    int pos = 0, below = 0;
    if (mr[e] < r && qm > 0) { pos = 1; below = qm; }
    const int lim = r * N;
    for (int i2 = 0, r2 = 0, j2 = 0; i2 < lim; ++i2) {
      const int v = qrow[r2 * s_phys + e_loc + j2];
      if (rm[i2] == e && v > 0) { ++pos; below += v; }
      if (++j2 == N) { j2 = 0; ++r2; }
    }
    rec[rl.cum + seg[e] + pos] = below + qrow[pi];
    rec[rl.inst + seg[e] + pos] = pi;
  }

  __syncthreads();   // split_e is complete
  // Cross-tile base of the stable rank, split experts only: exclusive prefix over the row's tiles.
  // One (split expert, tile) pair per thread-iteration so that all loads of a sweep are in flight.
  if (p.tiles > 0 && n_split > 0 && s >= p.rank_first && s < p.rank_first + p.rank_count) {
    const size_t trow = row * (size_t)p.max_tiles * E;
    if (p.tiles <= 32) {
      // a warp owns a split expert, a lane owns a tile
      for (int i = warp; i < n_split; i += nt >> 5) {
        const int e = split_e[i];
        const int v = lane < p.tiles ? __ldg(p.ws.tile_cnt + trow + (size_t)lane * E + e) : 0;
        int total;
        const int ex = warp_exclusive_scan(v, lane, &total);
        if (lane < p.tiles) {
          p.ws.tile_pref[trow + (size_t)lane * E + i] = ex;
          if (i < kSplitCap) {
            rec[rl.tp + lane * 3 * kSplitCap + i] = ex;
            // ranks [ex, ex + v) of this tile: inside one instance's quota interval?
            int lo = 0, res = -1;
            for (int k = seg[e]; k < seg[e] + nz[e]; ++k) {
              const int hi = rec[rl.cum + k];
              if (ex >= lo && ex + v <= hi) { res = rec[rl.inst + k]; break; }
              lo = hi;
            }
            rec[rl.tp + lane * 3 * kSplitCap + kSplitCap + i] = res;
            rec[rl.tp + lane * 3 * kSplitCap + 2 * kSplitCap + i] = e;
          }
        }
      }
    } else {
      for (int e = tid; e < E; e += nt) {
        if (nz[e] < 2) continue;
        const int32_t* c = p.ws.tile_cnt + trow + e;
        int32_t* o = p.ws.tile_pref + trow + sidx[e];
        int run = 0;
        for (int t0 = 0; t0 < p.tiles; t0 += 8) {
          int v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) v[u] = t0 + u < p.tiles ? __ldg(c + (size_t)(t0 + u) * E) : 0;
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (t0 + u < p.tiles) {
              o[(size_t)(t0 + u) * E] = run;
              if (sidx[e] < kSplitCap) {
                rec[rl.tp + (t0 + u) * 3 * kSplitCap + sidx[e]] = run;
                int lo = 0, res = -1;
                for (int k = seg[e]; k < seg[e] + nz[e]; ++k) {
                  const int hi = rec[rl.cum + k];
                  if (run >= lo && run + v[u] <= hi) { res = rec[rl.inst + k]; break; }
                  lo = hi;
                }
                rec[rl.tp + (t0 + u) * 3 * kSplitCap + kSplitCap + sidx[e]] = res;
                rec[rl.tp + (t0 + u) * 3 * kSplitCap + 2 * kSplitCap + sidx[e]] = e;
              }
              run += v[u];
            }
        }
      }
    }
  }

  // Send offsets of source s: exclusive scan over the destination ranks, total appended.
  if (warp == 0) {
    int32_t* send = p.out_offsets + (((size_t)b * 2 + 0) * R + s) * (R + 1);
    const int ch = (R + 31) / 32;
    const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
    int sum = 0;
    for (int r = i0; r < i1; ++r) sum += crow[r];
    int total;
    int pre = warp_exclusive_scan(sum, lane, &total);
    for (int r = i0; r < i1; ++r) { send[r] = pre; pre += crow[r]; }
    if (lane == 0) send[R] = total;
  }
}

}  // namespace

size_t route_smem_bytes(const Dims& d) { return route_layout(d).total; }

cudaError_t launch_route(const RouteParams& p, int batch, cudaStream_t stream) {
  const dim3 grid(p.d.R, batch);
  // few CTAs: 256 threads shorten each CTA's phases (latency); enough CTAs to fill the GPU twice
  // over: two warps per CTA spend far fewer issue slots on barriers, scans and idle lanes
  // (232 plans: solver + route stage 83.7 us with 256 threads, 62.9 with 128, 57.3 with 64)
  const int thr = (long long)p.d.R * batch >= 2 * 148 ? 64 : kRouteThreads;
  return launch_kernel(route_kernel, grid, dim3(thr), route_smem_bytes(p.d), stream,
                       p.pdl != 0, p);
}

cudaError_t configure_route(size_t smem) {
  return cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace topoep
