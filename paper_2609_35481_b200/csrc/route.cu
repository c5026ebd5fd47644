// Per-source routing tables and send offsets (paper, "System Design": the token-routing
// decisions q drive dispatch; Implementation, "DeepEP dispatch and combine" paragraph: the counts
// a rank will receive are computed on the device from the routing, with no host round trip).
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

struct RouteLayout { size_t rm, qrow, mr, ml, nz, single, sidx, seg, crow, split_e, warp_tot, cum_s, inst_s, total; };

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
  o.cum_s = at;    at += sizeof(int) * (size_t)d.P;
  o.inst_s = at;   at += sizeof(int) * (size_t)d.P;
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
  int* cum_s = reinterpret_cast<int*>(smem + lay.cum_s);     // [n_list] cumulative quotas
  int* inst_s = reinterpret_cast<int*>(smem + lay.inst_s);   // [n_list] instances

  const size_t row = (size_t)b * R + s;
  const int RN = R * N;
  // static tables before the solver is known to be done, its results after
#pragma unroll 4
  for (int e = tid; e < E; e += nt) {
    const int r = p.ws.main_rank[e];
    mr[e] = r;
    ml[e] = r * s_phys + p.ws.main_local[e];
  }
  pdl_wait();
#pragma unroll 4
  for (int i = tid; i < RN; i += nt) rm[i] = p.ws.replica_map[(size_t)b * RN + i];
#pragma unroll 4
  for (int i = tid; i < P; i += nt) qrow[i] = p.ws.q[row * P + i];
#pragma unroll 4
  for (int r = tid; r < R; r += nt) crow[r] = p.ws.counts[row * R + r];
  __syncthreads();

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
  block_scan2(nz, E, sidx, seg, warp_tot, tid, nt);
  const int n_split = sidx[E], n_list = seg[E];

  // second round of loads: tile counts of the split experts (prefix over tiles below)
  const SplitRec rl = split_rec_layout(E, P, p.max_tiles);
  int32_t* rec = p.ws.split_rec + row * (size_t)rl.ints;
  int32_t* route = p.ws.route + row * E;
#pragma unroll 1
  for (int e = tid; e < E; e += nt) {
    const bool split = nz[e] >= 2;
    route[e] = split ? -2 - sidx[e] : single[e];
    if (split) { rec[rl.seg + sidx[e]] = seg[e]; split_e[sidx[e]] = e; }
  }
  if (tid == 0) {   // rec[2] doubles as the reroute kernel's initial (empty) work-list length
    rec[0] = n_split; rec[1] = n_list; rec[2] = 0; rec[3] = 0;
    rec[rl.seg + n_split] = n_list;
  }

  __syncthreads();   // split_e is complete
  // Split lists, one warp per split expert: the instances with a share in ascending rank order
  // (the replica slots are already in rank order; the main instance goes in front of the first
  // slot on a higher rank) with cumulative quotas.  Lanes take the slots, positions come from a
  // ballot, quotas from a warp scan.  The same warp then turns the expert's tile counts into
  // tile prefixes and checks each tile's rank interval against the quotas.
  const bool in_window = s >= p.rank_first && s < p.rank_first + p.rank_count;
  const bool warp_tiles = p.tiles > 0 && p.tiles <= 32 && in_window;
  const size_t trow = row * (size_t)p.max_tiles * E;
#pragma unroll 1
  for (int i = warp; i < n_split; i += nt >> 5) {
    const int e = split_e[i];
    const int base = seg[e], qm = qrow[ml[e]], rmain = mr[e];
    // tile count of (e, tile = lane): in flight while the list is built
    int tv = 0;
    if (warp_tiles && lane < p.tiles)
      tv = p.ws.tile_cnt16 ? (int)__ldg(reinterpret_cast<const unsigned short*>(p.ws.tile_cnt) + trow + (size_t)lane * E + e)
                           : __ldg(p.ws.tile_cnt + trow + (size_t)lane * E + e);
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
      const unsigned m = __ballot_sync(0xffffffffu, v > 0);
      if (m == 0) continue;   // no instance of e among these 32 slots (the common case)
      int tot;
      const int ex = warp_exclusive_scan(v, lane, &tot);
      const bool below_main = v > 0 && r < rmain;
      main_pos += __popc(__ballot_sync(0xffffffffu, below_main));
      main_below += __reduce_add_sync(0xffffffffu, below_main ? v : 0);
      if (v > 0) {
        const bool after_main = qm > 0 && rmain < r;
        const int pos = carry_pos + __popc(m & lanemask_lt()) + (after_main ? 1 : 0);
        cum_s[CK(p.ws.status, base + pos, P)] = carry_cum + ex + v + (after_main ? qm : 0);
        inst_s[CK(p.ws.status, base + pos, P)] = pi;
      }
      carry_pos += __popc(m);
      carry_cum += tot;
    }
    if (lane == 0 && qm > 0) {
      cum_s[CK(p.ws.status, base + main_pos, P)] = main_below + qm;
      inst_s[CK(p.ws.status, base + main_pos, P)] = ml[e];
    }
    __syncwarp();
    const int n_e = nz[e];
#pragma unroll 1
    for (int k = lane; k < n_e; k += 32) {
      rec[rl.cum + base + k] = cum_s[base + k];
      rec[rl.inst + base + k] = inst_s[base + k];
    }
    if (warp_tiles) {
      // exclusive prefix over the row's tiles: the cross-tile base of the stable rank
      int total;
      const int ex = warp_exclusive_scan(tv, lane, &total);
      if (lane < p.tiles) {
        p.ws.tile_pref[trow + (size_t)lane * E + i] = ex;
        if (i < kSplitCap) {
          // ranks [ex, ex + tv) of this tile: inside one instance's quota interval?
          int lo = 0, res = -1;
#pragma unroll 1
          for (int k = base; k < base + n_e; ++k) {
            const int hi = cum_s[k];
            if (ex >= lo && ex + tv <= hi) { res = inst_s[k]; break; }
            lo = hi;
          }
          int32_t* t3 = rec + rl.tp + lane * 3 * kSplitCap + i;
          t3[0] = ex;
          t3[kSplitCap] = res;
          t3[2 * kSplitCap] = e;
        }
      }
    }
  }
  if (p.tiles > 32 && n_split > 0 && in_window) {   // long rows: a thread walks an expert's tiles
    __syncthreads();   // the lists of every split expert are in shared memory
#pragma unroll 1
    for (int e = tid; e < E; e += nt) {
      if (nz[e] < 2) continue;
      const int32_t* c = p.ws.tile_cnt + trow + e;
      const unsigned short* c16 = reinterpret_cast<const unsigned short*>(p.ws.tile_cnt) + trow + e;
      int32_t* o = p.ws.tile_pref + trow + sidx[e];
      int run = 0;
#pragma unroll 1
      for (int t0 = 0; t0 < p.tiles; t0 += 8) {
        int v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          v[u] = t0 + u >= p.tiles ? 0 : p.ws.tile_cnt16 ? (int)__ldg(c16 + (size_t)(t0 + u) * E)
                                                         : __ldg(c + (size_t)(t0 + u) * E);
#pragma unroll
        for (int u = 0; u < 8; ++u)
          if (t0 + u < p.tiles) {
            o[(size_t)(t0 + u) * E] = run;
            if (sidx[e] < kSplitCap) {
              int lo = 0, res = -1;
#pragma unroll 1
              for (int k = seg[e]; k < seg[e] + nz[e]; ++k) {
                const int hi = cum_s[k];
                if (run >= lo && run + v[u] <= hi) { res = inst_s[k]; break; }
                lo = hi;
              }
              int32_t* t3 = rec + rl.tp + (t0 + u) * 3 * kSplitCap + sidx[e];
              t3[0] = run;
              t3[kSplitCap] = res;
              t3[2 * kSplitCap] = e;
            }
            run += v[u];
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
#pragma unroll 1
    for (int r = i0; r < i1; ++r) sum += crow[r];
    int total;
    int pre = warp_exclusive_scan(sum, lane, &total);
#pragma unroll 1
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
  const int thr = (long long)p.d.R * batch >= 2ll * p.d.sms ? 64 : kRouteThreads;
  return launch_kernel(route_kernel, grid, dim3(thr), route_smem_bytes(p.d), stream,
                       p.pdl != 0, p);
}

cudaError_t configure_route(size_t smem) {
  return cudaFuncSetAttribute(route_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace topoep
