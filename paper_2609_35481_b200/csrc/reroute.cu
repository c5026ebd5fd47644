// Per-token replica assignment (paper, "System Design": the token-routing decisions q drive
// dispatch; here each assignment is told which physical instance executes it).
//
// Within a (plan, source rank, expert) group the assignments are ranked by flat index t*k+j
// and dealt to the expert's instances in ascending rank order, instance r taking q(s,e,r) of
// them.  For most (source, expert) pairs one instance takes everything, so the answer is one
// table lookup (route[e] >= 0) and the tile is streamed: load ids, look up, store.  Assignments
// of "split" experts (route[e] = -2-i) are pushed on a work list and patched afterwards; their
// stable rank is
//     [count of e in earlier tiles of the row]          prefix table written by the route kernel
//   + [count of e in earlier 128-id rows of this tile]  scan of the per-row totals
//   + [count of e in lower lanes of the row]            per-lane 4-bit counters, packed 8 per word
//   + [count of e earlier in the lane's own 4 ids]      compared in registers when pushed
// The counters are only ever summed and each 4-bit field belongs to one lane, the order of the
// work list is irrelevant (every item computes its own rank and writes its own output word), so
// no result depends on the order in which atomics arrive, and the output is identical for
// every tile size.  Split experts are ranked kSplitCap at a time; more of them only add passes.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

struct RerouteLayout { size_t cnt, base, route, seg, cum, inst, tbase, hdr, work, total; };

__host__ __device__ inline RerouteLayout reroute_layout(const Dims& d, int tile_ids) {
  const int rows = tile_ids / 128;
  RerouteLayout o;
  size_t at = 0;
  o.cnt = at;   at += sizeof(uint4) * (size_t)kSplitCap * rows;
  o.base = at;  at += sizeof(int) * (size_t)kSplitCap * rows;
  o.route = at; at += sizeof(int) * (size_t)d.E;
  o.seg = at;   at += sizeof(int) * (size_t)(d.E + 1);
  o.cum = at;   at += sizeof(int) * (size_t)d.P;
  o.inst = at;  at += sizeof(int) * (size_t)d.P;
  o.tbase = at; at += sizeof(int) * (size_t)kSplitCap;
  o.hdr = at;   at += sizeof(int) * 4;
  o.work = at;  at += sizeof(unsigned) * (size_t)tile_ids;
  o.total = at;
  return o;
}

// Sum of the eight 4-bit fields of x (each field <= 4 here).
__device__ __forceinline__ int nibble_sum(unsigned x) {
  const unsigned y = (x & 0x0f0f0f0fu) + ((x >> 4) & 0x0f0f0f0fu);
  return (int)((y * 0x01010101u) >> 24);
}

// Work item: position in the tile (14 bits) | earlier equal ids in the same lane group (2 bits)
// | split index (16 bits).
__device__ __forceinline__ void push(unsigned* work, int* n_work, int pos, int prev, int t) {
  const int slot = atomicAdd(n_work, 1);
  work[slot] = (unsigned)pos | ((unsigned)prev << 14) | ((unsigned)(-2 - t) << 16);
}

__global__ void __launch_bounds__(kMaxTileIds / kIdsPerThread) reroute_kernel(const RerouteParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const Dims d = p.d;
  const int E = d.E, P = d.P;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const int rows = 4 * nwarps;   // 128-id rows of the tile, in flat order
  const RerouteLayout lay = reroute_layout(d, p.tile_ids);
  uint4* cnt4 = reinterpret_cast<uint4*>(smem + lay.cnt);      // [kSplitCap][rows]
  unsigned* cntw = reinterpret_cast<unsigned*>(smem + lay.cnt);
  int* base = reinterpret_cast<int*>(smem + lay.base);         // [kSplitCap][rows]
  int* route = reinterpret_cast<int*>(smem + lay.route);
  int* seg = reinterpret_cast<int*>(smem + lay.seg);
  int* cum = reinterpret_cast<int*>(smem + lay.cum);
  int* inst = reinterpret_cast<int*>(smem + lay.inst);
  int* tbase = reinterpret_cast<int*>(smem + lay.tbase);
  int* hdr = reinterpret_cast<int*>(smem + lay.hdr);           // n_split, n_list, n_work
  unsigned* work = reinterpret_cast<unsigned*>(smem + lay.work);

  const size_t row = (size_t)b * d.R + s;
  const int begin = tile * p.tile_ids;
  const int count = min(p.tile_ids, p.n_ids - begin);
  const int32_t* ids = p.ids + row * (size_t)p.n_ids + begin;
  int32_t* out = p.out_token_replica + row * (size_t)p.n_ids + begin;

  // One round of independent loads: the ids, the route table, the head of the split record and
  // the tile bases of the first kSplitCap split experts (fetched before n_split is known; the
  // buffers are always large enough, surplus entries are ignored).
  int4 x[kIdsPerThread / 4];
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) x[j] = load_ids4(ids, j * nt + tid, count, p.vec_ok);
  const SplitRec rl = split_rec_layout(E, P);
  const int32_t* rec = p.ws.split_rec + row * (size_t)rl.ints;
  const int32_t* g_route = p.ws.route + row * E;
  const int32_t* g_tp = p.ws.tile_pref + (row * (size_t)p.max_tiles + tile) * E;
  const int fast_seg = min(E, kSplitCap) + 1, fast_list = min(P, kFastLists);
  for (int e = tid; e < E; e += nt) route[e] = g_route[e];
  for (int i = tid; i < fast_seg; i += nt) seg[i] = rec[rl.seg + i];
  for (int i = tid; i < fast_list; i += nt) { cum[i] = rec[rl.cum + i]; inst[i] = rec[rl.inst + i]; }
  if (tid < min(E, kSplitCap)) tbase[tid] = g_tp[tid];
  if (tid == 0) { hdr[0] = rec[0]; hdr[1] = rec[1]; hdr[2] = 0; }
  __syncthreads();

  // Stream: look up, store, push the split ones.  An ignored id and a split id both store -1
  // for now; the split ones are patched below.
  const unsigned uE = (unsigned)E;
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) {
    const int vec = j * nt + tid;
    const int e0 = x[j].x, e1 = x[j].y, e2 = x[j].z, e3 = x[j].w;
    const int t0 = (unsigned)e0 < uE ? route[e0] : -1;
    const int t1 = (unsigned)e1 < uE ? route[e1] : -1;
    const int t2 = (unsigned)e2 < uE ? route[e2] : -1;
    const int t3 = (unsigned)e3 < uE ? route[e3] : -1;
    if (min(min(t0, t1), min(t2, t3)) <= -2) {
      int* n_work = hdr + 2;
      if (t0 <= -2) push(work, n_work, 4 * vec + 0, 0, t0);
      if (t1 <= -2) push(work, n_work, 4 * vec + 1, (e0 == e1), t1);
      if (t2 <= -2) push(work, n_work, 4 * vec + 2, (e0 == e2) + (e1 == e2), t2);
      if (t3 <= -2) push(work, n_work, 4 * vec + 3, (e0 == e3) + (e1 == e3) + (e2 == e3), t3);
    }
    const int4 r = make_int4(max(t0, -1), max(t1, -1), max(t2, -1), max(t3, -1));
    if (p.vec_ok) {
      if (4 * vec < count) reinterpret_cast<int4*>(out)[vec] = r;
    } else {
      if (4 * vec + 0 < count) out[4 * vec + 0] = r.x;
      if (4 * vec + 1 < count) out[4 * vec + 1] = r.y;
      if (4 * vec + 2 < count) out[4 * vec + 2] = r.z;
      if (4 * vec + 3 < count) out[4 * vec + 3] = r.w;
    }
  }
  __syncthreads();   // also orders the stores above before the patches below
  const int n_work = hdr[2];
  if (n_work == 0) return;

  const int n_split = hdr[0], n_list = hdr[1];
  if (n_split > kSplitCap || n_list > kFastLists) {   // rare: fetch the rest of the record
    for (int i = tid; i <= n_split; i += nt) seg[i] = rec[rl.seg + i];
    for (int i = tid; i < n_list; i += nt) { cum[i] = rec[rl.cum + i]; inst[i] = rec[rl.inst + i]; }
  }
  bool broken = false;
  for (int p0 = 0; p0 < n_split; p0 += kSplitCap) {
    const int n_here = min(kSplitCap, n_split - p0);
    for (int i = tid; i < n_here * rows; i += nt) cnt4[i] = make_uint4(0u, 0u, 0u, 0u);
    if (p0 > 0 && tid < n_here) tbase[tid] = g_tp[p0 + tid];
    __syncthreads();
    // every item bumps the 4-bit counter of its (split expert, row, lane)
    for (int w = tid; w < n_work; w += nt) {
      const unsigned it = work[w];
      const int i = (int)(it >> 16) - p0;
      if (i < 0 || i >= n_here) continue;
      const int vec = (int)(it & 0x3fffu) >> 2;            // int4 index inside the tile
      const int rr = vec >> 5, ln = vec & 31;              // row, lane inside the row
      atomicAdd(&cntw[(i * rows + rr) * 4 + (ln >> 3)], 1u << (4 * (ln & 7)));
    }
    __syncthreads();
    // base[i][rr] = tile base + ids of split expert i in rows before rr
    for (int i = warp; i < n_here; i += nwarps) {
      int carry = tbase[i];
      for (int r0 = 0; r0 < rows; r0 += 32) {
        const int rr = r0 + lane;
        int tot = 0;
        if (rr < rows) {
          const uint4 c = cnt4[i * rows + rr];
          tot = nibble_sum(c.x) + nibble_sum(c.y) + nibble_sum(c.z) + nibble_sum(c.w);
        }
        int all;
        const int ex = warp_exclusive_scan(tot, lane, &all);
        if (rr < rows) base[i * rows + rr] = carry + ex;
        carry += all;
      }
    }
    __syncthreads();
    for (int w = tid; w < n_work; w += nt) {
      const unsigned it = work[w];
      const int i = (int)(it >> 16) - p0;
      if (i < 0 || i >= n_here) continue;
      const int pos = (int)(it & 0x3fffu), vec = pos >> 2;
      const int rr = vec >> 5, ln = vec & 31, word = ln >> 3, shift = 4 * (ln & 7);
      const uint4 c = cnt4[i * rows + rr];
      const unsigned cw[4] = {c.x, c.y, c.z, c.w};
      int rho = base[i * rows + rr] + (int)((it >> 14) & 3u);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (u < word) rho += nibble_sum(cw[u]);
        else if (u == word) rho += nibble_sum(cw[u] & ((1u << shift) - 1u));
      }
      int at = seg[p0 + i];
      const int end = seg[p0 + i + 1] - 1;
      while (at < end && rho >= cum[at]) ++at;
      broken |= rho >= cum[at];
      out[pos] = inst[at];
    }
    __syncthreads();
  }
  if (broken) atomicOr(p.ws.status, TOPOEP_FLAG_INTERNAL);
}

}  // namespace

size_t reroute_smem_bytes(const Dims& d, int tile_ids) { return reroute_layout(d, tile_ids).total; }

cudaError_t launch_reroute(const RerouteParams& p, int batch, cudaStream_t stream) {
  const dim3 grid(p.tiles, p.d.R, batch);
  const dim3 block(p.tile_ids / kIdsPerThread);
  reroute_kernel<<<grid, block, reroute_smem_bytes(p.d, p.tile_ids), stream>>>(p);
  return cudaGetLastError();
}

cudaError_t configure_reroute(size_t smem) {
  return cudaFuncSetAttribute(reroute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace topoep
