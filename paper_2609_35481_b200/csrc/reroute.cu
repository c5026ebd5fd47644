// Per-token replica assignment (paper, "System Design": the token-routing decisions q drive
// dispatch; here each assignment is told which physical instance executes it).
//
// Within a (plan, source rank, expert) group the assignments are ranked by flat index t*k+j
// and dealt to the expert's instances in ascending rank order, instance r taking q(s,e,r) of
// them.  The rank of an assignment is
//     [count of e in earlier tiles of the row]            (prefix table of the histogram kernel)
//   + [count of e in earlier warps of this tile]          (per-warp counters, scanned once)
//   + [count of e earlier in this warp]                   (__match_any_sync + popcount)
// so it never depends on atomic arrival order and is identical for every tile size.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

struct RerouteLayout { size_t seg, cum, inst, wh, total; };

__host__ __device__ inline RerouteLayout reroute_layout(const Dims& d, int warps) {
  RerouteLayout o;
  size_t at = 0;
  o.seg = at;  at += sizeof(int) * (size_t)(d.E + 1);
  o.cum = at;  at += sizeof(int) * (size_t)d.P;
  o.inst = at; at += sizeof(int) * (size_t)d.P;
  o.wh = at;   at += sizeof(int) * (size_t)warps * d.E;
  o.total = at;
  return o;
}

__global__ void __launch_bounds__(kMaxTileIds / kIdsPerThread) reroute_kernel(const RerouteParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const Dims d = p.d;
  const int E = d.E, P = d.P;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  const unsigned full = 0xffffffffu;
  const RerouteLayout lay = reroute_layout(d, nwarps);
  int* seg = reinterpret_cast<int*>(smem + lay.seg);
  int* cum = reinterpret_cast<int*>(smem + lay.cum);
  int* inst = reinterpret_cast<int*>(smem + lay.inst);
  int* wh = reinterpret_cast<int*>(smem + lay.wh);   // [nwarps][E]

  const size_t row = (size_t)b * d.R + s;
  const int32_t* ids = p.ids + row * (size_t)p.n_ids;
  int32_t* out = p.out_token_replica + row * (size_t)p.n_ids;

  // This warp's 512 ids: step j covers 32 consecutive ids, so (step, lane) is the flat order.
  const int base = tile * p.tile_ids + warp * (32 * kIdsPerThread);
  int x[kIdsPerThread];
#pragma unroll
  for (int j = 0; j < kIdsPerThread; ++j) {
    const int i = base + j * 32 + lane;
    x[j] = i < p.n_ids ? __ldg(ids + i) : -1;
  }

  // Quota table of source s: cumulative q over each expert's instances in ascending rank order.
  const int32_t* seg_g = p.ws.seg_start + (size_t)b * (E + 1);
  const int32_t* inst_g = p.ws.inst_sorted + (size_t)b * P;
  const int32_t* q_g = p.ws.q + row * (size_t)P;
  for (int e = tid; e <= E; e += nt) seg[e] = seg_g[e];
  for (int i = tid; i < nwarps * E; i += nt) wh[i] = 0;
  __syncthreads();
  for (int e = tid; e < E; e += nt) {
    int run = 0;
    for (int i = seg[e]; i < seg[e + 1]; ++i) {
      const int pi = inst_g[i];
      run += q_g[pi];
      cum[i] = run;
      inst[i] = pi;
    }
  }

  // In-warp stable rank, relative to the warp's first id.
  int* my = wh + warp * E;
  int rho[kIdsPerThread];
  const unsigned lt = lanemask_lt();
#pragma unroll
  for (int j = 0; j < kIdsPerThread; ++j) {
    const int e = x[j];
    const bool valid = e >= 0 && e < E;
    const unsigned mask = __ballot_sync(full, valid);
    int r = 0;
    if (valid) {
      const unsigned peers = __match_any_sync(mask, e);
      const int leader = __ffs(peers) - 1;
      int old = 0;
      if (lane == leader) { old = my[e]; my[e] = old + __popc(peers); }
      old = __shfl_sync(peers, old, leader);
      r = old + __popc(peers & lt);
    }
    rho[j] = r;
    __syncwarp();
  }
  __syncthreads();

  // Per-warp totals -> exclusive prefix over warps, on top of the earlier tiles' count.
  const int32_t* tp = p.ws.tile_pref + (row * (size_t)p.max_tiles + tile) * E;
  for (int e = tid; e < E; e += nt) {
    int run = tp[e];
    for (int w = 0; w < nwarps; ++w) {
      const int t = wh[w * E + e];
      wh[w * E + e] = run;
      run += t;
    }
  }
  __syncthreads();

  bool broken = false;
#pragma unroll
  for (int j = 0; j < kIdsPerThread; ++j) {
    const int i = base + j * 32 + lane;
    const int e = x[j];
    int res = -1;
    if (e >= 0 && e < E) {
      const int r = rho[j] + my[e];
      int at = seg[e];
      const int end = seg[e + 1] - 1;
      while (at < end && r >= cum[at]) ++at;
      broken |= r >= cum[at];
      res = inst[at];
    }
    if (i < p.n_ids) out[i] = res;
  }
  if (broken) atomicOr(p.ws.status, TOPOEP_FLAG_INTERNAL);
}

}  // namespace

size_t reroute_smem_bytes(const Dims& d, int tile_ids) {
  return reroute_layout(d, tile_ids / (32 * kIdsPerThread)).total;
}

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
