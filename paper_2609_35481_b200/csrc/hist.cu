// Routing-matrix histogram (paper, "System Model", Eq. Omega):
//   omega[s][e] = number of (token, expert) assignments of source rank s that select expert e.
//
// One CTA counts one tile of one source rank's flat id array in shared memory and writes the
// tile's counts.  The last CTA of a (plan, rank) row to finish turns the row's tile counts into
// exclusive prefixes over tiles (the reroute kernel's cross-tile base for the stable rank of an
// assignment) and writes the row of omega.  No global atomics on data, no zero-fill pass:
// the result never depends on arrival order.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

// Warp-aggregated add: lanes holding the same expert elect one leader that adds their count.
__device__ __forceinline__ void add_matched(int* cnt, int e, unsigned mask, unsigned lane) {
  const unsigned peers = __match_any_sync(mask, e);
  if ((unsigned)(__ffs(peers) - 1) == lane) atomicAdd(&cnt[e], __popc(peers));
}

template <int MODE>
__device__ __forceinline__ void count_one(int* cnt, int e, int E, bool in_range, unsigned lane,
                                          bool& bad) {
  const bool valid = in_range && e >= 0 && e < E;
  bad |= in_range && !valid && e != -1;
  if (MODE == 0) {
    const unsigned mask = __ballot_sync(0xffffffffu, valid);
    if (valid) add_matched(cnt, e, mask, lane);
  } else {
    if (valid) atomicAdd(&cnt[e], 1);
  }
}

template <int MODE>
__global__ void __launch_bounds__(kMaxTileIds / kIdsPerThread) hist_kernel(const HistParams p) {
  extern __shared__ int cnt[];   // [E]
  __shared__ bool is_last;
  const int E = p.d.E;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int nt = blockDim.x, tid = threadIdx.x;
  const unsigned lane = tid & 31;
  for (int e = tid; e < E; e += nt) cnt[e] = 0;
  __syncthreads();

  const size_t row = (size_t)b * p.d.R + s;
  const int32_t* ids = p.ids + row * (size_t)p.n_ids;
  const int begin = tile * p.tile_ids;
  const int count = min(p.tile_ids, p.n_ids - begin);   // may be <= 0 only when n_ids == 0
  bool bad = false;

  if (p.vec_ok) {
    const int4* v = reinterpret_cast<const int4*>(ids + begin);
    const int nvec = count > 0 ? count >> 2 : 0;
    int4 x[kIdsPerThread / 4];
#pragma unroll
    for (int j = 0; j < kIdsPerThread / 4; ++j) {
      const int i = j * nt + tid;
      x[j] = i < nvec ? __ldg(v + i) : make_int4(-1, -1, -1, -1);
    }
#pragma unroll
    for (int j = 0; j < kIdsPerThread / 4; ++j) {
      const bool in = j * nt + tid < nvec;
      count_one<MODE>(cnt, x[j].x, E, in, lane, bad);
      count_one<MODE>(cnt, x[j].y, E, in, lane, bad);
      count_one<MODE>(cnt, x[j].z, E, in, lane, bad);
      count_one<MODE>(cnt, x[j].w, E, in, lane, bad);
    }
  } else {
    int x[kIdsPerThread];
#pragma unroll
    for (int j = 0; j < kIdsPerThread; ++j) {
      const int i = j * nt + tid;
      x[j] = i < count ? __ldg(ids + begin + i) : -1;
    }
#pragma unroll
    for (int j = 0; j < kIdsPerThread; ++j)
      count_one<MODE>(cnt, x[j], E, j * nt + tid < count, lane, bad);
  }
  if (bad) atomicOr(p.ws.status, TOPOEP_FLAG_BAD_ID);
  __syncthreads();

  int32_t* row_tiles = p.ws.tile_pref + row * (size_t)p.max_tiles * E;
  for (int e = tid; e < E; e += nt) row_tiles[(size_t)tile * E + e] = cnt[e];

  // Last-block-done: publish this tile, take a ticket, the holder of the last ticket scans the row.
  __threadfence();
  __syncthreads();
  if (tid == 0) is_last = (atomicAdd(&p.ws.hist_tickets[row], 1u) == (unsigned)(p.tiles - 1));
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  int32_t* omega = p.ws.omega + row * (size_t)E;
  int32_t* user = p.out_omega ? p.out_omega + row * (size_t)E : nullptr;
  for (int e = tid; e < E; e += nt) {
    int run = 0;
    for (int t = 0; t < p.tiles; ++t) {
      int32_t* cell = row_tiles + (size_t)t * E + e;
      const int c = __ldcg(cell);
      *cell = run;
      run += c;
    }
    omega[e] = run;
    if (user) user[e] = run;
  }
  if (tid == 0) p.ws.hist_tickets[row] = 0;   // ready for the next launch
}

__global__ void empty_kernel() {}

}  // namespace

size_t hist_smem_bytes(const Dims& d) { return sizeof(int) * (size_t)d.E; }

cudaError_t launch_hist(const HistParams& p, int batch, int mode, cudaStream_t stream) {
  const dim3 grid(p.tiles, p.d.R, batch);
  const dim3 block(p.tile_ids / kIdsPerThread);
  const size_t smem = hist_smem_bytes(p.d);
  if (mode == 0) hist_kernel<0><<<grid, block, smem, stream>>>(p);
  else hist_kernel<1><<<grid, block, smem, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_empty(int count, cudaStream_t stream) {
  for (int i = 0; i < count; ++i) empty_kernel<<<1, 32, 0, stream>>>();
  return cudaGetLastError();
}

}  // namespace topoep
