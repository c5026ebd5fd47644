// Dispatch permutation: where every assignment sits in its source rank's send buffer and in its
// destination rank's receive buffer (the step right after the planning path; the paper's
// "DeepEP dispatch and combine" paragraph leaves the buffer layout to its dispatch library, so
// the layout is defined here, in include/topoep.h).
//
//   send buffer of source s : ordered by (physical instance p, flat index) -- p ascends with
//                             (destination rank, instance), so each destination's block is
//                             contiguous and starts at the plan's send offset;
//   recv buffer of rank r   : ordered by (instance, source rank, flat index) -- every instance's
//                             tokens contiguous (grouped GEMM), sources in rank order inside.
//
// Both are stable sorts of token_replica, done as counting sorts with P bins in four kernels:
//   1. per-tile histogram of p            (the histogram kernel, P bins instead of E)
//   2. pos_tile_prefix_kernel, CTA = (plan, source): prefix over tiles of the tile counts and the
//      totals per (source, instance); pos_base_kernel, CTA = (plan, source): from the totals of
//      all sources the bases A0[p] (send) and B0[p] (receive), the instance offsets and, for a
//      window of tokens, its own dispatch counts and offsets
//   3. pos_rank_kernel, CTA = tile: stable rank of each assignment among the tile's equal p
//      (per-warp counters; lanes of a warp step that share an instance are ordered by ballots),
//      added to the bases.
// Ranks come from counts and prefix sums only, never from atomic arrival order.  Kernel 3 is
// bound by instruction issue, not by HBM; it is off the planning path.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

constexpr int kPosThreads = 256;
// ids per thread of the ranking kernel = steps of a warp's dependent chain (measured per
// 232-plan call: 16 -> 3.08 ms, 8 -> 2.83 ms, 4 -> 3.73 ms)
constexpr int kPosIds = 8;

// 2a. CTA = (plan, source): exclusive prefix over tiles of the tile counts, in place, and the
// totals tot[s][p] = assignments of source s on instance p inside the window.
__global__ void __launch_bounds__(kPosThreads) pos_tile_prefix_kernel(const PosParams p) {
  const int P = p.d.P;
  const int s = blockIdx.x, b = blockIdx.y;
  const size_t row = (size_t)b * p.d.R + s;
  int32_t* cnt = p.pos_cnt + row * (size_t)p.tiles * P;
  for (int i = threadIdx.x; i < P; i += blockDim.x) {
    int run = 0;
    for (int t0 = 0; t0 < p.tiles; t0 += 8) {
      int v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = t0 + u < p.tiles ? cnt[(size_t)(t0 + u) * P + i] : 0;
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (t0 + u < p.tiles) { cnt[(size_t)(t0 + u) * P + i] = run; run += v[u]; }
    }
    p.pos_tot[row * P + i] = run;
  }
}

// 2b. CTA = (plan, source): bases of (source, instance) in the send and receive buffers, from the
// totals of every source -- nothing here depends on the plan in the workspace, so the positions
// of any window of tokens (a chunk of a two-chunk pipeline) come out the same way as a whole
// plan's.  Also the window's dispatch counts and offsets (row s) and the instance offsets.
__global__ void __launch_bounds__(kPosThreads) pos_base_kernel(const PosParams p) {
  extern __shared__ int sm[];   // mine[P], lower[P], U[P], per-warp totals, crow[R], lrow[R]
  const Dims d = p.d;
  const int R = d.R, P = d.P, s_phys = d.s_phys;
  const int s = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nw = nt >> 5;
  int* mine = sm;
  int* lower = sm + P;
  int* Us = sm + 2 * P;
  int* warp_tot = sm + 3 * P;
  int* crow = warp_tot + nw + 1;
  int* lrow = crow + R;
  const size_t row = (size_t)b * R + s;
  const int32_t* tot = p.pos_tot + (size_t)b * R * P;
  // column sums over the sources: everything (U) and the sources below s (loads eight at a time)
  for (int i = tid; i < P; i += nt) {
    int lo = 0, all = 0;
    for (int s0 = 0; s0 < R; s0 += 8) {
      int v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = s0 + u < R ? __ldg(tot + (size_t)(s0 + u) * P + i) : 0;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        all += v[u];
        lo += s0 + u < s ? v[u] : 0;
      }
    }
    Us[i] = all;
    lower[i] = lo;
    mine[i] = __ldg(tot + (size_t)s * P + i);
  }
  __syncthreads();
  // A0[p] = assignments of source s on instances below p (exclusive scan over p)
  int32_t* A0 = p.pos_a + row * P;
  {
    const int chunk = (P + nt - 1) / nt;
    const int i0 = min(P, tid * chunk), i1 = min(P, i0 + chunk);
    int sum = 0;
    for (int i = i0; i < i1; ++i) sum += mine[i];
    int total;
    int ex = warp_exclusive_scan(sum, lane, &total);
    if (lane == 0) warp_tot[warp] = total;
    __syncthreads();
    for (int w = 0; w < warp; ++w) ex += warp_tot[w];
    for (int i = i0; i < i1; ++i) { A0[i] = ex; ex += mine[i]; }
  }
  // B0[p] = start of instance p's segment in its rank's receive buffer + lower sources on p
  int32_t* B0 = p.pos_b + row * P;
  for (int i = tid; i < P; i += nt) {
    const int r = i / s_phys;
    int acc = lower[i];
    for (int j = r * s_phys; j < i; ++j) acc += Us[j];
    B0[i] = acc;
  }
  if (s == 0 && p.out_instance_offsets) {
    int32_t* off = p.out_instance_offsets + (size_t)b * R * (s_phys + 1);
    for (int i = tid; i < R * (s_phys + 1); i += nt) {
      const int r = i / (s_phys + 1), l = i - r * (s_phys + 1);
      int acc = 0;
      for (int j = 0; j < l; ++j) acc += Us[r * s_phys + j];
      off[i] = acc;
    }
  }
  if (p.out_counts || p.out_offsets) {
    // row s of the counts, and for each destination what the lower sources send to it
    for (int r = tid; r < R; r += nt) {
      int c = 0, lo = 0;
      for (int l = 0; l < s_phys; ++l) { c += mine[r * s_phys + l]; lo += lower[r * s_phys + l]; }
      crow[r] = c;
      lrow[r] = lo;
      if (p.out_counts) p.out_counts[row * R + r] = c;
    }
    __syncthreads();
    if (p.out_offsets) {
      int32_t* send = p.out_offsets + (((size_t)b * 2 + 0) * R + s) * (R + 1);
      int32_t* recv = p.out_offsets + ((size_t)b * 2 + 1) * R * (R + 1);
      if (warp == 0) {   // send offsets of source s: exclusive scan over the destinations
        const int ch = (R + 31) / 32;
        const int i0 = min(R, lane * ch), i1 = min(R, i0 + ch);
        int sum = 0;
        for (int r = i0; r < i1; ++r) sum += crow[r];
        int total;
        int pre = warp_exclusive_scan(sum, lane, &total);
        for (int r = i0; r < i1; ++r) { send[r] = pre; pre += crow[r]; }
        if (lane == 0) send[R] = total;
      }
      // receive offsets: entry s of every destination's row; the last source appends the total
      for (int r = tid; r < R; r += nt) {
        recv[(size_t)r * (R + 1) + s] = lrow[r];
        if (s == R - 1) recv[(size_t)r * (R + 1) + R] = lrow[r] + crow[r];
      }
    }
  }
}

__global__ void __launch_bounds__(kMaxTileIds / kPosIds) pos_rank_kernel(const PosParams p) {
  extern __shared__ int sm[];   // base_a[P], base_b[P], wh[nwarps][P]
  const Dims d = p.d;
  const int P = d.P;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
  int* base_a = sm;
  int* base_b = sm + P;
  int* wh = sm + 2 * P;
  const size_t row = (size_t)b * d.R + s;
  const int begin = tile * p.tile_ids;
  const int count = min(p.tile_ids, p.n_ids - begin);
  const int32_t* tr = p.token_replica + row * (size_t)p.row_stride + p.first_id + begin;

  // this warp's 512 assignments: step j covers 32 consecutive ones, so (step, lane) is flat order
  const int wbase = warp * (32 * kPosIds);
  int x[kPosIds];
#pragma unroll
  for (int j = 0; j < kPosIds; ++j) {
    const int i = wbase + j * 32 + lane;
    x[j] = i < count ? __ldg(tr + i) : -1;
  }
  const int32_t* tp = p.pos_cnt + (row * (size_t)p.tiles + tile) * P;
  for (int i = tid; i < P; i += nt) {
    const int t = tp[i];
    base_a[i] = p.pos_a[row * P + i] + t;
    base_b[i] = p.pos_b[row * P + i] + t;
  }
  for (int i = tid; i < nwarps * P; i += nt) wh[i] = 0;
  __syncthreads();

  // In-warp stable rank, 32 assignments per step.  All lanes add 1 to their instance's per-warp
  // counter; the counter value before the step is the rank of the step's FIRST lane with that
  // instance.  Only instances met twice or more in the step (the counter grew by more than one)
  // need their lanes ordered, which takes one ballot per such instance -- instead of a
  // __match_any_sync per step, whose cost on B200 grows with every distinct value in the warp.
  int* my = wh + warp * P;
  int rho[kPosIds];
  const unsigned lt = lanemask_lt();
#pragma unroll
  for (int j = 0; j < kPosIds; ++j) {
    const int v = x[j];
    const bool valid = v >= 0 && v < P;
    const int before = valid ? my[v] : 0;
    __syncwarp();
    if (valid) atomicAdd(&my[v], 1);
    __syncwarp();
    const int grown = valid ? my[v] - before : 0;
    int r = before;
    unsigned todo = __ballot_sync(0xffffffffu, grown > 1);
    while (todo) {   // uniform across the warp
      const int key = __shfl_sync(0xffffffffu, v, __ffs(todo) - 1);
      const unsigned peers = __ballot_sync(0xffffffffu, valid && v == key);
      if (valid && v == key) r = before + __popc(peers & lt);
      todo &= ~peers;
    }
    rho[j] = r;
  }
  __syncthreads();
  // per-warp totals -> exclusive prefix over the warps of the tile
  for (int i = tid; i < P; i += nt) {
    int run = 0;
    for (int w = 0; w < nwarps; ++w) {
      const int t = wh[w * P + i];
      wh[w * P + i] = run;
      run += t;
    }
  }
  __syncthreads();
  int32_t* send = p.out_send_pos + row * (size_t)p.n_ids + begin;
  int32_t* recv = p.out_recv_pos + row * (size_t)p.n_ids + begin;
#pragma unroll
  for (int j = 0; j < kPosIds; ++j) {
    const int i = wbase + j * 32 + lane;
    const int v = x[j];
    int a = -1, c = -1;
    if (v >= 0 && v < P) {
      const int k = rho[j] + my[v];
      a = base_a[v] + k;
      c = base_b[v] + k;
    }
    if (i < count) { send[i] = a; recv[i] = c; }
  }
}

}  // namespace

size_t pos_rank_smem_bytes(const Dims& d, int tile_ids) {
  return sizeof(int) * ((size_t)2 * d.P + (size_t)(tile_ids / (32 * kPosIds)) * d.P);
}

size_t pos_prefix_smem_bytes(const Dims& d) {
  return sizeof(int) * ((size_t)3 * d.P + kPosThreads / 32 + 1 + 2 * (size_t)d.R);
}

cudaError_t configure_dispatch(const Dims& d) {
  cudaError_t e = cudaFuncSetAttribute(pos_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)pos_rank_smem_bytes(d, kMaxTileIds));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(pos_base_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)pos_prefix_smem_bytes(d));
}

cudaError_t launch_dispatch(const PosParams& p, int batch, cudaStream_t stream) {
  // 1. per-tile histogram of the instance ids: the histogram kernel with P bins
  HistParams hp = {};
  hp.d = p.d;
  hp.d.E = p.d.P;
  hp.ws = p.ws;
  hp.ws.tile_cnt = p.pos_cnt;
  hp.ws.tile_cnt16 = 0;   // these counts become prefixes over tiles in place: 32 bits
  hp.ids = p.token_replica;
  hp.rank_first = 0;
  hp.rank_count = p.d.R;
  hp.n_ids = p.n_ids;
  hp.row_stride = p.row_stride;
  hp.first_id = p.first_id;
  hp.tiles = p.tiles;
  hp.max_tiles = p.tiles;
  hp.tile_ids = p.tile_ids;
  hp.vec_ok = (p.n_ids % 4 == 0) && (p.row_stride % 4 == 0) && (p.first_id % 4 == 0) &&
              ((reinterpret_cast<uintptr_t>(p.token_replica) & 15u) == 0);
  hp.ws.status = p.scratch_status;   // a stray instance id must not raise the plan's BAD_ID flag
  cudaError_t e = launch_hist(hp, batch, 0, stream);
  if (e != cudaSuccess) return e;
  // 2. bases and tile prefixes
  pos_tile_prefix_kernel<<<dim3(p.d.R, batch), kPosThreads, 0, stream>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  pos_base_kernel<<<dim3(p.d.R, batch), kPosThreads, pos_prefix_smem_bytes(p.d), stream>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // 3. stable ranks inside the tile
  const dim3 grid(p.tiles, p.d.R, batch);
  const dim3 block(p.tile_ids / kPosIds);
  pos_rank_kernel<<<grid, block, pos_rank_smem_bytes(p.d, p.tile_ids), stream>>>(p);
  return cudaGetLastError();
}

}  // namespace topoep
