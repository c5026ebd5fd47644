// Routing-matrix histogram (paper, "System Model", Eq. Omega):
//   omega[s][e] = number of (token, expert) assignments of source rank s that select expert e.
//
// hist_kernel: one CTA counts one tile of one source rank's flat id array in shared memory and
// writes the tile's counts.  omega_kernel: omega[s][e] = sum of the tile counts (plus the two
// derived layouts the solver reads).  No global
// atomics, no zero-fill pass, no inter-CTA hand-off: the result cannot depend on arrival order,
// and the per-tile counts are what the later kernels turn into the cross-tile base of an
// assignment's stable rank.
//
// Counting uses plain shared-memory atomics by default.  The warp-aggregated variant
// (__match_any_sync, one atomic per distinct id per warp) is kept behind a knob: on B200
// match.any costs ~160-250 issue cycles per warp instruction, several times the cost of the
// conflicts it removes, even on Zipf(1.5) routing.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

// Count one id, branch-free in the default mode: an id outside [0,E) is clamped onto the spare
// bin cnt[E].  `mx` tracks the largest (unsigned)(e + 1) seen: it exceeds E exactly when some id
// was neither in range nor the padding value -1.
template <int MODE>
__device__ __forceinline__ void count_one(int* cnt, int e, unsigned E, unsigned lane, unsigned& mx) {
  mx = max(mx, (unsigned)(e + 1));
  if (MODE == 1) {
    const bool valid = (unsigned)e < E;
    const unsigned mask = __ballot_sync(0xffffffffu, valid);
    if (valid) {
      const unsigned peers = __match_any_sync(mask, e);
      if ((unsigned)(__ffs(peers) - 1) == lane) atomicAdd(&cnt[e], __popc(peers));
    }
  } else {
    atomicAdd(&cnt[min((unsigned)e, E)], 1);
  }
}

// IPT ids per thread (IPT/4 int4 loads in flight per thread); blockDim.x = tile_ids / IPT.
template <int MODE, int IPT>
__global__ void __launch_bounds__(kMaxTileIds / kIdsPerThread) hist_kernel(const HistParams p) {
  extern __shared__ int cnt[];   // [E + 1]: the last bin collects ignored ids
  const int E = p.d.E;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int nt = blockDim.x, tid = threadIdx.x;
  const unsigned lane = tid & 31;

  // workspace rows are indexed by the global source rank, the caller's buffer by its window
  const size_t row = (size_t)b * p.d.R + p.rank_first + s;
  const int begin = tile * p.tile_ids;
  const int count = min(p.tile_ids, p.n_ids - begin);   // <= 0 only when n_ids == 0
  const int32_t* ids = p.ids + ((size_t)b * p.rank_count + s) * (size_t)p.row_stride + p.first_id + begin;
  int4 x[IPT / 4];
#pragma unroll
  for (int j = 0; j < IPT / 4; ++j) x[j] = load_ids4(ids, j * nt + tid, count, p.vec_ok);
  for (int e = tid; e <= E; e += nt) cnt[e] = 0;
  __syncthreads();
  unsigned mx = 0;
#pragma unroll
  for (int j = 0; j < IPT / 4; ++j) {
    count_one<MODE>(cnt, x[j].x, E, lane, mx);
    count_one<MODE>(cnt, x[j].y, E, lane, mx);
    count_one<MODE>(cnt, x[j].z, E, lane, mx);
    count_one<MODE>(cnt, x[j].w, E, lane, mx);
  }
  pdl_wait();   // the ids are nobody's output; everything written below may still be in use
  if (mx > (unsigned)E) atomicOr(p.ws.status, TOPOEP_FLAG_BAD_ID);
  if (p.pack) {
    // One-byte copy of the tile for the reroute kernel of a large call (E <= 256, rows of whole
    // 16-byte groups): the low byte of every id, four per word, same flat order.  Streaming
    // stores: the copy is read once, long after it has left L2.  An id outside [0, E) (padding
    // or invalid) cannot be told from a valid one in a byte: the tile is flagged and the reroute
    // kernel reads its 4-byte ids.
    unsigned* dst = reinterpret_cast<unsigned*>(p.ws.ids8 + row * (size_t)p.n_ids + begin);
    const unsigned uE = (unsigned)E;
    int outside = 0;
#pragma unroll
    for (int j = 0; j < IPT / 4; ++j) {
      const int vec = j * nt + tid;
      const unsigned lo = __byte_perm((unsigned)x[j].x, (unsigned)x[j].y, 0x0040);
      const unsigned hi = __byte_perm((unsigned)x[j].z, (unsigned)x[j].w, 0x0040);
      if (4 * vec < count) {
        __stcs(dst + vec, __byte_perm(lo, hi, 0x5410));
        outside |= ((unsigned)x[j].x >= uE) | ((unsigned)x[j].y >= uE) | ((unsigned)x[j].z >= uE) |
                   ((unsigned)x[j].w >= uE);
      }
    }
    outside = __syncthreads_or(outside);
    if (tid == 0) p.ws.tile_flag[row * (size_t)p.max_tiles + tile] = outside;
  } else {
    __syncthreads();
  }
  const size_t at = (row * (size_t)p.max_tiles + tile) * E;
  if (!p.ws.tile_cnt16) {
    int32_t* out = p.ws.tile_cnt + at;
    for (int e = tid; e < E; e += nt) out[e] = cnt[e];
  } else if (E % 2 == 0) {   // two 16-bit counts per word (at * 2 bytes is a multiple of 4)
    unsigned* out = reinterpret_cast<unsigned*>(reinterpret_cast<unsigned short*>(p.ws.tile_cnt) + at);
    for (int t = tid; t < E / 2; t += nt) out[t] = (unsigned)cnt[2 * t] | ((unsigned)cnt[2 * t + 1] << 16);
  } else {
    unsigned short* out = reinterpret_cast<unsigned short*>(p.ws.tile_cnt) + at;
    for (int e = tid; e < E; e += nt) out[e] = (unsigned short)cnt[e];
  }
}

// First kernel of the two-kernel chain for small calls: the tile histogram, and the tile's counts
// added straight into the routing-matrix and demand accumulators (see Workspace; paper, "System
// Model", Eq. Omega and Eq. D) -- integer adds, so the sums do not depend on arrival order --
// which replaces the omega kernel.  A lean kernel of its own: on this path the time goes into
// fetching instructions, so it carries no variant it does not run.  One 8192-id tile per block,
// 16 ids per thread; the dependents may become resident from the start.
template <bool VEC>
__global__ void __launch_bounds__(kPlan2TileIds / kIdsPerThread) hist_acc_kernel(const HistParams p) {
  extern __shared__ int cnt[];   // [E + 1]: the last bin collects ignored ids
  __shared__ unsigned call_state[4];   // pair serial, plans with sums in pair 0 / 1, plan-call serial
  const int E = p.d.E;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int nt = blockDim.x, tid = threadIdx.x;
  TL_MIN(p.ws, 0);
  pdl_trigger();
  const int row = b * p.d.R + s, dem_row = b * p.d.M + s / p.d.G;
  const int begin = tile * kPlan2TileIds;
  const int count = min(kPlan2TileIds, p.n_ids - begin);
  const int32_t* ids = p.ids + (size_t)row * p.n_ids + begin;
  int4 x[kIdsPerThread / 4];
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) x[j] = load_ids4(ids, j * nt + tid, count, VEC);
  unsigned checked_in = 0;
  if (tid == 0) {
    // One thread per block reads the bookkeeping words (in flight together with the ids) and
    // then checks in.  The block that checks in last knows that every block has read them, and
    // moves them on at its end: this call's sums go to pair (serial & 1), the other pair gets
    // cleared below, the serial number advances.  Whoever runs after this kernel sees the new
    // values.
    const unsigned ep = __ldcg(p.ws.epoch), d0 = __ldcg(p.ws.epoch + 1), d1 = __ldcg(p.ws.epoch + 2);
    const unsigned sn = __ldcg(p.ws.epoch + 4);
    call_state[0] = ep; call_state[1] = d0; call_state[2] = d1; call_state[3] = sn;
    __threadfence();
    checked_in = atomicAdd(p.ws.epoch + 3, 1u);
  }
#pragma unroll 1
  for (int e = tid; e <= E; e += nt) cnt[e] = 0;
  __syncthreads();
  const unsigned uE = (unsigned)E;
  unsigned mx = 0;
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) {
    const int v[4] = {x[j].x, x[j].y, x[j].z, x[j].w};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      mx = max(mx, (unsigned)(v[u] + 1));
      atomicAdd(&cnt[CK(p.ws.status, (long long)min((unsigned)v[u], uE), E + 1)], 1);   // ids outside [0,E): the spare bin
    }
  }
  if (mx > uE) atomicOr(p.ws.status, TOPOEP_FLAG_BAD_ID);
  __syncthreads();
  // the tile's counts (16 bits each: a tile has fewer than 65536 ids), and the sums
  const unsigned cur = call_state[0] & 1u;
  unsigned short* tc = reinterpret_cast<unsigned short*>(p.ws.tile_cnt) +
                       ((size_t)row * p.max_tiles + tile) * E;
  int32_t* om = p.ws.acc_omega[cur] + (size_t)row * E;
  int32_t* dem = p.ws.acc_demand[cur] + (size_t)dem_row * E;
#pragma unroll 1
  for (int e = tid; e < E; e += nt) {
    const int c = cnt[e];
    tc[e] = (unsigned short)c;
    if (c != 0) { atomicAdd(om + e, c); atomicAdd(dem + e, c); }
  }
  // clear the sums the previous call left in the other pair (nobody reads them any more: this
  // kernel is launched in plain stream order, after everything of the previous call)
  const unsigned dirty = min(cur ? call_state[1] : call_state[2], (unsigned)p.max_batch);
  const size_t n_om = (size_t)dirty * p.d.R * E, n_dem = (size_t)dirty * p.d.M * E;
  const unsigned ctas = gridDim.x * gridDim.y * gridDim.z;
  const unsigned cta = (b * gridDim.y + s) * gridDim.x + tile;
  int32_t* zo = p.ws.acc_omega[cur ^ 1u];
  int32_t* zd = p.ws.acc_demand[cur ^ 1u];
#pragma unroll 1
  for (size_t i = (size_t)cta * nt + tid; i < n_om; i += (size_t)ctas * nt) zo[i] = 0;
#pragma unroll 1
  for (size_t i = (size_t)cta * nt + tid; i < n_dem; i += (size_t)ctas * nt) zd[i] = 0;
  if (tid == 0 && checked_in == ctas - 1u) {
    const unsigned ep = call_state[0];
    p.ws.epoch[3] = 0u;
    p.ws.epoch[1 + (ep & 1u)] = gridDim.z;
    p.ws.epoch[1 + ((ep & 1u) ^ 1u)] = 0u;
    p.ws.epoch[4] = call_state[3] + 1u;
    __threadfence();
    p.ws.epoch[0] = ep + 1u;
  }
  TL_MAX(p.ws, 1);
}

// omega[b][s][e] = sum over the row's tiles (or a routing matrix handed in), written three ways
// for the solver: omega[s][e]; omega_m[main instance of e][s] (transposed, so that the columns a
// solver CTA needs are contiguous rows); and the domain demand D[d][e] = sum over the G ranks of d
// (paper, "System Model", Eq. D).  A warp covers one domain and epw = 32 / Gpad experts: lane =
// g * epw + i holds omega[d*G + g][e0 + i], and a butterfly over the g bits yields D.
__global__ void __launch_bounds__(128) omega_kernel(const OmegaParams p) {
  const int E = p.d.E, G = p.d.G, R = p.d.R, epw = p.epw;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int dm = blockIdx.y, b = blockIdx.z;
  if (p.pdl == 2) pdl_trigger();
  if (p.bump_serial && (blockIdx.x | blockIdx.y | blockIdx.z | threadIdx.x) == 0)
    p.ws.epoch[4] = __ldcg(p.ws.epoch + 4) + 1u;   // one writer; read by the kernel after this one
  const int g = lane / epw, e = (blockIdx.x * 4 + warp) * epw + (lane - g * epw);
  const bool on = g < G && e < E;
  const int s = p.rank_first + dm * G + g;   // global source rank
  const size_t row = (size_t)b * R + s;
  const size_t user_row = (size_t)b * p.rank_count + dm * G + g;   // row in the caller's window
  int sum = 0, mi = 0;
  if (on && p.ws.omega_m)   // row of the transposed copy: static tables, fetched before the wait
    mi = __ldg(p.ws.main_rank + e) * p.d.e_loc + __ldg(p.ws.main_local + e);
  pdl_wait();
  if (on) {
    if (p.src_omega) {
      sum = __ldg(p.src_omega + row * E + e);
    } else {
      const size_t at = row * (size_t)p.max_tiles * E + e;
      const int32_t* c = p.ws.tile_cnt + at;
      const unsigned short* c16 = reinterpret_cast<const unsigned short*>(p.ws.tile_cnt) + at;
      const bool n16 = p.ws.tile_cnt16 != 0;
      for (int t0 = 0; t0 < p.tiles; t0 += 16) {
        int v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u)
          v[u] = t0 + u >= p.tiles ? 0 : n16 ? (int)__ldg(c16 + (size_t)(t0 + u) * E)
                                              : __ldg(c + (size_t)(t0 + u) * E);
#pragma unroll
        for (int u = 0; u < 16; ++u) sum += v[u];
      }
    }
    if (p.ws.omega) p.ws.omega[row * E + e] = sum;
    if (p.out_omega) p.out_omega[user_row * E + e] = sum;
    if (p.ws.omega_m) p.ws.omega_m[((size_t)b * R * p.d.e_loc + mi) * R + s] = sum;
  }
  int dsum = sum;
  for (int o = epw; o < 32; o <<= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
  if (g == 0 && e < E && p.ws.demand) p.ws.demand[((size_t)b * p.d.M + dm) * E + e] = dsum;
}

// The same with 16-byte accesses: a lane holds FOUR consecutive experts of its rank (E % 4 == 0
// and 16-byte aligned rows), so a tile row is read in full sectors and a warp covers
// 4 * epw experts.  Used for calls that fill the GPU.
__global__ void __launch_bounds__(128) omega4_kernel(const OmegaParams p) {
  const int E = p.d.E, G = p.d.G, R = p.d.R, epw = p.epw;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int dm = blockIdx.y, b = blockIdx.z;
  if (p.pdl == 2) pdl_trigger();
  if (p.bump_serial && (blockIdx.x | blockIdx.y | blockIdx.z | threadIdx.x) == 0)
    p.ws.epoch[4] = __ldcg(p.ws.epoch + 4) + 1u;   // one writer; read by the kernel after this one
  const int g = lane / epw, e = 4 * ((blockIdx.x * 4 + warp) * epw + (lane - g * epw));
  const bool on = g < G && e < E;
  const int s = p.rank_first + dm * G + g;   // global source rank
  const size_t row = (size_t)b * R + s;
  const size_t user_row = (size_t)b * p.rank_count + dm * G + g;
  int4 sum = make_int4(0, 0, 0, 0), mr = sum, ml = sum;
  if (on && p.ws.omega_m) {   // static tables, fetched before the wait
    mr = __ldg(reinterpret_cast<const int4*>(p.ws.main_rank + e));
    ml = __ldg(reinterpret_cast<const int4*>(p.ws.main_local + e));
  }
  pdl_wait();
  if (on) {
    if (p.src_omega) {
      sum = __ldg(reinterpret_cast<const int4*>(p.src_omega + row * E + e));
    } else {
      const size_t at = row * (size_t)p.max_tiles * E + e;
      const size_t stride = (size_t)E / 4;
      if (p.ws.tile_cnt16) {   // four 16-bit counts = one 8-byte load
        const uint2* c = reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned short*>(p.ws.tile_cnt) + at);
        for (int t0 = 0; t0 < p.tiles; t0 += 8) {
          uint2 v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            v[u] = t0 + u < p.tiles ? __ldg(c + (size_t)(t0 + u) * stride) : make_uint2(0u, 0u);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            sum.x += (int)(v[u].x & 0xffffu); sum.y += (int)(v[u].x >> 16);
            sum.z += (int)(v[u].y & 0xffffu); sum.w += (int)(v[u].y >> 16);
          }
        }
      } else {
        const int4* c = reinterpret_cast<const int4*>(p.ws.tile_cnt + at);
        for (int t0 = 0; t0 < p.tiles; t0 += 8) {
          int4 v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            v[u] = t0 + u < p.tiles ? __ldg(c + (size_t)(t0 + u) * stride) : make_int4(0, 0, 0, 0);
#pragma unroll
          for (int u = 0; u < 8; ++u) { sum.x += v[u].x; sum.y += v[u].y; sum.z += v[u].z; sum.w += v[u].w; }
        }
      }
    }
    if (p.ws.omega) *reinterpret_cast<int4*>(p.ws.omega + row * E + e) = sum;
    if (p.out_omega) *reinterpret_cast<int4*>(p.out_omega + user_row * E + e) = sum;
    if (p.ws.omega_m) {
      int32_t* om = p.ws.omega_m + (size_t)b * R * p.d.e_loc * R + s;
      om[(size_t)(mr.x * p.d.e_loc + ml.x) * R] = sum.x;
      om[(size_t)(mr.y * p.d.e_loc + ml.y) * R] = sum.y;
      om[(size_t)(mr.z * p.d.e_loc + ml.z) * R] = sum.z;
      om[(size_t)(mr.w * p.d.e_loc + ml.w) * R] = sum.w;
    }
  }
  int4 ds = sum;
  for (int o = epw; o < 32; o <<= 1) {
    ds.x += __shfl_xor_sync(0xffffffffu, ds.x, o);
    ds.y += __shfl_xor_sync(0xffffffffu, ds.y, o);
    ds.z += __shfl_xor_sync(0xffffffffu, ds.z, o);
    ds.w += __shfl_xor_sync(0xffffffffu, ds.w, o);
  }
  if (g == 0 && e < E && p.ws.demand)
    *reinterpret_cast<int4*>(p.ws.demand + ((size_t)b * p.d.M + dm) * E + e) = ds;
}

__global__ void empty_kernel() {}

}  // namespace

size_t hist_smem_bytes(const Dims& d) { return sizeof(int) * ((size_t)d.E + 1); }

cudaError_t launch_hist(const HistParams& p, int batch, int mode, cudaStream_t stream) {
  const dim3 grid(p.tiles, p.rank_count, batch);
  const size_t smem = hist_smem_bytes(p.d);
  const bool wide = p.tile_ids >= 2048;   // 32 ids per thread once the CTA still has 2+ warps
  const dim3 block(p.tile_ids / (wide ? 32 : 16));
  const bool pdl = p.pdl != 0;
  if (p.acc) {   // the lean kernel of the two-kernel chain (plain atomics, its own tile size)
    const dim3 acc_block(kPlan2TileIds / kIdsPerThread);
    return p.vec_ok ? launch_kernel(hist_acc_kernel<true>, grid, acc_block, smem, stream, pdl, p)
                    : launch_kernel(hist_acc_kernel<false>, grid, acc_block, smem, stream, pdl, p);
  }
  if (mode == 1) {
    return wide ? launch_kernel(hist_kernel<1, 32>, grid, block, smem, stream, pdl, p)
                : launch_kernel(hist_kernel<1, 16>, grid, block, smem, stream, pdl, p);
  }
  return wide ? launch_kernel(hist_kernel<0, 32>, grid, block, smem, stream, pdl, p)
              : launch_kernel(hist_kernel<0, 16>, grid, block, smem, stream, pdl, p);
}

cudaError_t launch_omega(const OmegaParams& p, int batch, cudaStream_t stream) {
  auto al16 = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
  // large calls only: with few CTAs the four-times-longer per-thread chain costs latency
  // (one 32-rank plan: 6.7 us -> 8.1 us for histogram + omega; 232 plans: 338 -> 324 us)
  if ((long long)p.d.R * batch >= 2ll * p.d.sms && p.d.E % 4 == 0 && al16(p.src_omega) && al16(p.out_omega) && al16(p.ws.omega) &&
      al16(p.ws.demand) && al16(p.ws.tile_cnt) && al16(p.ws.main_rank) && al16(p.ws.main_local)) {
    const dim3 grid((p.d.E / 4 + 4 * p.epw - 1) / (4 * p.epw), p.d.M, batch);
    return launch_kernel(omega4_kernel, grid, dim3(128), 0, stream, p.pdl != 0, p);
  }
  const dim3 grid((p.d.E + 4 * p.epw - 1) / (4 * p.epw), p.d.M, batch);
  return launch_kernel(omega_kernel, grid, dim3(128), 0, stream, p.pdl != 0, p);
}

cudaError_t launch_empty(int count, cudaStream_t stream) {
  for (int i = 0; i < count; ++i) empty_kernel<<<1, 32, 0, stream>>>();
  return cudaGetLastError();
}

}  // namespace topoep
