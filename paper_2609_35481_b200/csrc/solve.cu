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
//
// The kernel is latency-bound (KBs of state; an L2 round trip costs ~0.7 us on B200 and a lone
// warp retires a dependent instruction every ~5 cycles), so:
//  * its inputs arrive by cp.async in one round before the first barrier: the demand D of every
//    domain (summed by omega_kernel), the main-rank tables, and the routing-matrix columns of the
//    domain's main instances, which omega_kernel stored as contiguous rows;
//  * the columns of the replicas chosen in stage 1 are fetched while the main columns are routed;
//  * stage 1 ranks the candidates of a domain all-pairs instead of selecting one maximum at a time.
#include "solve_body.cuh"

namespace topoep {

namespace {

template <bool LPT>
__global__ void __launch_bounds__(kSolveThreads) solve_kernel(const SolveParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  solve_body<LPT>(p, smem, blockIdx.x, blockIdx.y);
}

}  // namespace

size_t solve_smem_bytes(const Dims& d) { return solve_layout(d).total; }

size_t solve_static_bytes(const Dims& d) { return sizeof(int32_t) * solve_static_ints(d); }

void solve_static_fill(const Dims& d, int dm, const int32_t* main_rank, const int32_t* main_local,
                       const int32_t* main_inst_expert, int cost_rank_intra, int32_t* out) {
  const int E = d.E, G = d.G, C = d.C, R = d.R;
  int32_t* mrank = out;
  int32_t* mlocal = mrank + E;
  int32_t* host_lo = mlocal + E;
  int32_t* host_hi = host_lo + E;
  int32_t* col_expert = host_hi + E;
  int32_t* col_cr = col_expert + C;
  short* hostcol = reinterpret_cast<short*>(col_cr + C);
  short* sdom = hostcol + (size_t)G * E;
  short* col_rank = sdom + R;
  for (size_t i = 0; i < solve_static_ints(d); ++i) out[i] = 0;
  for (int e = 0; e < E; ++e) {
    mrank[e] = main_rank[e];
    mlocal[e] = main_local[e];
    const int md = main_rank[e] / G;   // the expert's main domain hosts it from the start
    host_lo[e] = md < 32 ? (int32_t)(1u << md) : 0;
    host_hi[e] = md < 32 ? 0 : (int32_t)(1u << (md - 32));
  }
  for (int i = 0; i < G * E; ++i) hostcol[i] = -1;
  for (int c = 0; c < C; ++c) {
    const int g = c / d.s_phys, l = c - g * d.s_phys;
    const int e = l < d.e_loc ? main_inst_expert[(size_t)(dm * G + g) * d.e_loc + l] : -1;
    col_expert[c] = e;
    col_cr[c] = cost_rank_intra;
    col_rank[c] = (short)g;
    if (e >= 0) hostcol[(size_t)g * E + e] = (short)c;
  }
  for (int s = 0; s < R; ++s) sdom[s] = (short)(s / G);
}

cudaError_t launch_solve(const SolveParams& p, int batch, cudaStream_t stream) {
  const dim3 grid(p.d.M, batch);
  // few CTAs: 512 threads shorten each CTA's phases (33.6 vs 35.1 us per single plan); enough
  // CTAs to fill the GPU twice over: 256 threads fit more CTAs per SM (91 vs 106 us per 232 plans)
  const int threads = (long long)p.d.M * batch >= 2ll * p.d.sms ? 256 : kSolveThreads;
  return p.stage1_lpt ? launch_kernel(solve_kernel<true>, grid, dim3(threads), solve_smem_bytes(p.d),
                                      stream, p.pdl != 0, p)
                      : launch_kernel(solve_kernel<false>, grid, dim3(threads), solve_smem_bytes(p.d),
                                      stream, p.pdl != 0, p);
}

cudaError_t configure_solve(size_t smem) {
  cudaError_t e = cudaFuncSetAttribute(solve_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(solve_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace topoep
