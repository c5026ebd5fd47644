// Derived figures of a finished plan (paper: objective terms T_comp = t_FFN L_max,
// T_token = 2 S_tok sum c q, T_replica = sum c(main(e),r) ||W|| x; max/mean rank-load ratio;
// inter-node and replica-served assignment fractions).  One CTA per plan; integer sums only
// (commutative, so the shared-memory atomics cannot change a bit), three divisions at the end.
#include "topoep_internal.cuh"

namespace topoep {

namespace {

__global__ void summary_kernel(const SummaryParams p) {
  __shared__ unsigned long long acc[8];
  const Dims d = p.d;
  const int b = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  if (tid < 8) acc[tid] = 0;
  __syncthreads();
  enum { kAssign, kLmax, kCross, kServed, kWeighted, kRepInter, kRepIntra, kRepCost };

  long long cross = 0, served = 0, weighted = 0;
  const int32_t* q = p.ws.q + (size_t)b * d.R * d.P;
  for (int idx = tid; idx < d.R * d.P; idx += nt) {
    const int s = idx / d.P, pi = idx - s * d.P;
    const int r = pi / d.s_phys, l = pi - r * d.s_phys;
    const long long v = q[idx];
    const bool same_dom = s / d.G == r / d.G;
    if (!same_dom) cross += v;
    if (l >= d.e_loc) served += v;
    weighted += v * (s == r ? 0 : (same_dom ? p.c_intra : p.c_inter));
  }
  atomicAdd(&acc[kCross], (unsigned long long)cross);
  atomicAdd(&acc[kServed], (unsigned long long)served);
  atomicAdd(&acc[kWeighted], (unsigned long long)weighted);

  long long total = 0, lmax = 0;
  for (int r = tid; r < d.R; r += nt) {
    const long long v = p.ws.rank_load[(size_t)b * d.R + r];
    total += v;
    lmax = v > lmax ? v : lmax;
  }
  atomicAdd(&acc[kAssign], (unsigned long long)total);
  atomicMax(&acc[kLmax], (unsigned long long)lmax);

  long long rinter = 0, rintra = 0, rcost = 0;
  for (int i = tid; i < d.R * d.N; i += nt) {
    const int e = p.ws.replica_map[(size_t)b * d.R * d.N + i];
    if (e < 0) continue;
    const int r = i / d.N;
    const bool same_dom = p.ws.main_rank[e] / d.G == r / d.G;
    if (same_dom) { rintra += 1; rcost += (long long)p.c_intra * p.expert_bytes; }
    else { rinter += 1; rcost += (long long)p.c_inter * p.expert_bytes; }
  }
  atomicAdd(&acc[kRepInter], (unsigned long long)rinter);
  atomicAdd(&acc[kRepIntra], (unsigned long long)rintra);
  atomicAdd(&acc[kRepCost], (unsigned long long)rcost);
  __syncthreads();

  if (tid == 0) {
    topoep_summary_t o;
    o.assignments = (int64_t)acc[kAssign];
    o.l_max = (int64_t)acc[kLmax];
    o.cross_assignments = (int64_t)acc[kCross];
    o.replica_served = (int64_t)acc[kServed];
    o.replicas_inter = (int64_t)acc[kRepInter];
    o.replicas_intra = (int64_t)acc[kRepIntra];
    o.t_comp = p.t_ffn * o.l_max;
    o.t_token = 2 * p.token_bytes * (int64_t)acc[kWeighted];
    o.t_replica = (int64_t)acc[kRepCost];
    o.cross_token_bytes = 2 * p.token_bytes * o.cross_assignments;
    long long iters = 0;
    for (int dd = 0; dd < d.M; ++dd) iters += p.ws.refine_iters[(size_t)b * d.M + dd];
    o.refine_iters = iters;
    o.reserved = 0;
    o.imbalance = 0.0; o.cross_fraction = 0.0; o.replica_fraction = 0.0;
    if (o.assignments > 0) {
      o.imbalance = (double)(o.l_max * d.R) / (double)o.assignments;
      o.cross_fraction = (double)o.cross_assignments / (double)o.assignments;
      o.replica_fraction = (double)o.replica_served / (double)o.assignments;
    }
    p.out[b] = o;
  }
}

}  // namespace

cudaError_t launch_summary(const SummaryParams& p, int batch, cudaStream_t stream) {
  summary_kernel<<<batch, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace topoep
