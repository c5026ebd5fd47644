// Internal declarations shared by the TopoEP planning kernels (sm_100a).
//
// Workspace layout, launch-parameter structs and the host-side launch
// functions of the three planning kernels plus the summary kernel.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/topoep.h"

namespace topoep {

constexpr int kIdsPerThread = 16;   // every histogram / reroute thread owns 16 ids of its tile
constexpr int kMinTileIds = 1024;
constexpr int kMaxTileIds = 16384;
constexpr int kSolveThreads = 512;

// Problem constants handed to every kernel by value.
struct Dims {
  int M, G, R, E, N, k;
  int e_loc, s_phys, P;
  int C;        // G * s_phys: instance columns of one domain
  int qstride;  // padded row stride of the shared q block (odd, avoids bank conflicts)
};

// Device pointers into the caller's workspace.
struct Workspace {
  const int32_t* main_rank;         // [E]
  const int32_t* main_local;        // [E] index l of e among the experts of its main rank
  const int32_t* main_inst_expert;  // [R][e_loc] expert of main instance l on rank r, -1 if none
  uint32_t* status;                 // [1]
  uint32_t* hist_tickets;           // [max_batch][R], zero between launches
  uint32_t* solve_tickets;          // [max_batch],    zero between launches
  int32_t* omega;                   // [max_batch][R][E]
  int32_t* tile_pref;               // [max_batch][R][max_tiles][E]: counts, then exclusive prefix
  int32_t* q;                       // [max_batch][R][P]
  int32_t* rank_load;               // [max_batch][R]
  int32_t* refine_iters;            // [max_batch][M]
  int32_t* inst_counts;             // [max_batch][P]
  int32_t* replica_map;             // [max_batch][R][N]
  int32_t* counts;                  // [max_batch][R][R]
  int32_t* seg_start;               // [max_batch][E+1] segment of expert e in inst_sorted
  int32_t* inst_sorted;             // [max_batch][P]   instances ordered by (expert, rank)
};

struct HistParams {
  Dims d;
  Workspace ws;
  const int32_t* ids;   // [B][R][n_ids]
  int32_t* out_omega;   // optional caller copy of omega [B][R][E]
  int n_ids;            // T * k
  int tiles;            // tiles per (plan, rank)
  int max_tiles;        // stride of tile_pref
  int tile_ids;
  int vec_ok;           // rows are 16-byte aligned and n_ids % 4 == 0
};

struct SolveParams {
  Dims d;
  Workspace ws;
  int64_t token_bytes, expert_bytes;
  int max_iters, min_delta;
  int cost_rank_intra, cost_rank_inter;   // dense ranks of {0, c_intra*W, c_inter*W}
  int32_t* out_replica_map;   // [B][R][N]
  int32_t* out_counts;        // [B][R][R]
  int32_t* out_offsets;       // [B][2][R][R+1]
  int32_t* out_inst_counts;   // [B][P] or NULL
};

struct RerouteParams {
  Dims d;
  Workspace ws;
  const int32_t* ids;
  int32_t* out_token_replica;
  int n_ids, tiles, max_tiles, tile_ids;
};

struct SummaryParams {
  Dims d;
  Workspace ws;
  int64_t token_bytes, expert_bytes, t_ffn;
  int c_intra, c_inter;
  topoep_summary_t* out;
};

size_t hist_smem_bytes(const Dims& d);
size_t solve_smem_bytes(const Dims& d);
size_t reroute_smem_bytes(const Dims& d, int tile_ids);

cudaError_t configure_solve(size_t smem);
cudaError_t configure_reroute(size_t smem);
cudaError_t launch_hist(const HistParams& p, int batch, int mode, cudaStream_t stream);
cudaError_t launch_solve(const SolveParams& p, int batch, cudaStream_t stream);
cudaError_t launch_reroute(const RerouteParams& p, int batch, cudaStream_t stream);
cudaError_t launch_summary(const SummaryParams& p, int batch, cudaStream_t stream);
cudaError_t launch_empty(int count, cudaStream_t stream);

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

}  // namespace topoep
