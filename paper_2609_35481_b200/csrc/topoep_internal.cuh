// Internal declarations shared by the TopoEP planning kernels (sm_100a).
//
// Workspace layout, launch-parameter structs and the host-side launch
// functions of the five planning kernels plus the summary kernel.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/topoep.h"

namespace topoep {

constexpr int kIdsPerThread = 16;   // every histogram / reroute thread owns 16 ids of its tile
constexpr int kMinTileIds = 1024;
constexpr int kMaxTileIds = 8192;
constexpr int kSolveThreads = 512;   // at most; large batches launch 256 (more CTAs per SM)
constexpr int kRouteThreads = 256;
constexpr int kSplitCap = 16;       // split experts the reroute kernel ranks per pass

// Problem constants handed to every kernel by value.
struct Dims {
  int M, G, R, E, N, k;
  int e_loc, s_phys, P;
  int C;        // G * s_phys: instance columns of one domain
  int qstride;  // padded row stride of the shared q block (odd, avoids bank conflicts)
  int sms;      // streaming multiprocessors of the device the workspace lives on (launch shapes)
};

// Device pointers into the caller's workspace.
struct Workspace {
  const int32_t* main_rank;         // [E]
  const int32_t* main_local;        // [E] index l of e among the experts of its main rank
  const int32_t* main_inst_expert;  // [R][e_loc] expert of main instance l on rank r, -1 if none
  const int32_t* solve_static;      // [M][solve_static_ints]: per-domain static block of the solver
  // static tables of the two-kernel chain (integer division is dozens of instructions on a path
  // where every instruction counts, so whatever depends only on the handle is tabulated)
  const int32_t* main_dom;          // [E] domain of the main rank
  const int32_t* main_inst;         // [E] instance id of the main instance
  const int32_t* slot_p;            // [M*G*N] instance of the slot the i-th winner of domain dd gets
                                    //   (entry dd*G*N + i: rank i mod G, slot i / G of the domain)
  const int32_t* slot_dd;           // [M*G*N] dd of the entry
  uint32_t* status;                 // [1]
  int32_t* omega;                   // [max_batch][R][E]
  int32_t* omega_m;                 // [max_batch][R*e_loc][R] omega transposed, one row per main
                                    //   instance (row = main_rank(e)*e_loc + main_local(e))
  int32_t* demand;                  // [max_batch][M][E] domain demand D
  int32_t* tile_cnt;                // [max_batch][R][max_tiles][E] per-tile histogram
  int tile_cnt16;                   // 1: the per-tile counts are 16-bit (a tile has < 65536 ids);
                                    //   same indexing, half the bytes.  0: 32-bit (dispatch, static)
  int32_t* tile_pref;               // [max_batch][R][max_tiles][E] exclusive prefix over tiles,
                                    //   column i = i-th split expert of the source
  int32_t* q;                       // [max_batch][R][P]
  int32_t* rank_load;               // [max_batch][R]
  int32_t* refine_iters;            // [max_batch][M]
  int32_t* inst_counts;             // [max_batch][P]
  int32_t* replica_map;             // [max_batch][R][N]
  int32_t* counts;                  // [max_batch][R][R]
  // per (plan, source) routing tables written by the route kernel
  int32_t* route;                   // [max_batch][R][E]  >= 0: the one instance; <= -2: -2 - split index
  int32_t* split_rec;               // [max_batch][R][split_rec_ints(d)]: see SplitRec
  // Two-kernel chain for small calls: the histogram CTAs add their tile counts straight into
  // accumulators (integer adds commute, so the sums do not depend on arrival order).  There are
  // two pairs; a call adds into pair (epoch & 1) and clears what the call before it left in the
  // other pair, so that nothing has to be zeroed between the kernels of one call and a captured
  // graph stays self-contained.  After the histogram kernel one pair holds this call's sums and
  // the other only zeros: readers add the two and need not know which is which.
  int32_t* acc_omega[2];            // [max_batch][R][E] each
  int32_t* acc_demand[2];           // [max_batch][M][E] each
  unsigned* epoch;                  // [0] calls of the accumulating histogram so far (its parity
                                    //   names the pair in use); [1], [2] plans with sums in pair
                                    //   0, 1; [3] histogram blocks that have started; [4] serial
                                    //   number of the running plan call, advanced by the kernel in
                                    //   front of the combined kernel: the tag of records and flags
  unsigned* done_flags;             // [max_batch][M] serial of the last call whose solver block
                                    //   (plan, domain) has finished
  unsigned long long* place_rec;    // [max_batch][M][G*N + 1] inter-node placement of (plan,
                                    //   domain) as published by its placement block: every
                                    //   word = call serial << 32 | value
  unsigned char* ids8;              // [max_batch][R][max ids per row] one-byte copy of the ids of a
                                    //   large topoep_plan call (E <= 256 only, else NULL): the
                                    //   histogram writes it, the reroute kernel reads it instead
                                    //   of the 4-byte ids
  int32_t* tile_flag;               // [max_batch][R][max_tiles] 1: the tile holds an id outside
                                    //   [0, E) (padding or invalid), which one byte cannot tell
                                    //   from a valid id: reroute reads that tile's 4-byte ids
};

// Record of one (plan, source) written by the route kernel, read by the reroute kernel:
//   [0] n_split  [1] n_list  [2..3] zero
//   seg  [E+1]  list i of the source's i-th split expert = [seg[i], seg[i+1])
//   cum  [P]    cumulative quota along each list (instances in ascending rank order)
//   inst [P]    physical instance ids along each list
//   tp   [max_tiles][3][kSplitCap]  per tile, for the first kSplitCap split experts: the tile
//               prefixes (the full table tile_pref is only read when a source has more split
//               experts than that); the tile's RESOLVED instance: when all ids of the expert in
//               this tile fall inside one instance's quota interval, that instance (no ranking
//               needed in this tile), else -1; and the expert ids themselves (-1 beyond n_split)
struct SplitRec {
  int seg, cum, inst, tp, ints;
};
__host__ __device__ inline SplitRec split_rec_layout(int E, int P, int max_tiles) {
  SplitRec r;
  r.seg = 4;
  r.cum = r.seg + ((E + 1 + 3) & ~3);
  r.inst = r.cum + ((P + 3) & ~3);
  r.tp = r.inst + ((P + 3) & ~3);
  r.ints = r.tp + max_tiles * 3 * kSplitCap;
  return r;
}
constexpr int kFastLists = 128;     // list entries the reroute kernel fetches before it knows n_list


struct HistParams {
  Dims d;
  Workspace ws;
  int pdl;   // launched with programmatic dependent launch
  int rank_first, rank_count;   // window of source ranks the caller's id buffers cover
  const int32_t* ids;   // [B][R][n_ids]
  int32_t* out_omega;   // optional caller copy of omega [B][R][E]
  int n_ids;            // ids of a row that are counted (T * k, or the ids of a token window)
  long long row_stride; // ids between the starts of consecutive rows of the buffer
  long long first_id;   // offset of the first counted id inside its row
  int tiles;            // tiles per (plan, rank)
  int max_tiles;        // stride of tile_cnt / tile_pref
  int tile_ids;
  int vec_ok;           // rows are 16-byte aligned and n_ids % 4 == 0
  int acc;              // two-kernel chain: also add the tile counts into the accumulators
  int max_batch;        // plans the accumulators are sized for
  int pack;             // also write the one-byte copy of the ids and the per-tile flag
};

struct OmegaParams {
  Dims d;
  Workspace ws;
  int pdl;   // launched with programmatic dependent launch
  int rank_first, rank_count;   // window of source ranks the caller's id buffers cover
  int bump_serial;            // advance the plan-call serial (this kernel runs in front of the
                              //   combined kernel of the four-kernel chain)
  const int32_t* src_omega;   // given routing matrix [B][R][E], or NULL: sum the tile counts
  int32_t* out_omega;         // optional caller copy of omega [B][R][E]
  int tiles, max_tiles;
  int epw;                    // experts per warp = 32 / (G rounded up to a power of two)
};

struct SolveParams {
  Dims d;
  Workspace ws;
  int pdl;   // launched with programmatic dependent launch
  int max_iters, min_delta;
  int stage1_lpt;     // policy: stage-1 winners go to the least-loaded rank, not round robin
  int stage1_slots;   // slots of a rank that inter-node placement may fill (N minus the reserve)
  int cand_thr;   // demand D of a stage-1 candidate exceeds this: floor(||W|| / (2 S_tok))
  int cost_rank_intra, cost_rank_inter;   // dense ranks of {0, c_intra*W, c_inter*W}
  int32_t* out_replica_map;   // [B][R][N]
  int32_t* out_counts;        // [B][R][R]
  int32_t* out_offsets;       // [B][2][R][R+1]
  int32_t* out_inst_counts;   // [B][P] or NULL
  int acc;            // demand and columns come from the accumulators (two-kernel chain)
  int fused;          // the block runs inside the combined kernel: it returns at once when the
                      //   plan is closed-form, and publishes a flag when it is done
};

// Per-token blocks of the second kernel of the two-kernel chain: per tile, the source's routing
// table (built in the block) and the per-token assignment.
struct TailParams {
  Dims d;
  Workspace ws;
  int pdl;   // launched with programmatic dependent launch
  int stage1_lpt, stage1_slots, cand_thr;   // as in SolveParams
  const int32_t* ids;
  int32_t* out_token_replica;
  int32_t* out_offsets;       // [B][2][R][R+1]: the send half is written here
  int n_ids, tiles, max_tiles, tile_ids;
  int vec_ok;
  int acc;         // row s of the routing matrix comes from the accumulators (two-kernel chain),
                   //   else from the matrix the omega kernel left in the workspace
};

struct RouteParams {
  Dims d;
  Workspace ws;
  int pdl;   // launched with programmatic dependent launch
  int rank_first, rank_count;   // window of source ranks the caller's id buffers cover
  int32_t* out_offsets;       // [B][2][R][R+1]: the send half is written here
  int tiles, max_tiles;       // shape of the tile counts now in the workspace (tiles 0: none)
};

struct RerouteParams {
  Dims d;
  Workspace ws;
  int pdl;   // launched with programmatic dependent launch
  int rank_first, rank_count;   // window of source ranks the caller's id buffers cover
  const int32_t* ids;
  int32_t* out_token_replica;
  int n_ids, tiles, max_tiles, tile_ids;
  int vec_ok;
  int packed;   // read the one-byte copy the histogram of this call left in the workspace
  int tiles_per_block;   // ... in the multi-tile kernel: consecutive tiles of a source per block
};

struct PosParams {
  Dims d;
  Workspace ws;
  const int32_t* token_replica;   // [B][R][n_ids]
  int32_t* out_send_pos;          // [B][R][n_ids]
  int32_t* out_recv_pos;          // [B][R][n_ids]
  int32_t* out_instance_offsets;  // [B][R][S_phys+1] or NULL
  int32_t* pos_cnt;               // scratch [B][R][tiles][P]: tile counts, then prefixes over tiles
  int32_t* pos_a;                 // scratch [B][R][P] send base of (source, instance)
  int32_t* pos_b;                 // scratch [B][R][P] receive base of (source, instance)
  int32_t* pos_tot;               // scratch [B][R][P] assignments of (source, instance) in the window
  int32_t* out_counts;            // [B][R][R] dispatch counts of the window, or NULL
  int32_t* out_offsets;           // [B][2][R][R+1] send / receive offsets of the window, or NULL
  long long row_stride, first_id; // the window inside token_replica's rows (ids)
  uint32_t* scratch_status;       // scratch word for the histogram kernel's flag
  int n_ids, tiles, tile_ids;
};

struct TransferParams {
  Dims d;
  Workspace ws;
  const int32_t* replica_map;   // [R][N] of ONE plan
  const void* src;              // pull: main_params [R][e_loc][W]; return: replica_buf [R][N][W]
  void* dst;                    // pull: replica_buf;  return: grad_acc [R][R][e_loc][W]
  unsigned long long param_bytes;   // W, a multiple of 16
  int selftest;                 // tests only: CTA 0 of the bulk engine runs its give-up path once
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
size_t solve_static_bytes(const Dims& d);   // bytes of one domain's static block
// fills one domain's static block (host memory) from the main-rank tables
void solve_static_fill(const Dims& d, int dm, const int32_t* main_rank, const int32_t* main_local,
                       const int32_t* main_inst_expert, int cost_rank_intra, int32_t* out);
size_t route_smem_bytes(const Dims& d);
size_t reroute_smem_bytes(const Dims& d, int tile_ids);
// second kernel of the two-kernel chain: solver blocks first, per-token blocks after them
constexpr unsigned kFlagWaitLimit = 1u << 20;   // polls (roughly a second) for a record or flag of another block
constexpr int kPlan2TileIds = kSolveThreads * kIdsPerThread;   // one block shape for both roles
size_t plan2_smem_bytes(const Dims& d, int tiles);
long long plan2_blocks(const Dims& d, int tiles, int batch);   // blocks of its grid (two-kernel chain)
cudaError_t configure_plan2(size_t smem);
// route_only: per-source route blocks that write the tables reroute_kernel reads (four-kernel
// chain) in place of the per-token blocks (two-kernel chain)
cudaError_t launch_plan2(const SolveParams& sp, const TailParams& tp, int batch, bool route_only,
                         cudaStream_t stream);
size_t plan2_route_smem_bytes(const Dims& d, int tiles);
size_t pos_rank_smem_bytes(const Dims& d, int tile_ids);
size_t pos_prefix_smem_bytes(const Dims& d);

cudaError_t configure_solve(size_t smem);
cudaError_t configure_route(size_t smem);
cudaError_t configure_reroute(size_t smem);
cudaError_t configure_dispatch(const Dims& d);
cudaError_t launch_hist(const HistParams& p, int batch, int mode, cudaStream_t stream);
cudaError_t launch_omega(const OmegaParams& p, int batch, cudaStream_t stream);
cudaError_t launch_solve(const SolveParams& p, int batch, cudaStream_t stream);
cudaError_t launch_route(const RouteParams& p, int batch, cudaStream_t stream);
cudaError_t launch_reroute(const RerouteParams& p, int batch, cudaStream_t stream);
cudaError_t launch_dispatch(const PosParams& p, int batch, cudaStream_t stream);
cudaError_t launch_summary(const SummaryParams& p, int batch, cudaStream_t stream);
size_t transfer_smem_bytes(const Dims& d, int mode);
cudaError_t configure_transfer(const Dims& d);
// direction 0 = parameter pull, 1 = gradient return; mode 0 = bulk copy unit, 1 = plain loads
cudaError_t launch_transfer(const TransferParams& p, int direction, int mode, int sms,
                            cudaStream_t stream);
cudaError_t launch_empty(int count, cudaStream_t stream);

// Programmatic dependent launch (PDL).  The kernels after the histogram are launched with the
// programmatic-serialization attribute: their blocks may be scheduled as soon as the predecessor's
// blocks have all exited, without waiting for the full kernel boundary, and do whatever does not
// depend on the predecessor -- loading the ids, static tables, clearing shared memory -- before
// pdl_wait(), which returns once the predecessor grid has completed and its writes are visible.
// Every block calls pdl_wait() before its first global write and before it exits, so completion
// stays transitive along the chain.  Whether a kernel also triggers its dependents at its own
// start (pdl == 2) depends on the size of the call: measured on B200, early-resident successor
// blocks take SM resources from the running kernel when the call fills the GPU (a 232-plan call
// went from 1.15 ms to 1.32 ms), so large calls rely on the implicit trigger at block exit
// (pdl == 1, ~1.5 us saved per plan over plain stream order); when the whole chain fits the GPU
// at once (a single plan), the early trigger lets every later kernel finish its prologue --
// static tables, the ids of the reroute tiles -- before its predecessor is done (1-2 us more).
// The histogram never triggers early: the reroute blocks would read the ids at the same time.
// Bounds-checked build (-DTOPOEP_CHECKED; a second library for the tests, never the product):
// CK(status, i, n) wraps an index that is derived from DATA -- an expert id read from a record, an
// instance id, a list position, a work-list entry.  An index outside [0, n) sets
// TOPOEP_FLAG_INTERNAL in the status word and is clamped into range: nothing traps, nothing
// faults, and the tests see the flag.  In the normal build CK is the index itself.
#ifdef TOPOEP_CHECKED
__device__ __forceinline__ int ck_index(uint32_t* status, long long i, long long n) {
  if (i < 0 || i >= n) {
    atomicOr(status, TOPOEP_FLAG_INTERNAL);
    return (int)(i < 0 || n <= 0 ? 0 : n - 1);
  }
  return (int)i;
}
#define CK(status, i, n) ck_index((status), (i), (n))
#else
#define CK(status, i, n) (i)
#endif

// Phase stamps for tuning (compiled out unless TOPOEP_TIMELINE is defined): thread 0 of a block
// folds the global nanosecond timer into slot `slot` of a table behind the status word -- the
// earliest (TL_MIN) or latest (TL_MAX) block to pass the point.  The host reads the table.
#ifdef TOPOEP_TIMELINE
__device__ __forceinline__ unsigned long long tl_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define TL_MIN(ws, slot) do { if (threadIdx.x == 0) atomicMin(reinterpret_cast<unsigned long long*>((ws).status) + 2 + (slot), tl_now()); } while (0)
#define TL_MAX(ws, slot) do { if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned long long*>((ws).status) + 2 + (slot), tl_now()); } while (0)
#else
#define TL_MIN(ws, slot) do { } while (0)
#define TL_MAX(ws, slot) do { } while (0)
#endif

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the dependent kernel's blocks become resident now (they still stop at their pdl_wait()).
__device__ __forceinline__ void pdl_trigger() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Launch `kernel`, allowing it to overlap the tail of the previous kernel in the stream when
// `pdl` is set (the kernel must then follow the protocol above).
template <typename Params>
inline cudaError_t launch_kernel(void (*kernel)(Params), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, bool pdl, const Params& params) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, params);
}

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// Exclusive prefix sum across the lanes of a full warp; *total gets the warp's sum.
__device__ __forceinline__ int warp_exclusive_scan(int v, int lane, int* total) {
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  *total = __shfl_sync(0xffffffffu, inc, 31);
  return inc - v;
}

// Asynchronous global -> shared copies (no register staging); 16-byte form needs both addresses
// 16-byte aligned.  cp_async_wait_all() makes the calling thread's copies visible to itself; a
// __syncthreads() after it makes them visible to the CTA.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

// The 16 ids a thread owns: four groups of four consecutive ids; group j of thread t is vector
// j*blockDim.x + t of the tile, so a warp reads 512 contiguous bytes per group.
__device__ __forceinline__ int4 load_ids4(const int32_t* tile_ids, int vec, int count, bool vec_ok) {
  if (vec_ok) {
    return 4 * vec < count ? __ldg(reinterpret_cast<const int4*>(tile_ids) + vec)
                           : make_int4(-1, -1, -1, -1);
  }
  int4 r;
  const int i = 4 * vec;
  r.x = i + 0 < count ? __ldg(tile_ids + i + 0) : -1;
  r.y = i + 1 < count ? __ldg(tile_ids + i + 1) : -1;
  r.z = i + 2 < count ? __ldg(tile_ids + i + 2) : -1;
  r.w = i + 3 < count ? __ldg(tile_ids + i + 3) : -1;
  return r;
}

}  // namespace topoep
