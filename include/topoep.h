/*
 * topoep.h -- C boundary of the TopoEP planning step for one GPU (sm_100a).
 *
 * One call, topoep_plan(), turns the router's top-k expert ids of a whole
 * expert-parallel (EP) group into a replica placement x, a token routing q,
 * a per-token physical-instance assignment and the dispatch layout, for a
 * batch of independent (layer, microbatch) plans.  Everything is integer
 * arithmetic; the result is a pure function of (configuration, topk_ids) and
 * is bitwise reproducible across runs and launch configurations.
 *
 * Notation (paper, "System Model"): M NVLink domains (nodes), G GPUs per
 * node, R = M*G EP ranks, E logical experts, N_slot replica slots per rank,
 * k experts per token, T tokens per rank, B plans per call.
 * dom(r) = r / G.  main(e) is the fixed main rank of expert e.
 *
 * Physical instances.  E_loc = max_r |{e : main(e) = r}|, S_phys = E_loc +
 * N_slot, P = R * S_phys.  Instance id p = r * S_phys + l lives on rank r;
 * l < E_loc is the l-th expert (ascending e) whose main rank is r, and
 * l = E_loc + j is replica slot j of rank r.  rank(p) = p / S_phys.
 *
 * Pointers.  Every pointer named dev_* or documented "device" is a device
 * pointer owned by the caller; every other pointer is a host pointer.  The
 * library allocates no device memory: tables and scratch live in a workspace
 * the caller hands over with topoep_set_workspace().  topoep_plan() and the
 * other enqueue calls copy nothing to the host, never synchronise, and only
 * enqueue kernels on the given stream.
 *
 * Errors.  Every int-returning function returns TOPOEP_OK (0) or a negative
 * topoep_status code; nothing aborts or throws.  Conditions only the device
 * can see (an id outside [0,E) other than -1, the refinement cap binding) set
 * bits in a device status word read by topoep_read_status(); the plan stays
 * well defined (invalid ids are ignored and map to -1).
 */
#ifndef TOPOEP_H_
#define TOPOEP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct topoep_ctx* topoep_handle_t;
/* Same type as cudaStream_t; NULL is the legacy default stream. */
typedef struct CUstream_st* topoep_stream_t;

typedef enum {
  TOPOEP_OK = 0,
  TOPOEP_ERR_NULL = -1,        /* a required pointer is NULL                     */
  TOPOEP_ERR_CONFIG = -2,      /* topology / expert / slot numbers out of range  */
  TOPOEP_ERR_MAIN_MAP = -3,    /* main_rank entry outside [0,R), or E % R != 0
                                  with a NULL map                                */
  TOPOEP_ERR_COST = -4,        /* negative byte size or cost coefficient         */
  TOPOEP_ERR_WORKSPACE = -5,   /* workspace missing, too small or misaligned     */
  TOPOEP_ERR_SIZE = -6,        /* tokens_per_rank or batch outside [0, max]      */
  TOPOEP_ERR_ALIGN = -7,       /* an int32 buffer is not 4-byte aligned          */
  TOPOEP_ERR_CUDA = -8,        /* a CUDA runtime call failed (see last error)    */
  TOPOEP_ERR_SMEM = -9,        /* problem does not fit one SM's shared memory    */
  TOPOEP_ERR_ARG = -10,        /* unknown selector / knob / value                */
  TOPOEP_ERR_SCRATCH = -11     /* problem exceeds the library's built-in scratch  */
} topoep_status;

/* Device status bits (topoep_read_status). */
#define TOPOEP_FLAG_BAD_ID      1u  /* some id was outside [0,E) and not -1      */
#define TOPOEP_FLAG_REFINE_CAP  2u  /* refinement stopped by max_refine_iters    */
#define TOPOEP_FLAG_INTERNAL    4u  /* a device-side self check failed           */

/*
 * Cost model (paper, "System Model" and Eq. for b_{d,e}, T_token, T_replica).
 * The communication-time matrix C has two levels: c_intra between ranks of
 * one domain, c_inter between domains, 0 on the diagonal.  All experts share
 * one parameter size.
 */
typedef struct {
  int64_t token_bytes;      /* S_tok: bytes of one routed activation             */
  int64_t expert_bytes;     /* ||W_e||: bytes of one expert's parameters         */
  int32_t c_intra;          /* per-byte time inside a domain, integer units      */
  int32_t c_inter;          /* per-byte time across domains, integer units       */
  int64_t t_ffn;            /* per-assignment compute time; summaries only       */
  int32_t max_refine_iters; /* cap per domain; <= 0 selects 256                  */
  int32_t min_delta;        /* smallest transfer refinement commits; <= 0 -> 1   */
} topoep_cost_params;

/*
 * Derived figures of one plan (paper: objective terms T_comp, T_token,
 * T_replica; max/mean rank-load ratio; inter-node and replica-served
 * fractions of the "Topology-Aware Token Routing" evaluation).  Integers are
 * exact; the three doubles are one IEEE division each of the integers beside
 * them.
 */
typedef struct {
  int64_t assignments;        /* valid (token, expert) pairs = sum_r L_r          */
  int64_t l_max;              /* max_r L_r                                        */
  int64_t cross_assignments;  /* executed in another domain than their source     */
  int64_t replica_served;     /* executed on a rank other than main(e)            */
  int64_t replicas_inter;     /* replicas in a domain other than their main's     */
  int64_t replicas_intra;     /* replicas in their main's domain                  */
  int64_t t_comp;             /* t_ffn * l_max                                    */
  int64_t t_token;            /* 2 * S_tok * sum c(s,r) q(s,e,r)                  */
  int64_t t_replica;          /* sum over replicas c(main(e),r) * ||W||           */
  int64_t cross_token_bytes;  /* 2 * S_tok * cross_assignments (exposed half)     */
  int64_t refine_iters;       /* refinement commits summed over domains           */
  int64_t reserved;
  double  imbalance;          /* l_max * R / assignments  (0 if none)             */
  double  cross_fraction;     /* cross_assignments / assignments                  */
  double  replica_fraction;   /* replica_served / assignments                     */
} topoep_summary_t;

/* Selectors for topoep_debug_tensor (all device int32, laid out as stated). */
enum {
  TOPOEP_T_OMEGA = 0,       /* [max_batch][R][E]   routing matrix Omega           */
  TOPOEP_T_Q = 1,           /* [max_batch][R][P]   q(s, instance)                 */
  TOPOEP_T_RANK_LOAD = 2,   /* [max_batch][R]      L_r                            */
  TOPOEP_T_REFINE_ITERS = 3,/* [max_batch][M]      commits per domain             */
  TOPOEP_T_D = 4,           /* [max_batch][M][E]   domain demand D                */
  TOPOEP_T_U = 5            /* [max_batch][P]      per-instance load U            */
};

/* Knobs for topoep_set_tuning; no knob may change any output bit. */
enum {
  TOPOEP_KNOB_TILE_IDS = 0,     /* ids per histogram / reroute tile: 1024..8192,
                                   power of two                                   */
  TOPOEP_KNOB_HIST_MODE = 1,    /* 0 = plain shared-memory atomics (default),
                                   1 = warp-aggregated (__match_any_sync) atomics */
  TOPOEP_KNOB_PDL = 2,          /* programmatic dependent launch of the kernels after
                                   the histogram.  0: plain stream order; 1 (default):
                                   on, and a call small enough to be resident on the
                                   GPU all at once also lets each kernel start its
                                   dependents early; 2: on, never early; 3: on,
                                   always early                                   */
  TOPOEP_KNOB_TRANSFER_MODE = 3,/* replica transfers: 0 (default) the bulk
                                   asynchronous copy unit through shared memory,
                                   1 plain 16-byte loads and stores               */
  TOPOEP_KNOB_CHAIN = 5,        /* kernels of a topoep_plan call.  1: five (tile
                                   histogram, omega, solver, route tables, reroute);
                                   2: two whenever the tables fit shared memory (a
                                   histogram that also sums the routing matrix, then
                                   one grid of placement, solver, rank and per-token
                                   blocks; a per-token block builds its source's
                                   route table itself and, when inter-node placement
                                   used every slot, does not wait for the solver);
                                   3: four whenever the tables fit (histogram, omega,
                                   the same grid with one route block per source in
                                   place of the per-token blocks, reroute); 0
                                   (default): two for calls small enough to be
                                   resident on the GPU at once, where latency
                                   counts; four for a single plan whose second grid
                                   is resident at once; else five                 */
  TOPOEP_KNOB_PACKED_IDS = 6,   /* five-kernel chain (topoep_plan, or the stage calls
                                   on the same id buffer) with at most 256
                                   experts: the histogram also writes a one-byte
                                   copy of every id into the workspace and the
                                   reroute kernel reads that instead of the 4-byte
                                   ids a second time (a tile that holds padding or
                                   an invalid id is read in full again).  0
                                   (default): when the ids of the call exceed the
                                   L2 cache; 1: never; 2: whenever possible       */
  TOPOEP_KNOB_REROUTE_TILES = 7,/* consecutive tiles of one source a block of the
                                   reroute kernel walks when it reads the one-byte
                                   copy: 1..64, default 2                         */
  TOPOEP_KNOB_TRANSFER_SELFTEST = 4 /* tests only (the one knob that does change
                                   output): 1 makes one block of the bulk engine
                                   wait for a copy it never issued, so its bounded
                                   wait runs out: the transfer sets
                                   TOPOEP_FLAG_INTERNAL, skips that block's chunks
                                   and returns by itself; 0 (default) off         */
};

/*
 * Create a planner for an M x G topology.  (Paper, "System Model": sets D, R,
 * E, dom(), main(), N_slot, C, S_tok, ||W||, t_FFN.)
 *   nodes M in [1,64]; gpus_per_node G in [1,32]; experts E >= 1;
 *   slots_per_rank N_slot >= 0; top_k k >= 1;
 *   max_tokens_per_rank, max_batch >= 1 bound later topoep_plan sizes.
 *   main_rank_host: host array of E ranks, or NULL for the blocked map
 *   main(e) = e / (E / R), which needs E % R == 0.  Copied; not retained.
 *   cost: host struct, copied.
 * Allocates host memory only.  *out is untouched on error.
 */
int topoep_create(topoep_handle_t* out, int nodes, int gpus_per_node, int experts,
                  int slots_per_rank, int top_k, int max_tokens_per_rank,
                  int max_batch, const int32_t* main_rank_host,
                  const topoep_cost_params* cost);

/* Frees host state.  The workspace stays the caller's.  NULL is a no-op. */
void topoep_destroy(topoep_handle_t h);

/* Bytes of device workspace the handle needs (a multiple of 256). 0 if h NULL. */
size_t topoep_workspace_bytes(topoep_handle_t h);

/*
 * Hand over the workspace: dev_ptr is device memory, 256-byte aligned, at
 * least topoep_workspace_bytes(h) long, and stays valid and untouched by the
 * caller until topoep_destroy or the next topoep_set_workspace.  Uploads the
 * constant tables and zeroes the counters on the CURRENT device, then
 * synchronises the device: call it outside stream capture.
 */
int topoep_set_workspace(topoep_handle_t h, void* dev_ptr, size_t bytes);

/*
 * Plan B batches.  (Paper: routing matrix Omega; "Two-Stage GPU-Native
 * Solver": inter-node placement with b_{d,e}, routing construction, loads
 * U and L, intra-node refinement with the half-gap delta; constraints
 * C1-C5; Implementation, "DeepEP dispatch and combine": receive counts are
 * computed on the device from the routing.)
 *
 *   dev_topk_ids        in  [B][R][T][k] int32, expert id per assignment; ids
 *                           outside [0,E) are ignored (-1 is the padding value)
 *   tokens_per_rank     T in [0, max_tokens_per_rank]
 *   batch               B in [0, max_batch]
 *   dev_replica_map     out [B][R][N_slot] expert in replica slot j, -1 if free
 *                           (may be NULL only when N_slot == 0)
 *   dev_token_replica   out [B][R][T][k] physical instance id executing the
 *                           assignment, -1 for an ignored id
 *   dev_dispatch_counts out [B][R][R]   counts[s][r] = assignments of source s
 *                           executed on rank r
 *   dev_dispatch_offsets out [B][2][R][R+1]: [0][s][.] exclusive scan over r of
 *                           counts[s][.] (send offsets; entry R = row total),
 *                           [1][r][.] exclusive scan over s of counts[.][r]
 *                           (receive offsets; entry R = L_r)
 *   dev_instance_counts out [B][P] U: assignments per physical instance, or NULL
 *
 * Within a (plan, source, expert) group, assignments are ranked by flat index
 * t*k+j and dealt to the expert's instances in ascending rank order, each
 * taking q(s,e,r) of them.  Equivalent to topoep_histogram, topoep_solve and
 * topoep_reroute in a row: enqueues five kernels on `stream` (two or four for
 * smaller calls, see TOPOEP_KNOB_CHAIN); capturable in a CUDA graph.  Two plans on one
 * handle must not overlap on the device.  The stage calls below continue from
 * stage calls: topoep_reroute after a topoep_plan returns TOPOEP_ERR_SIZE.
 */
int topoep_plan(topoep_handle_t h, const int32_t* dev_topk_ids, int tokens_per_rank,
                int batch, int32_t* dev_replica_map, int32_t* dev_token_replica,
                int32_t* dev_dispatch_counts, int32_t* dev_dispatch_offsets,
                int32_t* dev_instance_counts, topoep_stream_t stream);

/*
 * Histogram step alone (paper, Eq. Omega): dev_omega [B][R][E] int32 gets the
 * number of assignments of source rank s that select expert e; it may be NULL,
 * the routing matrix is always left in the workspace as well (TOPOEP_T_OMEGA).
 * Uses the workspace for per-tile counts.  Same argument rules as topoep_plan.
 */
int topoep_histogram(topoep_handle_t h, const int32_t* dev_topk_ids, int tokens_per_rank,
                     int batch, int32_t* dev_omega, topoep_stream_t stream);

/*
 * Histogram for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of topoep_histogram, same result.)
 *
 * Who needs it: code that may not call cudaMalloc where it runs -- a plugin
 * living inside another framework's capture region or stream callback, a
 * process whose device pool is sized once and then frozen, a test harness that
 * bans allocation after start-up -- and so cannot supply the workspace that
 * topoep_histogram keeps its per-tile counts in.  Here that scratch is a fixed
 * 8 MiB array built into the library (held by every GPU context that loads the
 * library until the context ends).  No handle, no workspace; the call itself
 * performs no allocation of any kind.
 *
 *   dev_topk_ids  in  [batch][ranks][tokens_per_rank][top_k] int32 (device)
 *   dev_omega     out [batch][ranks][experts] int32 (device)
 *   dev_flags     out optional device uint32: TOPOEP_FLAG_BAD_ID if some id was
 *                     outside [0,experts) and not -1; NULL to ignore
 * Limit: 256 + 4 * batch * ranks * ceil(tokens_per_rank*top_k / 4096) * experts
 * bytes must fit in the 8 MiB array, else TOPOEP_ERR_SCRATCH (nothing is
 * enqueued; there is no fallback).  experts <= 12287.
 *
 * The first call on a device looks up the array's device address (once per
 * device, with that device current); make that first call outside any stream
 * capture.  The address is remembered per device ordinal, that is, for the
 * runtime's primary context: a second (driver-API) context on the same device
 * is not supported.  All calls share the one array, which keeps the previous call's
 * contents: the call clears the only word that must start at zero itself, and
 * two calls that overlap on the GPU (different streams, or graphs replayed
 * concurrently) race on it -- serialise them.
 */
int topoep_histogram_static(const int32_t* dev_topk_ids, int batch, int ranks,
                            int tokens_per_rank, int top_k, int experts,
                            int32_t* dev_omega, uint32_t* dev_flags,
                            topoep_stream_t stream);

/*
 * Solver step alone (paper, "Two-Stage GPU-Native Solver" and the dispatch
 * layout): inter-node placement, routing construction, loads, intra-node
 * refinement, counts and offsets, from a routing matrix.
 *   dev_omega  in  [B][R][E] int32 routing matrix, or NULL to use the one the
 *                  last topoep_histogram / topoep_plan on this handle left in
 *                  the workspace (e.g. rows gathered from other ranks go here)
 * Outputs as in topoep_plan.  Leaves q, U, L and the per-expert instance lists
 * in the workspace for topoep_reroute and topoep_summary.
 */
int topoep_solve(topoep_handle_t h, const int32_t* dev_omega, int batch,
                 int32_t* dev_replica_map, int32_t* dev_dispatch_counts,
                 int32_t* dev_dispatch_offsets, int32_t* dev_instance_counts,
                 topoep_stream_t stream);

/*
 * Per-token assignment step alone (paper, "System Design": token-routing
 * decisions drive dispatch).  Needs, in the workspace, the tile prefixes of a
 * topoep_histogram over the SAME dev_topk_ids, tokens_per_rank and batch, and
 * the routing of a topoep_solve after it.  Returns TOPOEP_ERR_SIZE when
 * tokens_per_rank or batch differ from that histogram call.
 */
int topoep_reroute(topoep_handle_t h, const int32_t* dev_topk_ids, int tokens_per_rank,
                   int batch, int32_t* dev_token_replica, topoep_stream_t stream);

/*
 * Dispatch permutation of the last topoep_plan (the step after the planning
 * path; the paper's "DeepEP dispatch and combine" leaves the buffer layout to
 * its dispatch library, so the layout is defined here):
 *   send buffer of source rank s: its assignments ordered by (physical instance
 *     executing them, flat index t*k+j).  Instance ids ascend with (rank,
 *     instance), so destination r's block is contiguous and starts at
 *     dev_dispatch_offsets[0][s][r].
 *   receive buffer of rank r: the assignments it executes ordered by (instance,
 *     source rank, flat index): every instance's tokens are contiguous, ready for
 *     a grouped GEMM, sources in rank order inside.
 *
 *   dev_token_replica    in  [B][R][T][k] as written by topoep_plan
 *   dev_send_pos         out [B][R][T][k] index in the source's send buffer, -1
 *                            for an ignored id
 *   dev_recv_pos         out [B][R][T][k] index in the destination rank's receive
 *                            buffer, -1 for an ignored id
 *   dev_instance_offsets out [B][R][S_phys+1] start of each instance's segment in
 *                            its rank's receive buffer (entry S_phys = L_r); or NULL
 *   dev_scratch          device memory, 256-byte aligned, at least
 *                            topoep_dispatch_scratch_bytes(h, T, B) long; contents
 *                            need not be kept between calls
 * Works from dev_token_replica alone (nothing of the plan in the workspace is
 * read).  Enqueues four kernels; capturable after its first call.  Off the
 * planning path: the ranking kernel is bound by instruction issue, not by HBM.
 *
 * topoep_dispatch_window is the same for a window of tokens, first_token ..
 * first_token + token_count - 1 of every source rank -- one chunk of the paper's
 * two-chunk pipeline ("Fine-Grained Pipelined Execution": the routed tokens are
 * partitioned into two disjoint chunks that are dispatched one after the other;
 * the paper does not say how they are cut, here a chunk is a range of token
 * indices).  dev_token_replica stays the whole [B][R][T][k] tensor; the chunk has
 * its own send and receive buffers:
 *   dev_send_pos, dev_recv_pos out [B][R][token_count][k] positions inside the
 *                                  chunk's buffers
 *   dev_instance_offsets       out [B][R][S_phys+1] of the chunk, or NULL
 *   dev_counts                 out [B][R][R] assignments of the chunk from source
 *                                  s executed on rank r, or NULL
 *   dev_offsets                out [B][2][R][R+1] the chunk's send / receive
 *                                  offsets (layout of dev_dispatch_offsets), or NULL
 *   dev_scratch                at least topoep_dispatch_scratch_bytes(h,
 *                                  token_count, B) long
 * The counts of disjoint windows that cover all tokens add up to the plan's
 * dev_dispatch_counts.  TOPOEP_ERR_SIZE if the window leaves [0, T].
 */
size_t topoep_dispatch_scratch_bytes(topoep_handle_t h, int tokens_per_rank, int batch);
int topoep_dispatch_window(topoep_handle_t h, const int32_t* dev_token_replica,
                           int tokens_per_rank, int batch, int first_token, int token_count,
                           int32_t* dev_send_pos, int32_t* dev_recv_pos,
                           int32_t* dev_instance_offsets, int32_t* dev_counts,
                           int32_t* dev_offsets, void* dev_scratch, size_t scratch_bytes,
                           topoep_stream_t stream);
int topoep_dispatch_positions(topoep_handle_t h, const int32_t* dev_token_replica,
                              int tokens_per_rank, int batch, int32_t* dev_send_pos,
                              int32_t* dev_recv_pos, int32_t* dev_instance_offsets,
                              void* dev_scratch, size_t scratch_bytes, topoep_stream_t stream);

/*
 * Summaries of the last topoep_plan (paper: objective terms and evaluation
 * ratios, see topoep_summary_t).  dev_out: [batch] topoep_summary_t, 8-byte
 * aligned.  Enqueues one kernel; off the planning path.
 */
int topoep_summary(topoep_handle_t h, int batch, topoep_summary_t* dev_out,
                   topoep_stream_t stream);

/*
 * Copy the device status word to *host_flags and clear it.  Synchronises the
 * stream's device: for tests and health checks, not for the planning path.
 */
int topoep_read_status(topoep_handle_t h, uint32_t* host_flags);

/* Device address and byte size of an intermediate tensor inside the workspace. */
int topoep_debug_tensor(topoep_handle_t h, int which, const void** dev_ptr, size_t* bytes);

/* Change a launch-shape knob; outputs are identical for every legal value. */
int topoep_set_tuning(topoep_handle_t h, int knob, int value);

/*
 * Policy variants (NOT tuning: they change the plan).  The defaults reproduce the paper's
 * procedure as read here.
 *   TOPOEP_POLICY_RESERVE_SLOTS = r (0 <= r <= N_slot, default 0): inter-node placement fills at
 *     most N_slot - r replica slots of a rank, leaving r to the intra-node refinement.  The paper
 *     does not say whether slots are held back; by default none are, and with one slot per rank
 *     the refinement then has nothing to work with (paper, slot-count experiment).
 *   TOPOEP_POLICY_STAGE1_RANK = 0 | 1 (default 0): which rank of a domain takes the next
 *     inter-node candidate.  0: the rank with the fewest used slots (the paper's "least occupied
 *     ranks with free slots", as read here); 1: the rank with a free slot and the smallest
 *     estimated token load (demand on its main instances plus the domain demand of the replicas
 *     it already took), ties to the lowest rank -- the other reading of the same words.  The set
 *     of replicated experts is the same, only their ranks differ.
 * Takes effect from the next topoep_plan / topoep_solve.
 */
enum { TOPOEP_POLICY_RESERVE_SLOTS = 0, TOPOEP_POLICY_STAGE1_RANK = 1 };
int topoep_set_policy(topoep_handle_t h, int policy, int value);

/*
 * Replica parameter executor (paper, "Device-initiated replica transfers", with the three
 * buffers that subsection lists).  Copies driven by the device-resident replica map of ONE plan
 * (dev_replica_map [R][N_slot], e.g. one plan's slice of topoep_plan's output): no host read of
 * the plan, nothing allocated, asynchronous on `stream`, capturable.  Buffers hold all ranks of
 * the simulated group side by side, blocks of param_bytes bytes each (|W|):
 *   dev_main_params [R][E_loc][W]     rank m's main instances by local index l (ascending e);
 *   dev_replica_buf [R][N_slot][W]    rank r's replica slots;
 *   dev_grad_acc    [R][R][E_loc][W]  [main rank][source rank][local index]: the accumulation
 *                                     buffer of each main rank, partitioned by source rank.
 * topoep_replica_pull (forward): for every occupied slot (r, j) with expert e,
 *   replica_buf[r][j] <- main_params[main(e)][l(e)]; empty slots keep their bytes.
 * topoep_replica_grad_return (backward): the slot now holds the replica's gradient;
 *   grad_acc[main(e)][r][l(e)] <- replica_buf[r][j]; every other block keeps its bytes (plain
 *   copy, one writer per block; summing the regions is the main rank's later step).
 * param_bytes must be a multiple of 16 and the two data pointers 16-byte aligned
 * (TOPOEP_ERR_ALIGN); the buffers must not overlap.  A map entry >= E sets TOPOEP_FLAG_BAD_ID
 * and is skipped.  param_bytes == 0 or N_slot == 0: nothing is done, TOPOEP_OK.
 */
int topoep_replica_pull(topoep_handle_t h, const int32_t* dev_replica_map,
                        const void* dev_main_params, void* dev_replica_buf, size_t param_bytes,
                        topoep_stream_t stream);
int topoep_replica_grad_return(topoep_handle_t h, const int32_t* dev_replica_map,
                               const void* dev_replica_buf, void* dev_grad_acc, size_t param_bytes,
                               topoep_stream_t stream);

/*
 * Sharded deployment (paper, "GPU-Native Load Balancer": an EP-group all-gather gives every rank
 * the same routing matrix, and every rank derives the same plan without a coordinator).  A GPU
 * that IS EP rank r holds only its own tokens.  After topoep_set_rank_window(h, first, count):
 *   topoep_histogram  takes dev_topk_ids [B][count][T][k] of source ranks first..first+count-1
 *                     and writes dev_omega [B][count][E] (the rows to all-gather);
 *   topoep_solve      must be given the gathered dev_omega [B][R][E]; it plans the whole group
 *                     (outputs for all R ranks, identical on every rank) and builds the
 *                     routing tables of the window;
 *   topoep_reroute    takes dev_topk_ids / writes dev_token_replica [B][count][T][k].
 * topoep_plan and topoep_dispatch_positions need the full window (0, R) and return
 * TOPOEP_ERR_ARG otherwise.  The default window is (0, R).
 */
int topoep_set_rank_window(topoep_handle_t h, int first_rank, int rank_count);

/*
 * Number of kernels topoep_plan would enqueue for a call of this size with the
 * current knobs: 5, 4 or 2 (see TOPOEP_KNOB_CHAIN).  Needs the
 * workspace (the answer depends on the device).  Negative status on a bad
 * handle or size.  Not part of the method: for benchmarks and tests.
 */
int topoep_plan_kernels(topoep_handle_t h, int tokens_per_rank, int batch);

/*
 * 1 when a topoep_plan call of this size, with the current knobs, leaves a
 * one-byte copy of the ids for its reroute kernel (TOPOEP_KNOB_PACKED_IDS;
 * given 16-byte aligned id and output buffers), else 0.  Needs the workspace
 * (the rule looks at the device's L2 size); negative error code otherwise.
 */
int topoep_plan_byte_copy(topoep_handle_t h, int tokens_per_rank, int batch);

/* Derived sizes: E_loc, S_phys, P.  Any output pointer may be NULL. */
int topoep_get_layout(topoep_handle_t h, int* e_loc, int* s_phys, int* instances);

/*
 * Enqueue `count` empty kernels on the stream: the launch floor a plan's
 * kernel chain is compared against.  Not part of the method.
 */
int topoep_launch_floor(int count, topoep_stream_t stream);

/* Static text for a status code. */
const char* topoep_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* TOPOEP_H_ */
