// C boundary of the TopoEP planning library: argument checks, workspace carving, kernel
// enqueue.  Nothing here allocates, frees or copies device memory on the planning path; the
// plan call enqueues five kernels (tile histogram, omega, solver, route tables, reroute) on the
// caller's stream.
#include <algorithm>
#include <climits>
#include <new>

#include "topoep_internal.cuh"

using namespace topoep;

struct topoep_ctx {
  Dims d;
  int max_tokens, max_batch;
  topoep_cost_params cost;
  int max_iters, min_delta, cost_rank_intra, cost_rank_inter;
  std::vector<int32_t> main_rank, main_local, main_inst_expert;
  int tile_ids, hist_mode, pdl;
  int stage1_lpt;      // policy: 1 = stage-1 candidates to the least-loaded rank
  int reserve_slots;   // policy: slots per rank left to the refinement by inter-node placement
  int rank_first, rank_count;   // window of source ranks of the histogram / reroute buffers
  size_t dispatch_smem;   // shared memory the dispatch ranking kernel was configured for
  int transfer_ready, transfer_mode, sms;   // replica executor: configured?, copy engine, SM count
  int transfer_selftest;   // tests only: the bulk engine's bounded wait is made to run out once
  int max_tiles;
  int chain;           // knob: 0 choose by size, 1 always five kernels, 2 two kernels when they fit,
                       //   3 four kernels when they fit
  int reroute_tiles_per_block;   // multi-tile reroute kernel: tiles of a source per block
  const int32_t* packed_src;   // ids whose one-byte copy the workspace holds (NULL: none)
  int pack_ids;        // knob: 0 choose by size, 1 never, 2 whenever possible (one-byte id copy)
  int l2_bytes;        // L2 size of the device the workspace lives on
  size_t plan2_smem;   // shared memory the second kernel of the two-kernel chain may use
  bool aux_valid;      // omega_m and demand in the workspace belong to the omega now there
  bool routes_valid;   // route tables in the workspace belong to the tile counts now there
  int hist_tile_ids, hist_tokens, hist_batch;   // shape of the tile prefixes now in the workspace
  // workspace
  bool have_ws;
  Workspace ws;
  size_t off[32];
  size_t ws_bytes;
  cudaError_t last_cuda;
};

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

enum WsSlot {
  W_MAIN_RANK, W_MAIN_LOCAL, W_MAIN_INST, W_SOLVE_STATIC, W_MAIN_DOM, W_MAIN_INSTANCE, W_SLOT_P, W_SLOT_DD, W_STATUS, W_OMEGA, W_OMEGA_M, W_DEMAND, W_TILE_CNT, W_TILE_PREF, W_Q, W_LOAD,
  W_ITERS, W_INST_COUNTS, W_REPLICA_MAP, W_COUNTS, W_ROUTE, W_SPLIT_REC, W_IDS8, W_TILE_FLAG,
  W_ACC_OMEGA0, W_ACC_OMEGA1, W_ACC_DEMAND0, W_ACC_DEMAND1, W_EPOCH, W_DONE, W_PLACE_REC, W_SLOTS
};
static_assert(W_SLOTS <= 32, "offset table size");

void carve(topoep_ctx* h) {
  const Dims& d = h->d;
  const size_t B = (size_t)h->max_batch, R = d.R, E = d.E, P = d.P;
  size_t sz[W_SLOTS];
  sz[W_MAIN_RANK] = 4 * E;
  sz[W_MAIN_LOCAL] = 4 * E;
  sz[W_MAIN_INST] = 4 * R * (size_t)std::max(d.e_loc, 1);
  sz[W_SOLVE_STATIC] = (size_t)d.M * solve_static_bytes(d);
  sz[W_MAIN_DOM] = 4 * E;
  sz[W_MAIN_INSTANCE] = 4 * E;
  sz[W_SLOT_P] = sz[W_SLOT_DD] = 4 * (R * (size_t)d.N + 1);
  sz[W_STATUS] = 4;
  sz[W_OMEGA] = 4 * B * R * E;
  sz[W_OMEGA_M] = 4 * B * R * (size_t)std::max(d.e_loc, 1) * R;
  sz[W_DEMAND] = 4 * B * (size_t)d.M * E;
  sz[W_TILE_CNT] = 4 * B * R * (size_t)h->max_tiles * E;
  sz[W_TILE_PREF] = sz[W_TILE_CNT];
  sz[W_Q] = 4 * B * R * P;
  sz[W_LOAD] = 4 * B * R;
  sz[W_ITERS] = 4 * B * (size_t)d.M;
  sz[W_INST_COUNTS] = 4 * B * P;
  sz[W_REPLICA_MAP] = 4 * B * R * (size_t)std::max(d.N, 1);
  sz[W_COUNTS] = 4 * B * R * R;
  sz[W_ROUTE] = 4 * B * R * E;
  sz[W_SPLIT_REC] = 4 * B * R * (size_t)split_rec_layout(d.E, d.P, h->max_tiles).ints;
  // one byte per id, only where a byte holds an expert id; rows keep the 4-byte rows' alignment / 4
  sz[W_IDS8] = E <= 256 ? B * R * (size_t)h->max_tokens * d.k : 0;
  sz[W_TILE_FLAG] = 4 * B * R * (size_t)h->max_tiles;
  sz[W_ACC_OMEGA0] = sz[W_ACC_OMEGA1] = 4 * B * R * E;
  sz[W_ACC_DEMAND0] = sz[W_ACC_DEMAND1] = 4 * B * (size_t)d.M * E;
  sz[W_EPOCH] = 32;
  sz[W_DONE] = 4 * B * (size_t)d.M;
  sz[W_PLACE_REC] = 8 * B * (size_t)d.M * ((size_t)d.G * d.N + 1);
  size_t at = 0;
  for (int i = 0; i < W_SLOTS; ++i) { h->off[i] = at; at += align_up(sz[i]); }
  h->ws_bytes = at;
}

template <typename T>
T* at(void* base, size_t off) { return reinterpret_cast<T*>(static_cast<char*>(base) + off); }

int check_sizes(topoep_ctx* h, int tokens_per_rank, int batch) {
  if (!h) return TOPOEP_ERR_NULL;
  if (!h->have_ws) return TOPOEP_ERR_WORKSPACE;
  if (tokens_per_rank < 0 || tokens_per_rank > h->max_tokens) return TOPOEP_ERR_SIZE;
  if (batch < 0 || batch > h->max_batch) return TOPOEP_ERR_SIZE;
  return TOPOEP_OK;
}

inline bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }

HistParams make_hist(topoep_ctx* h, const int32_t* ids, int T, int32_t* out_omega) {
  HistParams p;
  p.d = h->d;
  p.ws = h->ws;
  p.ids = ids;
  p.out_omega = out_omega;
  p.n_ids = T * h->d.k;
  p.row_stride = p.n_ids;
  p.first_id = 0;
  p.tile_ids = h->tile_ids;
  p.tiles = std::max(1, (p.n_ids + h->tile_ids - 1) / h->tile_ids);
  p.max_tiles = h->max_tiles;
  p.vec_ok = (p.n_ids % 4 == 0) && ((reinterpret_cast<uintptr_t>(ids) & 15u) == 0);
  // The first kernel of the chain is never launched early: whatever produced the ids (a router
  // kernel, a copy) must be complete before it reads them.
  p.pdl = 0;
  p.rank_first = h->rank_first;
  p.rank_count = h->rank_count;
  p.acc = 0;
  p.pack = 0;
  p.max_batch = h->max_batch;
  return p;
}

// How the kernels after the histogram are launched for a call of `batch` plans: 0 plain stream
// order, 1 programmatic launch with the implicit trigger, 2 also triggering dependents at kernel
// start.  The early trigger pays only while the whole chain fits the GPU at once: at most one
// wave of reroute blocks (eight per SM).
int chain_pdl(const topoep_ctx* h, int batch) {
  if (h->pdl == 0) return 0;
  if (h->pdl == 2) return 1;
  if (h->pdl == 3) return 2;
  long long tiles = 1;
  if (h->hist_tokens >= 0 && h->hist_tile_ids > 0)
    tiles = std::max(1ll, ((long long)h->hist_tokens * h->d.k + h->hist_tile_ids - 1) / h->hist_tile_ids);
  return tiles * h->rank_count * batch <= 8ll * h->d.sms ? 2 : 1;
}

OmegaParams make_omega(topoep_ctx* h, const int32_t* src, int32_t* out_omega, int tiles, int batch) {
  OmegaParams op;
  op.d = h->d;
  op.ws = h->ws;
  op.pdl = chain_pdl(h, batch);
  op.src_omega = src;
  op.out_omega = out_omega;
  op.tiles = tiles;
  op.max_tiles = h->max_tiles;
  int gpad = 1;
  while (gpad < h->d.G) gpad <<= 1;
  op.epw = 32 / gpad;
  op.rank_first = 0;
  op.rank_count = h->d.R;
  op.bump_serial = 0;
  return op;
}

}  // namespace

extern "C" {

int topoep_create(topoep_handle_t* out, int nodes, int gpus_per_node, int experts,
                  int slots_per_rank, int top_k, int max_tokens_per_rank, int max_batch,
                  const int32_t* main_rank_host, const topoep_cost_params* cost) {
  if (!out || !cost) return TOPOEP_ERR_NULL;
  if (nodes < 1 || nodes > 64 || gpus_per_node < 1 || gpus_per_node > 32) return TOPOEP_ERR_CONFIG;
  if (experts < 1 || experts >= (1 << 23) || slots_per_rank < 0 || slots_per_rank > 1024)
    return TOPOEP_ERR_CONFIG;
  if (top_k < 1 || max_tokens_per_rank < 1 || max_batch < 1 || max_batch > 65535)
    return TOPOEP_ERR_CONFIG;
  const long long R = (long long)nodes * gpus_per_node;
  const long long n_ids = (long long)max_tokens_per_rank * top_k;
  // every count the plan derives is at most the R * T * k assignments of one plan (the rank load
  // L_r, the receive offsets and the column sums of the dispatch counts can reach it under
  // skewed routing): it must fit an int32
  if (R * n_ids >= (1ll << 31)) return TOPOEP_ERR_CONFIG;
  if (cost->token_bytes < 0 || cost->expert_bytes < 0 || cost->c_intra < 0 || cost->c_inter < 0 ||
      cost->t_ffn < 0)
    return TOPOEP_ERR_COST;
  if (cost->token_bytes > (1ll << 30) || cost->expert_bytes > (1ll << 60)) return TOPOEP_ERR_COST;
  if (!main_rank_host && experts % R != 0) return TOPOEP_ERR_MAIN_MAP;

  topoep_ctx* h = new (std::nothrow) topoep_ctx();
  if (!h) return TOPOEP_ERR_CONFIG;
  Dims& d = h->d;
  d.M = nodes; d.G = gpus_per_node; d.R = (int)R; d.E = experts; d.N = slots_per_rank; d.k = top_k;
  h->main_rank.resize(experts);
  for (int e = 0; e < experts; ++e) {
    const long long r = main_rank_host ? main_rank_host[e] : e / (experts / R);
    if (r < 0 || r >= R) { delete h; return TOPOEP_ERR_MAIN_MAP; }
    h->main_rank[e] = (int32_t)r;
  }
  std::vector<int> per_rank((size_t)R, 0);
  h->main_local.resize(experts);
  for (int e = 0; e < experts; ++e) h->main_local[e] = per_rank[h->main_rank[e]]++;
  d.e_loc = *std::max_element(per_rank.begin(), per_rank.end());
  d.s_phys = d.e_loc + d.N;
  d.P = d.R * d.s_phys;
  d.C = d.G * d.s_phys;
  d.qstride = d.C | 1;
  d.sms = 0;   // read from the device in topoep_set_workspace
  if (d.s_phys < 1 || (long long)d.C > 32767) { delete h; return TOPOEP_ERR_CONFIG; }
  h->main_inst_expert.assign((size_t)R * std::max(d.e_loc, 1), -1);
  for (int e = 0; e < experts; ++e)
    h->main_inst_expert[(size_t)h->main_rank[e] * d.e_loc + h->main_local[e]] = e;

  h->cost = *cost;
  h->max_iters = cost->max_refine_iters > 0 ? cost->max_refine_iters : 256;
  h->min_delta = cost->min_delta > 0 ? cost->min_delta : 1;
  // Dense ranks of the replica-creation costs {0, c_intra*W, c_inter*W}: W is common, so the
  // coefficients are ranked instead (everything ties at 0 when W == 0).
  {
    const long long ci = cost->expert_bytes > 0 ? cost->c_intra : 0;
    const long long cx = cost->expert_bytes > 0 ? cost->c_inter : 0;
    auto dense_rank = [&](long long c) {
      int r = 0;
      if (0 < c) ++r;
      if (ci < c && ci != 0) ++r;
      if (cx < c && cx != 0 && cx != ci) ++r;
      return r;
    };
    h->cost_rank_intra = dense_rank(ci);
    h->cost_rank_inter = dense_rank(cx);
  }
  h->max_tokens = max_tokens_per_rank;
  h->max_batch = max_batch;
  h->tile_ids = 4096;
  h->chain = 0;
  h->pack_ids = 0;
  h->packed_src = nullptr;
  h->reroute_tiles_per_block = 2;
  h->l2_bytes = 0;
  h->plan2_smem = 0;
  h->aux_valid = false;
  h->routes_valid = false;
  h->hist_mode = 0;
  h->pdl = 1;
  h->reserve_slots = 0;
  h->stage1_lpt = 0;
  h->rank_first = 0;
  h->rank_count = (int)R;
  h->dispatch_smem = 0;
  h->transfer_ready = 0;
  h->transfer_mode = 0;
  h->transfer_selftest = 0;
  h->sms = 0;
  h->max_tiles = (int)std::max(1ll, (n_ids + kMinTileIds - 1) / kMinTileIds);
  h->have_ws = false;
  h->hist_tile_ids = h->hist_tokens = h->hist_batch = -1;
  h->last_cuda = cudaSuccess;
  if (solve_smem_bytes(d) > 227 * 1024 || reroute_smem_bytes(d, kMaxTileIds) > 227 * 1024 ||
      route_smem_bytes(d) > 227 * 1024 ||
      hist_smem_bytes(d) > 48 * 1024) {
    delete h;
    return TOPOEP_ERR_SMEM;
  }
  carve(h);
  *out = h;
  return TOPOEP_OK;
}

void topoep_destroy(topoep_handle_t h) { delete h; }

size_t topoep_workspace_bytes(topoep_handle_t h) { return h ? h->ws_bytes : 0; }

int topoep_set_workspace(topoep_handle_t h, void* dev_ptr, size_t bytes) {
  if (!h || !dev_ptr) return TOPOEP_ERR_NULL;
  if (bytes < h->ws_bytes || (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) != 0)
    return TOPOEP_ERR_WORKSPACE;
  h->have_ws = false;
  Workspace& w = h->ws;
  w.main_rank = at<int32_t>(dev_ptr, h->off[W_MAIN_RANK]);
  w.main_local = at<int32_t>(dev_ptr, h->off[W_MAIN_LOCAL]);
  w.main_inst_expert = at<int32_t>(dev_ptr, h->off[W_MAIN_INST]);
  w.solve_static = at<int32_t>(dev_ptr, h->off[W_SOLVE_STATIC]);
  w.main_dom = at<int32_t>(dev_ptr, h->off[W_MAIN_DOM]);
  w.main_inst = at<int32_t>(dev_ptr, h->off[W_MAIN_INSTANCE]);
  w.slot_p = at<int32_t>(dev_ptr, h->off[W_SLOT_P]);
  w.slot_dd = at<int32_t>(dev_ptr, h->off[W_SLOT_DD]);
  w.status = at<uint32_t>(dev_ptr, h->off[W_STATUS]);
  w.omega = at<int32_t>(dev_ptr, h->off[W_OMEGA]);
  w.omega_m = at<int32_t>(dev_ptr, h->off[W_OMEGA_M]);
  w.demand = at<int32_t>(dev_ptr, h->off[W_DEMAND]);
  w.tile_cnt = at<int32_t>(dev_ptr, h->off[W_TILE_CNT]);
  w.tile_cnt16 = 1;
  w.tile_pref = at<int32_t>(dev_ptr, h->off[W_TILE_PREF]);
  w.q = at<int32_t>(dev_ptr, h->off[W_Q]);
  w.rank_load = at<int32_t>(dev_ptr, h->off[W_LOAD]);
  w.refine_iters = at<int32_t>(dev_ptr, h->off[W_ITERS]);
  w.inst_counts = at<int32_t>(dev_ptr, h->off[W_INST_COUNTS]);
  w.replica_map = at<int32_t>(dev_ptr, h->off[W_REPLICA_MAP]);
  w.counts = at<int32_t>(dev_ptr, h->off[W_COUNTS]);
  w.route = at<int32_t>(dev_ptr, h->off[W_ROUTE]);
  w.split_rec = at<int32_t>(dev_ptr, h->off[W_SPLIT_REC]);
  w.acc_omega[0] = at<int32_t>(dev_ptr, h->off[W_ACC_OMEGA0]);
  w.acc_omega[1] = at<int32_t>(dev_ptr, h->off[W_ACC_OMEGA1]);
  w.acc_demand[0] = at<int32_t>(dev_ptr, h->off[W_ACC_DEMAND0]);
  w.acc_demand[1] = at<int32_t>(dev_ptr, h->off[W_ACC_DEMAND1]);
  w.epoch = at<unsigned>(dev_ptr, h->off[W_EPOCH]);
  w.done_flags = at<unsigned>(dev_ptr, h->off[W_DONE]);
  w.place_rec = at<unsigned long long>(dev_ptr, h->off[W_PLACE_REC]);
  w.ids8 = h->d.E <= 256 ? at<unsigned char>(dev_ptr, h->off[W_IDS8]) : nullptr;
  w.tile_flag = at<int32_t>(dev_ptr, h->off[W_TILE_FLAG]);

  cudaError_t e;
  const size_t E = h->d.E;
  {
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) goto fail;
    if ((e = cudaDeviceGetAttribute(&h->d.sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) goto fail;
    h->sms = h->d.sms;
    if ((e = cudaDeviceGetAttribute(&h->l2_bytes, cudaDevAttrL2CacheSize, dev)) != cudaSuccess) goto fail;
  }
  if ((e = cudaMemcpy(const_cast<int32_t*>(w.main_rank), h->main_rank.data(), 4 * E,
                      cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
  if ((e = cudaMemcpy(const_cast<int32_t*>(w.main_local), h->main_local.data(), 4 * E,
                      cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
  if ((e = cudaMemcpy(const_cast<int32_t*>(w.main_inst_expert), h->main_inst_expert.data(),
                      4 * h->main_inst_expert.size(), cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
  {
    const size_t per = solve_static_bytes(h->d) / sizeof(int32_t);
    std::vector<int32_t> blocks((size_t)h->d.M * per);
    for (int dm = 0; dm < h->d.M; ++dm)
      solve_static_fill(h->d, dm, h->main_rank.data(), h->main_local.data(),
                        h->main_inst_expert.data(), h->cost_rank_intra, blocks.data() + dm * per);
    e = cudaMemcpy(const_cast<int32_t*>(w.solve_static), blocks.data(), 4 * blocks.size(),
                   cudaMemcpyHostToDevice);
    if (e != cudaSuccess) goto fail;
  }
  {
    const Dims& d = h->d;
    const int GN = d.G * d.N;
    std::vector<int32_t> mdom(E), minst(E), sp((size_t)d.M * GN + 1), sd((size_t)d.M * GN + 1);
    for (size_t x = 0; x < E; ++x) {
      mdom[x] = h->main_rank[x] / d.G;
      minst[x] = h->main_rank[x] * d.s_phys + h->main_local[x];
    }
    for (int dd = 0; dd < d.M; ++dd)
      for (int i = 0; i < GN; ++i) {
        sp[(size_t)dd * GN + i] = (dd * d.G + i % d.G) * d.s_phys + d.e_loc + i / d.G;
        sd[(size_t)dd * GN + i] = dd;
      }
    if ((e = cudaMemcpy(const_cast<int32_t*>(w.main_dom), mdom.data(), 4 * E, cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
    if ((e = cudaMemcpy(const_cast<int32_t*>(w.main_inst), minst.data(), 4 * E, cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
    if ((e = cudaMemcpy(const_cast<int32_t*>(w.slot_p), sp.data(), 4 * sp.size(), cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
    if ((e = cudaMemcpy(const_cast<int32_t*>(w.slot_dd), sd.data(), 4 * sd.size(), cudaMemcpyHostToDevice)) != cudaSuccess) goto fail;
  }
  if ((e = cudaMemset(w.status, 0, 4)) != cudaSuccess) goto fail;
  // accumulators, serial number and flags of the two-kernel chain start at zero (each call
  // leaves the accumulators clean for the next)
  if ((e = cudaMemset(w.acc_omega[0], 0, h->ws_bytes - h->off[W_ACC_OMEGA0])) != cudaSuccess) goto fail;
  h->plan2_smem = std::min<size_t>(plan2_smem_bytes(h->d, h->max_tiles), 227 * 1024);
  if ((e = configure_plan2(h->plan2_smem)) != cudaSuccess) goto fail;
  h->aux_valid = false;
  if ((e = configure_solve(solve_smem_bytes(h->d))) != cudaSuccess) goto fail;
  if ((e = configure_route(route_smem_bytes(h->d))) != cudaSuccess) goto fail;
  if ((e = configure_reroute(reroute_smem_bytes(h->d, kMaxTileIds))) != cudaSuccess) goto fail;
  if ((e = cudaDeviceSynchronize()) != cudaSuccess) goto fail;
  h->packed_src = nullptr;   // a new workspace holds no copy of anybody's ids
  h->hist_tile_ids = h->hist_tokens = h->hist_batch = -1;
  h->have_ws = true;
  return TOPOEP_OK;
fail:
  h->last_cuda = e;
  return TOPOEP_ERR_CUDA;
}

namespace {

int enqueue_hist(topoep_ctx* h, const int32_t* ids, int T, int batch, int32_t* out_omega,
                 cudaStream_t stream, bool two = false, bool four = false, bool pack = false) {
  HistParams hp = make_hist(h, ids, T, out_omega);
  if (two) {   // the second kernel of the two-kernel chain has one block shape: its tile size
    hp.tile_ids = kPlan2TileIds;
    hp.tiles = std::max(1, (hp.n_ids + hp.tile_ids - 1) / hp.tile_ids);
  }
  h->hist_tile_ids = hp.tile_ids;
  h->hist_tokens = T;
  h->hist_batch = batch;
  h->routes_valid = false;
  h->aux_valid = !two && h->rank_count == h->d.R;
  hp.acc = two ? 1 : 0;
  hp.pack = pack ? 1 : 0;
  h->packed_src = pack ? ids : nullptr;
  cudaError_t e = launch_hist(hp, batch, h->hist_mode, stream);
  if (e == cudaSuccess && !two) {
    OmegaParams op = make_omega(h, nullptr, out_omega, hp.tiles, batch);
    op.bump_serial = four ? 1 : 0;   // the combined kernel follows: a new serial for its records
    // ... and its blocks (few: the call is a single mid-size plan) may become resident while this
    // small kernel runs, to fetch their static tables
    if (four) op.pdl = h->pdl != 0 ? 2 : 0;
    if (h->rank_count != h->d.R) {
      // a window of ranks: plain tile sums, rank by rank; the demand and the transposed copy need
      // every rank's row and are derived later, from the gathered matrix handed to topoep_solve
      op.d.M = h->rank_count;
      op.d.G = 1;
      op.epw = 32;
      op.ws.omega_m = nullptr;
      op.ws.demand = nullptr;
      op.rank_first = h->rank_first;
      op.rank_count = h->rank_count;
    }
    e = launch_omega(op, batch, stream);
  }
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

// Solver, then the per-source routing tables.  The tile prefixes are (re)built only when the tile
// counts in the workspace belong to this batch size.
SolveParams make_solve(topoep_ctx* h, int batch, int32_t* replica_map, int32_t* counts,
                       int32_t* offsets, int32_t* inst_counts) {
  SolveParams sp;
  sp.d = h->d;
  sp.ws = h->ws;
  sp.pdl = chain_pdl(h, batch);
  sp.acc = 0;
  sp.fused = 0;
  sp.max_iters = h->max_iters;
  sp.min_delta = h->min_delta;
  // 2 D S_tok - ||W|| > 0  <=>  D > floor(||W|| / (2 S_tok)); S_tok = 0 admits no candidate
  {
    const long long st = h->cost.token_bytes, wb = h->cost.expert_bytes;
    const long long thr = st > 0 ? wb / (2 * st) : (long long)INT_MAX;
    sp.cand_thr = (int)std::min<long long>(thr, INT_MAX);
  }
  sp.stage1_slots = std::max(0, h->d.N - h->reserve_slots);
  sp.stage1_lpt = h->stage1_lpt;
  sp.cost_rank_intra = h->cost_rank_intra;
  sp.cost_rank_inter = h->cost_rank_inter;
  sp.out_replica_map = replica_map;
  sp.out_counts = counts;
  sp.out_offsets = offsets;
  sp.out_inst_counts = inst_counts;
  return sp;
}

int enqueue_solve(topoep_ctx* h, const int32_t* omega, int batch, int32_t* replica_map,
                  int32_t* counts, int32_t* offsets, int32_t* inst_counts, cudaStream_t stream) {
  const SolveParams sp = make_solve(h, batch, replica_map, counts, offsets, inst_counts);
  cudaError_t e = cudaSuccess;
  // a routing matrix handed in from outside: derive the demand and the transposed copy from it;
  // likewise when the matrix in the workspace was left by the two-kernel chain, which does not
  // keep those two layouts
  if (omega) e = launch_omega(make_omega(h, omega, nullptr, 0, batch), batch, stream);
  else if (!h->aux_valid)
    e = launch_omega(make_omega(h, h->ws.omega, nullptr, 0, batch), batch, stream);
  h->aux_valid = true;
  if (e == cudaSuccess) e = launch_solve(sp, batch, stream);
  if (e == cudaSuccess) {
    RouteParams rp;
    rp.d = h->d;
    rp.ws = h->ws;
    rp.pdl = chain_pdl(h, batch);
    rp.rank_first = h->rank_first;
    rp.rank_count = h->rank_count;
    rp.out_offsets = offsets;
    rp.max_tiles = h->max_tiles;
    rp.tiles = 0;
    if (h->hist_batch == batch && h->hist_tokens >= 0) {
      const int n_ids = h->hist_tokens * h->d.k;
      rp.tiles = std::max(1, (n_ids + h->hist_tile_ids - 1) / h->hist_tile_ids);
    }
    e = launch_route(rp, batch, stream);
    h->routes_valid = rp.tiles > 0;
  }
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

int enqueue_reroute(topoep_ctx* h, const int32_t* ids, int T, int batch, int32_t* token_replica,
                    cudaStream_t stream, bool packed = false) {
  if (T == 0) return TOPOEP_OK;
  RerouteParams rp;
  rp.d = h->d;
  rp.ws = h->ws;
  rp.pdl = chain_pdl(h, batch) != 0;
  rp.rank_first = h->rank_first;
  rp.rank_count = h->rank_count;
  rp.ids = ids;
  rp.out_token_replica = token_replica;
  rp.n_ids = T * h->d.k;
  rp.tile_ids = h->hist_tile_ids;
  rp.tiles = std::max(1, (rp.n_ids + rp.tile_ids - 1) / rp.tile_ids);
  rp.max_tiles = h->max_tiles;
  rp.vec_ok = (rp.n_ids % 4 == 0) && ((reinterpret_cast<uintptr_t>(ids) & 15u) == 0) &&
              ((reinterpret_cast<uintptr_t>(token_replica) & 15u) == 0);
  rp.packed = packed && rp.vec_ok ? 1 : 0;
  rp.tiles_per_block = std::max(1, std::min(rp.tiles, h->reroute_tiles_per_block));
  const cudaError_t e = launch_reroute(rp, batch, stream);
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

// Five-kernel chain (topoep_plan, or topoep_histogram ... topoep_reroute): should the histogram
// leave a one-byte copy of the ids for the reroute kernel?  It trades 1 byte written + 1 byte read per assignment for the second
// 4-byte read, which pays once the ids no longer survive in L2 between the two kernels.  Needs
// E <= 256, 16-byte aligned buffers and whole groups of four ids per row.
bool use_packed_ids(const topoep_ctx* h, const int32_t* ids, int T, int batch) {
  if (h->pack_ids == 1 || !h->ws.ids8 || T == 0 || h->rank_count != h->d.R) return false;
  const long long n_ids = (long long)T * h->d.k;
  if (n_ids % 4 != 0 || (reinterpret_cast<uintptr_t>(ids) & 15u)) return false;
  if (h->pack_ids == 2) return true;
  return 4ll * n_ids * h->d.R * batch > (long long)h->l2_bytes;
}

// The combined kernel: placement, solver and rank blocks in one grid, and either the per-token
// blocks (two-kernel chain: the accumulating histogram in front) or one route block per source
// (four-kernel chain: histogram and omega kernels in front, reroute kernel behind).
int enqueue_plan2(topoep_ctx* h, const int32_t* ids, int T, int batch, int32_t* replica_map,
                  int32_t* token_replica, int32_t* counts, int32_t* offsets, int32_t* inst_counts,
                  bool route_only, cudaStream_t stream) {
  SolveParams sp = make_solve(h, batch, replica_map, counts, offsets, inst_counts);
  sp.pdl = h->pdl != 0;
  sp.acc = route_only ? 0 : 1;
  sp.fused = 1;
  TailParams tp;
  tp.d = h->d;
  tp.ws = h->ws;
  tp.pdl = h->pdl != 0;
  tp.acc = sp.acc;
  tp.stage1_lpt = sp.stage1_lpt;
  tp.stage1_slots = sp.stage1_slots;
  tp.cand_thr = sp.cand_thr;
  tp.ids = ids;
  tp.out_token_replica = token_replica;
  tp.out_offsets = offsets;
  tp.n_ids = T * h->d.k;
  tp.tile_ids = h->hist_tile_ids;
  tp.tiles = std::max(1, (tp.n_ids + tp.tile_ids - 1) / tp.tile_ids);
  tp.max_tiles = h->max_tiles;
  tp.vec_ok = (tp.n_ids % 4 == 0) && ((reinterpret_cast<uintptr_t>(ids) & 15u) == 0) &&
              ((reinterpret_cast<uintptr_t>(token_replica) & 15u) == 0);
  const cudaError_t e = launch_plan2(sp, tp, batch, route_only, stream);
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  if (route_only) h->routes_valid = true;
  return TOPOEP_OK;
}

// Which chain plans this call: two kernels when the per-token blocks' tables fit their shared
// memory and (unless forced) the whole call is resident on the GPU at once.
bool use_two_kernels(const topoep_ctx* h, int T, int batch) {
  if (h->chain == 1 || h->chain == 3 || T <= 0 || h->rank_count != h->d.R) return false;
  const long long n_ids = (long long)T * h->d.k;
  const long long tiles = std::max(1ll, (n_ids + kPlan2TileIds - 1) / kPlan2TileIds);
  if (tiles > h->max_tiles) return false;
  const size_t smem = plan2_smem_bytes(h->d, (int)tiles);
  if (smem > h->plan2_smem) return false;
  if (h->chain == 2) return true;
  const long long per_sm = std::max<long long>(1, std::min<long long>(2, (227 * 1024) / (long long)smem));
  return plan2_blocks(h->d, (int)tiles, batch) <= per_sm * h->d.sms;
}

// Four kernels (histogram, omega, the combined kernel with route blocks, reroute) for the other
// calls, when the route blocks' tables fit shared memory.
bool use_four_kernels(const topoep_ctx* h, int T, int batch) {
  if (h->chain == 1 || h->chain == 2 || T <= 0 || h->rank_count != h->d.R) return false;
  const long long n_ids = (long long)T * h->d.k;
  const long long tiles = std::max(1ll, (n_ids + h->tile_ids - 1) / h->tile_ids);
  if (plan2_route_smem_bytes(h->d, (int)tiles) > h->plan2_smem) return false;
  if (h->chain == 3) return true;
  // by size: only while the combined kernel's grid is resident at once (a single mid-size plan:
  // 62 against 69 us at 128 ranks); with hundreds of plans its blocks cost more than the solver
  // and route kernels they replace (1142 against 926 us for 232 plans)
  return (2ll * h->d.M + 2ll * h->d.R) * batch <= 2ll * h->d.sms;
}

}  // namespace

int topoep_histogram(topoep_handle_t h, const int32_t* dev_topk_ids, int tokens_per_rank,
                     int batch, int32_t* dev_omega, topoep_stream_t stream) {
  int rc = check_sizes(h, tokens_per_rank, batch);
  if (rc != TOPOEP_OK) return rc;
  if (batch == 0) return TOPOEP_OK;
  if (!dev_topk_ids && tokens_per_rank > 0) return TOPOEP_ERR_NULL;
  if (!aligned4(dev_topk_ids) || !aligned4(dev_omega)) return TOPOEP_ERR_ALIGN;
  const bool pack = use_packed_ids(h, dev_topk_ids, tokens_per_rank, batch);
  return enqueue_hist(h, dev_topk_ids, tokens_per_rank, batch, dev_omega, stream, false, false, pack);
}

int topoep_solve(topoep_handle_t h, const int32_t* dev_omega, int batch, int32_t* dev_replica_map,
                 int32_t* dev_dispatch_counts, int32_t* dev_dispatch_offsets,
                 int32_t* dev_instance_counts, topoep_stream_t stream) {
  int rc = check_sizes(h, 0, batch);
  if (rc != TOPOEP_OK) return rc;
  if (batch == 0) return TOPOEP_OK;
  if (!dev_dispatch_counts || !dev_dispatch_offsets) return TOPOEP_ERR_NULL;
  if (h->d.N > 0 && !dev_replica_map) return TOPOEP_ERR_NULL;
  if (!aligned4(dev_omega) || !aligned4(dev_replica_map) || !aligned4(dev_dispatch_counts) ||
      !aligned4(dev_dispatch_offsets) || !aligned4(dev_instance_counts))
    return TOPOEP_ERR_ALIGN;
  // with a window of ranks the workspace holds only the window's rows: the gathered matrix is required
  if (h->rank_count != h->d.R && !dev_omega) return TOPOEP_ERR_NULL;
  return enqueue_solve(h, dev_omega, batch, dev_replica_map, dev_dispatch_counts,
                       dev_dispatch_offsets, dev_instance_counts, stream);
}

int topoep_reroute(topoep_handle_t h, const int32_t* dev_topk_ids, int tokens_per_rank, int batch,
                   int32_t* dev_token_replica, topoep_stream_t stream) {
  int rc = check_sizes(h, tokens_per_rank, batch);
  if (rc != TOPOEP_OK) return rc;
  if (batch == 0) return TOPOEP_OK;
  if (tokens_per_rank != h->hist_tokens || batch != h->hist_batch || !h->routes_valid)
    return TOPOEP_ERR_SIZE;
  if (tokens_per_rank > 0 && (!dev_topk_ids || !dev_token_replica)) return TOPOEP_ERR_NULL;
  if (!aligned4(dev_topk_ids) || !aligned4(dev_token_replica)) return TOPOEP_ERR_ALIGN;
  // the one-byte copy the histogram call left, if it was made from these very ids
  const bool packed = h->packed_src != nullptr && h->packed_src == dev_topk_ids;
  return enqueue_reroute(h, dev_topk_ids, tokens_per_rank, batch, dev_token_replica, stream, packed);
}

int topoep_plan(topoep_handle_t h, const int32_t* dev_topk_ids, int tokens_per_rank, int batch,
                int32_t* dev_replica_map, int32_t* dev_token_replica, int32_t* dev_dispatch_counts,
                int32_t* dev_dispatch_offsets, int32_t* dev_instance_counts,
                topoep_stream_t stream) {
  int rc = check_sizes(h, tokens_per_rank, batch);
  if (rc != TOPOEP_OK) return rc;
  if (batch == 0) return TOPOEP_OK;
  if (!dev_dispatch_counts || !dev_dispatch_offsets) return TOPOEP_ERR_NULL;
  if (h->d.N > 0 && !dev_replica_map) return TOPOEP_ERR_NULL;
  if (tokens_per_rank > 0 && (!dev_topk_ids || !dev_token_replica)) return TOPOEP_ERR_NULL;
  if (!aligned4(dev_topk_ids) || !aligned4(dev_replica_map) || !aligned4(dev_token_replica) ||
      !aligned4(dev_dispatch_counts) || !aligned4(dev_dispatch_offsets) ||
      !aligned4(dev_instance_counts))
    return TOPOEP_ERR_ALIGN;
  if (h->rank_count != h->d.R) return TOPOEP_ERR_ARG;   // a whole plan needs every rank's ids
  if (use_two_kernels(h, tokens_per_rank, batch)) {
    rc = enqueue_hist(h, dev_topk_ids, tokens_per_rank, batch, nullptr, stream, true);
    if (rc != TOPOEP_OK) return rc;
    return enqueue_plan2(h, dev_topk_ids, tokens_per_rank, batch, dev_replica_map, dev_token_replica,
                         dev_dispatch_counts, dev_dispatch_offsets, dev_instance_counts, false, stream);
  }
  if (use_four_kernels(h, tokens_per_rank, batch)) {
    rc = enqueue_hist(h, dev_topk_ids, tokens_per_rank, batch, nullptr, stream, false, true);
    if (rc != TOPOEP_OK) return rc;
    rc = enqueue_plan2(h, dev_topk_ids, tokens_per_rank, batch, dev_replica_map, dev_token_replica,
                       dev_dispatch_counts, dev_dispatch_offsets, dev_instance_counts, true, stream);
    if (rc != TOPOEP_OK) return rc;
    return enqueue_reroute(h, dev_topk_ids, tokens_per_rank, batch, dev_token_replica, stream);
  }
  const bool pack = use_packed_ids(h, dev_topk_ids, tokens_per_rank, batch);
  rc = enqueue_hist(h, dev_topk_ids, tokens_per_rank, batch, nullptr, stream, false, false, pack);
  if (rc != TOPOEP_OK) return rc;
  rc = enqueue_solve(h, nullptr, batch, dev_replica_map, dev_dispatch_counts, dev_dispatch_offsets,
                     dev_instance_counts, stream);
  if (rc != TOPOEP_OK) return rc;
  return enqueue_reroute(h, dev_topk_ids, tokens_per_rank, batch, dev_token_replica, stream, pack);
}

size_t topoep_dispatch_scratch_bytes(topoep_handle_t h, int tokens_per_rank, int batch) {
  if (!h || tokens_per_rank < 0 || batch < 0) return 0;
  const size_t n_ids = (size_t)tokens_per_rank * h->d.k;
  const size_t tiles = std::max<size_t>(1, (n_ids + h->tile_ids - 1) / h->tile_ids);
  const size_t rows = (size_t)batch * h->d.R;
  return kAlign + align_up(4 * rows * h->d.P) * 3 + align_up(4 * rows * tiles * h->d.P);
}

int topoep_dispatch_window(topoep_handle_t h, const int32_t* dev_token_replica,
                           int tokens_per_rank, int batch, int first_token, int token_count,
                           int32_t* dev_send_pos, int32_t* dev_recv_pos,
                           int32_t* dev_instance_offsets, int32_t* dev_counts,
                           int32_t* dev_offsets, void* dev_scratch, size_t scratch_bytes,
                           topoep_stream_t stream) {
  int rc = check_sizes(h, tokens_per_rank, batch);
  if (rc != TOPOEP_OK) return rc;
  if (first_token < 0 || token_count < 0 || first_token > tokens_per_rank - token_count)
    return TOPOEP_ERR_SIZE;
  if (batch == 0) return TOPOEP_OK;
  if (!dev_scratch) return TOPOEP_ERR_NULL;
  if (h->rank_count != h->d.R) return TOPOEP_ERR_ARG;   // needs every rank's assignments
  if (token_count > 0 && (!dev_token_replica || !dev_send_pos || !dev_recv_pos))
    return TOPOEP_ERR_NULL;
  if (!aligned4(dev_token_replica) || !aligned4(dev_send_pos) || !aligned4(dev_recv_pos) ||
      !aligned4(dev_instance_offsets) || !aligned4(dev_counts) || !aligned4(dev_offsets))
    return TOPOEP_ERR_ALIGN;
  if (scratch_bytes < topoep_dispatch_scratch_bytes(h, token_count, batch) ||
      (reinterpret_cast<uintptr_t>(dev_scratch) % kAlign) != 0)
    return TOPOEP_ERR_WORKSPACE;
  if (((size_t)h->d.P + 1) * sizeof(int) > 48 * 1024 ||
      pos_rank_smem_bytes(h->d, h->tile_ids) > 227 * 1024 ||
      pos_prefix_smem_bytes(h->d) > 227 * 1024)
    return TOPOEP_ERR_SMEM;
  PosParams p;
  p.d = h->d;
  p.ws = h->ws;
  p.token_replica = dev_token_replica;
  p.out_send_pos = dev_send_pos;
  p.out_recv_pos = dev_recv_pos;
  p.out_instance_offsets = dev_instance_offsets;
  p.out_counts = dev_counts;
  p.out_offsets = dev_offsets;
  p.n_ids = token_count * h->d.k;
  p.row_stride = (long long)tokens_per_rank * h->d.k;
  p.first_id = (long long)first_token * h->d.k;
  p.tile_ids = h->tile_ids;
  p.tiles = std::max(1, (p.n_ids + p.tile_ids - 1) / p.tile_ids);
  const size_t rows = (size_t)batch * h->d.R;
  const size_t per = align_up(4 * rows * h->d.P);
  char* base = static_cast<char*>(dev_scratch);
  p.scratch_status = reinterpret_cast<uint32_t*>(base);
  p.pos_a = reinterpret_cast<int32_t*>(base + kAlign);
  p.pos_b = reinterpret_cast<int32_t*>(base + kAlign + per);
  p.pos_tot = reinterpret_cast<int32_t*>(base + kAlign + 2 * per);
  p.pos_cnt = reinterpret_cast<int32_t*>(base + kAlign + 3 * per);
  cudaError_t e = cudaSuccess;
  if (!h->dispatch_smem) {
    // first use: opt in to the shared memory the kernels need (host-side attribute only)
    e = configure_dispatch(h->d);
    if (e == cudaSuccess) h->dispatch_smem = 1;
  }
  if (e == cudaSuccess) e = launch_dispatch(p, batch, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

int topoep_dispatch_positions(topoep_handle_t h, const int32_t* dev_token_replica,
                              int tokens_per_rank, int batch, int32_t* dev_send_pos,
                              int32_t* dev_recv_pos, int32_t* dev_instance_offsets,
                              void* dev_scratch, size_t scratch_bytes, topoep_stream_t stream) {
  return topoep_dispatch_window(h, dev_token_replica, tokens_per_rank, batch, 0, tokens_per_rank,
                                dev_send_pos, dev_recv_pos, dev_instance_offsets, nullptr, nullptr,
                                dev_scratch, scratch_bytes, stream);
}

namespace {

// Shared body of the two replica transfers.
int enqueue_transfer(topoep_handle_t h, int direction, const int32_t* dev_replica_map,
                     const void* src, void* dst, size_t param_bytes, cudaStream_t stream) {
  if (!h) return TOPOEP_ERR_NULL;
  if (!h->have_ws) return TOPOEP_ERR_WORKSPACE;
  if (h->d.N == 0 || param_bytes == 0) return TOPOEP_OK;   // no slots or nothing to move
  if (!dev_replica_map || !src || !dst) return TOPOEP_ERR_NULL;
  if (!aligned4(dev_replica_map) || (reinterpret_cast<uintptr_t>(src) & 15u) ||
      (reinterpret_cast<uintptr_t>(dst) & 15u) || (param_bytes & 15u))
    return TOPOEP_ERR_ALIGN;
  // block indices are 32-bit: [R][R][e_loc] blocks in the largest buffer
  if ((unsigned long long)h->d.R * h->d.R * h->d.e_loc >= (1ull << 32)) return TOPOEP_ERR_SIZE;
  if (transfer_smem_bytes(h->d, h->transfer_mode) > 113 * 1024) return TOPOEP_ERR_SMEM;
  cudaError_t e = cudaSuccess;
  if (!h->transfer_ready) {
    // first use: host-side attributes only (shared-memory opt-in)
    e = configure_transfer(h->d);
    if (e == cudaSuccess) h->transfer_ready = 1;
  }
  if (e == cudaSuccess) {
    TransferParams p;
    p.d = h->d;
    p.ws = h->ws;
    p.replica_map = dev_replica_map;
    p.src = src;
    p.dst = dst;
    p.param_bytes = param_bytes;
    p.selftest = h->transfer_selftest;
    e = launch_transfer(p, direction, h->transfer_mode, h->sms, stream);
  }
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

}  // namespace

int topoep_replica_pull(topoep_handle_t h, const int32_t* dev_replica_map,
                        const void* dev_main_params, void* dev_replica_buf, size_t param_bytes,
                        topoep_stream_t stream) {
  return enqueue_transfer(h, 0, dev_replica_map, dev_main_params, dev_replica_buf, param_bytes,
                          static_cast<cudaStream_t>(stream));
}

int topoep_replica_grad_return(topoep_handle_t h, const int32_t* dev_replica_map,
                               const void* dev_replica_buf, void* dev_grad_acc, size_t param_bytes,
                               topoep_stream_t stream) {
  return enqueue_transfer(h, 1, dev_replica_map, dev_replica_buf, dev_grad_acc, param_bytes,
                          static_cast<cudaStream_t>(stream));
}

int topoep_summary(topoep_handle_t h, int batch, topoep_summary_t* dev_out, topoep_stream_t stream) {
  if (!h) return TOPOEP_ERR_NULL;
  if (!h->have_ws) return TOPOEP_ERR_WORKSPACE;
  if (batch < 0 || batch > h->max_batch) return TOPOEP_ERR_SIZE;
  if (batch == 0) return TOPOEP_OK;
  if (!dev_out) return TOPOEP_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(dev_out) & 7u) return TOPOEP_ERR_ALIGN;
  SummaryParams p;
  p.d = h->d;
  p.ws = h->ws;
  p.token_bytes = h->cost.token_bytes;
  p.expert_bytes = h->cost.expert_bytes;
  p.t_ffn = h->cost.t_ffn;
  p.c_intra = h->cost.c_intra;
  p.c_inter = h->cost.c_inter;
  p.out = dev_out;
  cudaError_t e = launch_summary(p, batch, stream);
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

int topoep_read_status(topoep_handle_t h, uint32_t* host_flags) {
  if (!h || !host_flags) return TOPOEP_ERR_NULL;
  if (!h->have_ws) return TOPOEP_ERR_WORKSPACE;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(host_flags, h->ws.status, 4, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemset(h->ws.status, 0, 4);
  if (e != cudaSuccess) { h->last_cuda = e; return TOPOEP_ERR_CUDA; }
  return TOPOEP_OK;
}

int topoep_debug_tensor(topoep_handle_t h, int which, const void** dev_ptr, size_t* bytes) {
  if (!h || !dev_ptr || !bytes) return TOPOEP_ERR_NULL;
  if (!h->have_ws) return TOPOEP_ERR_WORKSPACE;
  const Dims& d = h->d;
  const size_t B = (size_t)h->max_batch;
  switch (which) {
    case TOPOEP_T_OMEGA: *dev_ptr = h->ws.omega; *bytes = 4 * B * d.R * d.E; break;
    case TOPOEP_T_Q: *dev_ptr = h->ws.q; *bytes = 4 * B * d.R * d.P; break;
    case TOPOEP_T_RANK_LOAD: *dev_ptr = h->ws.rank_load; *bytes = 4 * B * d.R; break;
    case TOPOEP_T_REFINE_ITERS: *dev_ptr = h->ws.refine_iters; *bytes = 4 * B * d.M; break;
    case TOPOEP_T_D: *dev_ptr = h->ws.demand; *bytes = 4 * B * d.M * d.E; break;
    case TOPOEP_T_U: *dev_ptr = h->ws.inst_counts; *bytes = 4 * B * d.P; break;
    default: return TOPOEP_ERR_ARG;
  }
  return TOPOEP_OK;
}

int topoep_set_tuning(topoep_handle_t h, int knob, int value) {
  if (!h) return TOPOEP_ERR_NULL;
  switch (knob) {
    case TOPOEP_KNOB_TILE_IDS:
      if (value < kMinTileIds || value > kMaxTileIds || (value & (value - 1))) return TOPOEP_ERR_ARG;
      h->tile_ids = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_HIST_MODE:
      if (value != 0 && value != 1) return TOPOEP_ERR_ARG;
      h->hist_mode = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_PDL:
      if (value < 0 || value > 3) return TOPOEP_ERR_ARG;
      h->pdl = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_TRANSFER_MODE:
      if (value != 0 && value != 1) return TOPOEP_ERR_ARG;
      h->transfer_mode = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_CHAIN:
      if (value < 0 || value > 3) return TOPOEP_ERR_ARG;
      h->chain = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_TRANSFER_SELFTEST:
      if (value != 0 && value != 1) return TOPOEP_ERR_ARG;
      h->transfer_selftest = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_PACKED_IDS:
      if (value < 0 || value > 2) return TOPOEP_ERR_ARG;
      h->pack_ids = value;
      return TOPOEP_OK;
    case TOPOEP_KNOB_REROUTE_TILES:
      if (value < 1 || value > 64) return TOPOEP_ERR_ARG;
      h->reroute_tiles_per_block = value;
      return TOPOEP_OK;
    default:
      return TOPOEP_ERR_ARG;
  }
}

int topoep_set_policy(topoep_handle_t h, int policy, int value) {
  if (!h) return TOPOEP_ERR_NULL;
  switch (policy) {
    case TOPOEP_POLICY_RESERVE_SLOTS:
      if (value < 0 || value > h->d.N) return TOPOEP_ERR_ARG;
      h->reserve_slots = value;
      return TOPOEP_OK;
    case TOPOEP_POLICY_STAGE1_RANK:
      if (value != 0 && value != 1) return TOPOEP_ERR_ARG;
      h->stage1_lpt = value;
      return TOPOEP_OK;
    default:
      return TOPOEP_ERR_ARG;
  }
}

int topoep_set_rank_window(topoep_handle_t h, int first_rank, int rank_count) {
  if (!h) return TOPOEP_ERR_NULL;
  if (first_rank < 0 || rank_count < 1 || first_rank + rank_count > h->d.R) return TOPOEP_ERR_ARG;
  h->rank_first = first_rank;
  h->rank_count = rank_count;
  h->hist_tile_ids = h->hist_tokens = h->hist_batch = -1;   // earlier tile counts no longer apply
  h->packed_src = nullptr;
  return TOPOEP_OK;
}

int topoep_plan_kernels(topoep_handle_t h, int tokens_per_rank, int batch) {
  const int rc = check_sizes(h, tokens_per_rank, batch);
  if (rc != TOPOEP_OK) return rc;
  return use_two_kernels(h, tokens_per_rank, batch) ? 2
         : use_four_kernels(h, tokens_per_rank, batch) ? 4 : 5;
}

int topoep_plan_byte_copy(topoep_handle_t h, int tokens_per_rank, int batch) {
  const int rc = check_sizes(h, tokens_per_rank, batch);
  if (rc != TOPOEP_OK) return rc;
  if (use_two_kernels(h, tokens_per_rank, batch) || use_four_kernels(h, tokens_per_rank, batch)) return 0;
  // alignment aside: the query has no buffers
  return use_packed_ids(h, nullptr, tokens_per_rank, batch) ? 1 : 0;
}

int topoep_get_layout(topoep_handle_t h, int* e_loc, int* s_phys, int* instances) {
  if (!h) return TOPOEP_ERR_NULL;
  if (e_loc) *e_loc = h->d.e_loc;
  if (s_phys) *s_phys = h->d.s_phys;
  if (instances) *instances = h->d.P;
  return TOPOEP_OK;
}

int topoep_launch_floor(int count, topoep_stream_t stream) {
  if (count < 0 || count > 1024) return TOPOEP_ERR_ARG;
  return launch_empty(count, stream) == cudaSuccess ? TOPOEP_OK : TOPOEP_ERR_CUDA;
}

const char* topoep_strerror(int status) {
  switch (status) {
    case TOPOEP_OK: return "ok";
    case TOPOEP_ERR_NULL: return "a required pointer is NULL";
    case TOPOEP_ERR_CONFIG: return "topology, expert, slot or size numbers out of range";
    case TOPOEP_ERR_MAIN_MAP: return "main_rank entry out of range, or E % R != 0 with no map";
    case TOPOEP_ERR_COST: return "negative or oversized cost parameter";
    case TOPOEP_ERR_WORKSPACE: return "workspace missing, too small or not 256-byte aligned";
    case TOPOEP_ERR_SIZE: return "tokens_per_rank or batch outside [0, max]";
    case TOPOEP_ERR_ALIGN: return "a device buffer is misaligned";
    case TOPOEP_ERR_CUDA: return "a CUDA runtime call failed";
    case TOPOEP_ERR_SMEM: return "problem does not fit one SM's shared memory";
    case TOPOEP_ERR_ARG: return "unknown selector, knob or value";
    case TOPOEP_ERR_SCRATCH: return "problem exceeds the 8 MiB scratch array built into the library";
    default: return "unknown status";
  }
}

}  // extern "C"
