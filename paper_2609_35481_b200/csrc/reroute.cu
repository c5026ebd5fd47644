// Per-token replica assignment (paper, "System Design": the token-routing decisions q drive
// dispatch; here each assignment is told which physical instance executes it).
//
// Within a (plan, source rank, expert) group the assignments are ranked by flat index t*k+j
// and dealt to the expert's instances in ascending rank order, instance r taking q(s,e,r) of
// them.  For most (source, expert) pairs one instance takes everything, so the answer is one
// table lookup (route[e] >= 0) and the tile is streamed: load ids, look up, store.  Assignments
// of "split" experts (route[e] = -2-i) are pushed on a work list and patched afterwards; their
// stable rank is
//     [count of e in earlier tiles of the row]          prefix table written by the route kernel
//   + [count of e in earlier 128-id rows of this tile]  scan of the per-row totals
//   + [count of e in lower lanes of the row]            per-lane 4-bit counters, packed 8 per word
//   + [count of e earlier in the lane's own 4 ids]      compared in registers when pushed
// The counters are only ever summed and each 4-bit field belongs to one lane, the order of the
// work list is irrelevant (every item computes its own rank and writes its own output word), so
// no result depends on the order in which atomics arrive, and the output is identical for
// every tile size.  Split experts are ranked kSplitCap at a time; more of them only add passes.
#include "topoep_internal.cuh"
#include "reroute_tail.cuh"

namespace topoep {

namespace {

struct RerouteLayout { size_t cnt, base, route, hdr, seg, cum, inst, tbase, tbase1, work, total; };

// Every region starts on a 16-byte boundary (cp.async destinations).  hdr and seg are adjacent,
// like in the split record, so that one copy brings both.
__host__ __device__ inline RerouteLayout reroute_layout(const Dims& d, int tile_ids) {
  const int rows = tile_ids / 128;
  auto pad4 = [](size_t ints) { return (ints + 3) & ~(size_t)3; };
  RerouteLayout o;
  size_t at = 0;
  o.cnt = at;   at += sizeof(uint4) * (size_t)kSplitCap * rows;
  o.base = at;  at += sizeof(int) * (size_t)kSplitCap * rows;
  o.route = at; at += sizeof(int) * pad4(d.E + 1);
  o.hdr = at;   at += sizeof(int) * 4;                       // n_split, n_list, n_work
  o.seg = at;   at += sizeof(int) * pad4(d.E + 1 > kSplitCap + 4 ? d.E + 1 : kSplitCap + 4);
  o.cum = at;   at += sizeof(int) * pad4(d.P);
  o.inst = at;  at += sizeof(int) * pad4(d.P);
  o.tbase = at; at += sizeof(int) * (size_t)3 * kSplitCap;   // tile prefixes, resolved instances, experts
  o.tbase1 = at; at += sizeof(int) * (size_t)3 * kSplitCap;  // the same of the next tile (multi-tile kernel); directly behind tbase
  o.work = at;  at += sizeof(unsigned short) * (size_t)tile_ids;
  o.total = at;
  return o;
}

// 32 registers per thread: eight 256-thread CTAs per SM; measured faster than 40 or 48 registers
#ifndef TOPOEP_REROUTE_MIN_CTAS
#define TOPOEP_REROUTE_MIN_CTAS 4
#endif
template <bool VEC>
__global__ void __launch_bounds__(kMaxTileIds / kIdsPerThread, TOPOEP_REROUTE_MIN_CTAS) reroute_kernel(const RerouteParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const Dims d = p.d;
  const int E = d.E, P = d.P;
  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5, nwarps = nt >> 5;
  const int rows = 4 * nwarps;   // 128-id rows of the tile, in flat order
  const RerouteLayout lay = reroute_layout(d, p.tile_ids);
  uint4* cnt4 = reinterpret_cast<uint4*>(smem + lay.cnt);      // [kSplitCap][rows]
  unsigned* cntw = reinterpret_cast<unsigned*>(smem + lay.cnt);
  int* base = reinterpret_cast<int*>(smem + lay.base);         // [kSplitCap][rows]
  int* route = reinterpret_cast<int*>(smem + lay.route);
  int* seg = reinterpret_cast<int*>(smem + lay.seg);
  int* cum = reinterpret_cast<int*>(smem + lay.cum);
  int* inst = reinterpret_cast<int*>(smem + lay.inst);
  int* tbase = reinterpret_cast<int*>(smem + lay.tbase);
  int* hdr = reinterpret_cast<int*>(smem + lay.hdr);           // n_split, n_list, n_work
  unsigned short* work = reinterpret_cast<unsigned short*>(smem + lay.work);

  // workspace rows are indexed by the global source rank, the caller's buffers by their window
  const size_t row = (size_t)b * d.R + p.rank_first + s;
  const size_t user_row = (size_t)b * p.rank_count + s;
  const int begin = tile * p.tile_ids;
  const int count = min(p.tile_ids, p.n_ids - begin);
  const int32_t* ids = p.ids + user_row * (size_t)p.n_ids + begin;
  int32_t* out = p.out_token_replica + user_row * (size_t)p.n_ids + begin;

  // The ids go to registers first: sixteen per thread, all four loads in flight.
  int4 x[kIdsPerThread / 4];
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) x[j] = load_ids4(ids, j * nt + tid, count, VEC);
  pdl_wait();   // the ids above are nobody's output; the tables below are the route kernel's
  const SplitRec rl = split_rec_layout(E, P, p.max_tiles);
  const int32_t* rec = p.ws.split_rec + row * (size_t)rl.ints;
  const int32_t* g_route = p.ws.route + row * E;
  const int32_t* g_tp = p.ws.tile_pref + (row * (size_t)p.max_tiles + tile) * E;
  // Tables go global -> shared asynchronously, one 16-byte piece per thread, without passing
  // through registers (the ids above need those): the route table, the head of the split record
  // (header + first list segments, first kFastLists quotas and instances) and this tile's prefix
  // bases of the first kSplitCap split experts.  All of it is fetched before n_split is known;
  // the buffers are always large enough, surplus entries are ignored.
  {
    const int n_route = (E % 4 == 0) ? E / 4 : 0;            // 16-byte pieces of the route table
    const int n_head = (4 + min(E, kSplitCap) + 1 + 3) / 4;  // header + segment starts
    const int n_list4 = (min(P, kFastLists) + 3) / 4;
    const int n_tp = 3 * kSplitCap / 4;   // this tile's prefixes, resolved instances, experts
    int i = tid;
    if (i < n_route) cp_async16(route + 4 * i, g_route + 4 * i);
    i -= n_route;
    if (i >= 0 && i < n_head) cp_async16(hdr + 4 * i, rec + 4 * i);
    i -= n_head;
    if (i >= 0 && i < n_list4) cp_async16(cum + 4 * i, rec + rl.cum + 4 * i);
    i -= n_list4;
    if (i >= 0 && i < n_list4) cp_async16(inst + 4 * i, rec + rl.inst + 4 * i);
    i -= n_list4;
    if (i >= 0 && i < n_tp) cp_async16(tbase + 4 * i, rec + rl.tp + tile * 3 * kSplitCap + 4 * i);
    // shapes these fixed assignments do not cover: more pieces than threads, or E % 4 != 0
#pragma unroll 1
    for (int j = tid + nt; j < n_route + n_head + 2 * n_list4 + n_tp; j += nt) {
      int u = j;
      if (u < n_route) { cp_async16(route + 4 * u, g_route + 4 * u); continue; }
      u -= n_route;
      if (u < n_head) { cp_async16(hdr + 4 * u, rec + 4 * u); continue; }
      u -= n_head;
      if (u < n_list4) { cp_async16(cum + 4 * u, rec + rl.cum + 4 * u); continue; }
      u -= n_list4;
      if (u < n_list4) { cp_async16(inst + 4 * u, rec + rl.inst + 4 * u); continue; }
      u -= n_list4;
      cp_async16(tbase + 4 * u, rec + rl.tp + tile * 3 * kSplitCap + 4 * u);
    }
    if (E % 4 != 0) {
#pragma unroll 1
      for (int e = tid; e < E; e += nt) cp_async4(route + e, g_route + e);
    }
  }
  if (tid == 0) route[E] = -1;   // every id outside [0,E) is clamped onto this entry
  cp_async_wait_all();           // hdr[2], the work-list length, arrives as the record's zero
  __syncthreads();
  // A split expert whose ids of THIS tile all fall inside one instance's quota interval (the
  // route kernel checked the tile's rank interval against the quotas) is not split here: its
  // table entry becomes that instance and its ids stream like everyone else's.  Only tiles that
  // straddle a quota boundary -- about one in ten on the benchmark workloads -- rank anything.
  int marks = 0;   // does the table still hold a split mark for this tile?
  if (hdr[0] > 0) {   // uniform: the source has split experts at all
    int mine = 0;
    if (tid < kSplitCap) {
      const int res = tbase[kSplitCap + tid], e = tbase[2 * kSplitCap + tid];
      if (tid < hdr[0] && e >= 0) {
        if (res >= 0) route[e] = res; else mine = 1;
      }
    }
    marks = __syncthreads_or(mine) | (hdr[0] > kSplitCap);
  }
  if (!marks) {
    // Most tiles: no entry of the table is a split mark, so every entry is an instance or the -1
    // of an ignored id: look up, store, done (no mask of split ids, no work list, no barrier).
    const unsigned uE = (unsigned)E;
#pragma unroll
    for (int j = 0; j < kIdsPerThread / 4; ++j) {
      const int vec = j * nt + tid;
      const int4 r = make_int4(route[min((unsigned)x[j].x, uE)], route[min((unsigned)x[j].y, uE)],
                               route[min((unsigned)x[j].z, uE)], route[min((unsigned)x[j].w, uE)]);
      if (VEC) {
        if (4 * vec < count) __stcs(reinterpret_cast<int4*>(out) + vec, r);
      } else {
        if (4 * vec + 0 < count) out[4 * vec + 0] = r.x;
        if (4 * vec + 1 < count) out[4 * vec + 1] = r.y;
        if (4 * vec + 2 < count) out[4 * vec + 2] = r.z;
        if (4 * vec + 3 < count) out[4 * vec + 3] = r.w;
      }
    }
    return;
  }

  // Stream: look up and store.  An ignored id and a split id both store -1 for now; the split
  // ones are remembered in a 16-bit mask, pushed on the work list afterwards and patched below.
  const unsigned uE = (unsigned)E;
  unsigned split_mask = 0;
#pragma unroll
  for (int j = 0; j < kIdsPerThread / 4; ++j) {
    const int vec = j * nt + tid;
    // branch-free lookups: an id outside [0,E) reads the -1 stored at route[E]
    const int t0 = route[min((unsigned)x[j].x, uE)];
    const int t1 = route[min((unsigned)x[j].y, uE)];
    const int t2 = route[min((unsigned)x[j].z, uE)];
    const int t3 = route[min((unsigned)x[j].w, uE)];
    // t <= -2  <=>  t + 1 < 0: collect the sign bits
    split_mask |= (((unsigned)(t0 + 1) >> 31) | ((unsigned)(t1 + 1) >> 31) << 1 |
                   ((unsigned)(t2 + 1) >> 31) << 2 | ((unsigned)(t3 + 1) >> 31) << 3) << (4 * j);
    const int4 r = make_int4(max(t0, -1), max(t1, -1), max(t2, -1), max(t3, -1));
    if (VEC) {
      if (4 * vec < count) __stcs(reinterpret_cast<int4*>(out) + vec, r);
    } else {
      if (4 * vec + 0 < count) out[4 * vec + 0] = r.x;
      if (4 * vec + 1 < count) out[4 * vec + 1] = r.y;
      if (4 * vec + 2 < count) out[4 * vec + 2] = r.z;
      if (4 * vec + 3 < count) out[4 * vec + 3] = r.w;
    }
  }
  while (split_mask) {   // ~3% of the ids on the benchmark workloads
    const int k = __ffs(split_mask) - 1;
    split_mask &= split_mask - 1;
    work[CK(p.ws.status, atomicAdd(hdr + 2, 1), p.tile_ids)] =
        (unsigned short)(4 * ((k >> 2) * nt + tid) + (k & 3));
  }
  __syncthreads();   // also orders the stores above before the patches below
  const int n_work = hdr[2];
  if (n_work == 0) return;

  // The ranking's first pass expects its counters zeroed: only the tiles that rank pay for it.
  // rows = blockDim.x / 8, so the kSplitCap * rows counter words are exactly kSplitCap / 8 per
  // thread: straight-line stores (a counted loop here cost a hundred instructions per warp).
  static_assert(kSplitCap % 8 == 0, "counter words per thread");
#pragma unroll
  for (int u = 0; u < kSplitCap / 8; ++u) cnt4[u * nt + tid] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  const SplitCtx c = {cnt4, cntw, base, route, seg, cum, inst, tbase, work, rec, g_tp, ids, out,
                      rl, rows, hdr[0], hdr[1], n_work, p.ws.status, false};
  rank_and_patch(c, tid, nt, warp, nwarps);
}

// The same for a large topoep_plan call with at most 256 experts, reading the one-byte copy of the
// ids the histogram of the call left in the workspace (a quarter of the bytes of a second read of
// the ids).  With that read gone the single-tile kernel above is bound by its per-block set-up
// (table fetches, two dependent round trips to memory, ~280 of its ~450 instructions per warp),
// so here a block walks `tiles_per_block` consecutive tiles of one source: the route table and the
// split record are fetched once, the next tile's ids and tile bases are fetched while the
// current tile is processed, and the per-tile work is the table patch, the stream and the (rare)
// ranking of split ids.
__global__ void __launch_bounds__(kMaxTileIds / kIdsPerThread, TOPOEP_REROUTE_MIN_CTAS) reroute_rows_kernel(const RerouteParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  const Dims d = p.d;
  const int E = d.E, P = d.P;
  const int s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, nt = blockDim.x, warp = tid >> 5, nwarps = nt >> 5;
  const int rows = 4 * nwarps;   // 128-id rows of a tile, in flat order
  const RerouteLayout lay = reroute_layout(d, p.tile_ids);
  uint4* cnt4 = reinterpret_cast<uint4*>(smem + lay.cnt);      // [kSplitCap][rows]
  unsigned* cntw = reinterpret_cast<unsigned*>(smem + lay.cnt);
  int* base = reinterpret_cast<int*>(smem + lay.base);         // [kSplitCap][rows]
  int* route = reinterpret_cast<int*>(smem + lay.route);
  int* seg = reinterpret_cast<int*>(smem + lay.seg);
  int* cum = reinterpret_cast<int*>(smem + lay.cum);
  int* inst = reinterpret_cast<int*>(smem + lay.inst);
  int* tb0 = reinterpret_cast<int*>(smem + lay.tbase);         // two buffers of 3 * kSplitCap, back to back
  int* hdr = reinterpret_cast<int*>(smem + lay.hdr);           // n_split, n_list, n_work (even, odd tiles)
  unsigned short* work = reinterpret_cast<unsigned short*>(smem + lay.work);

  const size_t row = (size_t)b * d.R + s;   // whole plans only: the caller's rows are the workspace's
  const int t_first = blockIdx.x * p.tiles_per_block;
  const int t_end = min(p.tiles, t_first + p.tiles_per_block);
  const SplitRec rl = split_rec_layout(E, P, p.max_tiles);
  const int32_t* rec = p.ws.split_rec + row * (size_t)rl.ints;
  const int32_t* g_route = p.ws.route + row * E;
  const unsigned char* row8 = p.ws.ids8 + row * (size_t)p.n_ids;
  const int32_t* flags = p.ws.tile_flag + row * (size_t)p.max_tiles;
  const int n_tp = 3 * kSplitCap / 4;   // 16-byte pieces of a tile's bases

  pdl_wait();   // the byte copy is this call's histogram's, the tables are the route kernel's
  // ids of the first tile: four words = sixteen ids per thread, all loads in flight
  unsigned xb[kIdsPerThread / 4];
  int reread;
  {
    const int begin = t_first * p.tile_ids, count = min(p.tile_ids, p.n_ids - begin);
    const unsigned* pk = reinterpret_cast<const unsigned*>(row8 + begin);
#pragma unroll
    for (int j = 0; j < kIdsPerThread / 4; ++j) xb[j] = 4 * (j * nt + tid) < count ? __ldcs(pk + j * nt + tid) : 0u;
    reread = __ldg(flags + t_first);
  }
  {   // tables of the source, once: global -> shared, 16 bytes per piece
    const int n_route = (E % 4 == 0) ? E / 4 : 0;
    const int n_head = (4 + min(E, kSplitCap) + 1 + 3) / 4;
    const int n_list4 = (min(P, kFastLists) + 3) / 4;
#pragma unroll 1
    for (int j = tid; j < n_route + n_head + 2 * n_list4 + n_tp; j += nt) {
      int u = j;
      if (u < n_route) { cp_async16(route + 4 * u, g_route + 4 * u); continue; }
      u -= n_route;
      if (u < n_head) { cp_async16(hdr + 4 * u, rec + 4 * u); continue; }
      u -= n_head;
      if (u < n_list4) { cp_async16(cum + 4 * u, rec + rl.cum + 4 * u); continue; }
      u -= n_list4;
      if (u < n_list4) { cp_async16(inst + 4 * u, rec + rl.inst + 4 * u); continue; }
      u -= n_list4;
      cp_async16(tb0 + 4 * u, rec + rl.tp + t_first * 3 * kSplitCap + 4 * u);
    }
    if (E % 4 != 0) {
#pragma unroll 1
      for (int e = tid; e < E; e += nt) cp_async4(route + e, g_route + e);
    }
  }
  if (tid == 0) route[E] = -1;   // an id outside [0,E) (re-read tiles) is clamped onto this entry

#pragma unroll 1
  for (int tile = t_first; tile < t_end; ++tile) {
    const int cur = (tile - t_first) & 1;
    int* tbase = tb0 + cur * 3 * kSplitCap;
    cp_async_wait_all();   // first pass: every table; later: this tile's bases
    __syncthreads();       // ... visible; the tile before this one is finished with every buffer
    const int begin = tile * p.tile_ids;
    const int count = min(p.tile_ids, p.n_ids - begin);
    const int32_t* ids = p.ids + row * (size_t)p.n_ids + begin;
    int32_t* out = p.out_token_replica + row * (size_t)p.n_ids + begin;
    // the next tile's ids, flag and bases travel while this one is processed
    unsigned xn[kIdsPerThread / 4];
    int reread_n = 0;
    if (tile + 1 < t_end) {
      const int nbegin = begin + p.tile_ids, ncount = min(p.tile_ids, p.n_ids - nbegin);
      const unsigned* pk = reinterpret_cast<const unsigned*>(row8 + nbegin);
#pragma unroll
      for (int j = 0; j < kIdsPerThread / 4; ++j) xn[j] = 4 * (j * nt + tid) < ncount ? __ldcs(pk + j * nt + tid) : 0u;
      reread_n = __ldg(flags + tile + 1);
      if (tid < n_tp) cp_async16(tb0 + (cur ^ 1) * 3 * kSplitCap + 4 * tid, rec + rl.tp + (tile + 1) * 3 * kSplitCap + 4 * tid);
    } else {
#pragma unroll
      for (int j = 0; j < kIdsPerThread / 4; ++j) xn[j] = 0u;
    }
    const int n_split = hdr[0];
    if (tid == 0) hdr[2 + (cur ^ 1)] = 0;   // the next tile's work counter; nobody reads it now
    // A split expert whose ids of THIS tile all fall inside one instance's quota interval is not
    // split here: its table entry becomes that instance, else (again) the split mark.
    int marks = 0;   // does the table hold a split mark for this tile?
    if (n_split > 0) {   // uniform
      int mine = 0;
      if (tid < kSplitCap && tid < n_split) {
        const int res = tbase[kSplitCap + tid], e = tbase[2 * kSplitCap + tid];
        if (e >= 0) { route[e] = res >= 0 ? res : -2 - tid; mine = res < 0; }
      }
      marks = __syncthreads_or(mine) | (n_split > kSplitCap);
    }
    int* n_work_p = hdr + 2 + cur;
    if (!reread && !marks) {
      // Nine tiles in ten: every id is a valid expert and no entry of the table is a split mark
      // (each split expert's ids of this tile lie inside one instance's quota): look up, store.
      const char* rb = reinterpret_cast<const char*>(route);
#pragma unroll
      for (int j = 0; j < kIdsPerThread / 4; ++j) {
        const int vec = j * nt + tid;
        const unsigned w = xb[j];
        const int t0 = *reinterpret_cast<const int*>(rb + ((w << 2) & 0x3fcu));
        const int t1 = *reinterpret_cast<const int*>(rb + ((w >> 6) & 0x3fcu));
        const int t2 = *reinterpret_cast<const int*>(rb + ((w >> 14) & 0x3fcu));
        const int t3 = *reinterpret_cast<const int*>(rb + ((w >> 22) & 0x3fcu));
        if (4 * vec < count) __stcs(reinterpret_cast<int4*>(out) + vec, make_int4(t0, t1, t2, t3));
      }
    } else if (!reread) {
      // Every id of the tile is a valid expert (the histogram saw none outside [0, E)), so a table
      // entry is an instance (>= 0) or a split mark (< 0): no clamp, and the sign alone tells the
      // split ids.  Their marks are stored as they are: each of them is patched below.  The byte
      // becomes a byte offset into the table with one shift and one mask.
      const char* rb = reinterpret_cast<const char*>(route);
      unsigned sm4[kIdsPerThread / 4];   // bit 8u+7: id u of group j is split
#pragma unroll
      for (int j = 0; j < kIdsPerThread / 4; ++j) {
        const int vec = j * nt + tid;
        const unsigned w = xb[j];
        const int t0 = *reinterpret_cast<const int*>(rb + ((w << 2) & 0x3fcu));
        const int t1 = *reinterpret_cast<const int*>(rb + ((w >> 6) & 0x3fcu));
        const int t2 = *reinterpret_cast<const int*>(rb + ((w >> 14) & 0x3fcu));
        const int t3 = *reinterpret_cast<const int*>(rb + ((w >> 22) & 0x3fcu));
        const unsigned top = __byte_perm(__byte_perm((unsigned)t0, (unsigned)t1, 0x0073),
                                         __byte_perm((unsigned)t2, (unsigned)t3, 0x0073), 0x5410);
        const bool in = 4 * vec < count;
        sm4[j] = in ? top & 0x80808080u : 0u;
        if (in) __stcs(reinterpret_cast<int4*>(out) + vec, make_int4(t0, t1, t2, t3));
      }
#pragma unroll
      for (int j = 0; j < kIdsPerThread / 4; ++j) {
        unsigned mm = sm4[j];
        while (mm) {
          const int u = (__ffs(mm) - 1) >> 3;
          mm &= mm - 1;
          work[CK(p.ws.status, atomicAdd(n_work_p, 1), p.tile_ids)] = (unsigned short)(4 * (j * nt + tid) + u);
        }
      }
    } else {
      // padding or invalid ids in the tile (rare): its 4-byte ids, clamped lookups
      const unsigned uE = (unsigned)E;
#pragma unroll 1
      for (int j = 0; j < kIdsPerThread / 4; ++j) {
        const int vec = j * nt + tid;
        const int4 x = load_ids4(ids, vec, count, true);
        const int t[4] = {route[min((unsigned)x.x, uE)], route[min((unsigned)x.y, uE)],
                          route[min((unsigned)x.z, uE)], route[min((unsigned)x.w, uE)]};
        if (4 * vec < count) __stcs(reinterpret_cast<int4*>(out) + vec, make_int4(max(t[0], -1), max(t[1], -1), max(t[2], -1), max(t[3], -1)));
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (t[u] < -1) work[CK(p.ws.status, atomicAdd(n_work_p, 1), p.tile_ids)] = (unsigned short)(4 * vec + u);
      }
    }
    if (reread || marks) {   // uniform: something may have been pushed
      __syncthreads();   // also orders the stores above before the patches below
      const int n_work = *n_work_p;
      if (n_work > 0) {   // uniform
        const int32_t* g_tp = p.ws.tile_pref + (row * (size_t)p.max_tiles + tile) * E;
        const SplitCtx c = {cnt4, cntw, base, route, seg, cum, inst, tbase, work, rec, g_tp, ids, out,
                            rl, rows, n_split, hdr[1], n_work, p.ws.status, false};
        // the ranking's first pass expects its counters zeroed: only the tiles that rank pay for it
#pragma unroll
        for (int u = 0; u < kSplitCap / 8; ++u) cnt4[u * nt + tid] = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
        rank_and_patch(c, tid, nt, warp, nwarps);
      }
    }
#pragma unroll
    for (int j = 0; j < kIdsPerThread / 4; ++j) xb[j] = xn[j];
    reread = reread_n;
  }
}

}  // namespace

size_t reroute_smem_bytes(const Dims& d, int tile_ids) { return reroute_layout(d, tile_ids).total; }

cudaError_t launch_reroute(const RerouteParams& p, int batch, cudaStream_t stream) {
  const dim3 block(p.tile_ids / kIdsPerThread);
  const size_t smem = reroute_smem_bytes(p.d, p.tile_ids);
  if (p.packed && p.vec_ok && p.ws.ids8) {
    const dim3 grid((p.tiles + p.tiles_per_block - 1) / p.tiles_per_block, p.rank_count, batch);
    return launch_kernel(reroute_rows_kernel, grid, block, smem, stream, p.pdl != 0, p);
  }
  const dim3 grid(p.tiles, p.rank_count, batch);
  return p.vec_ok ? launch_kernel(reroute_kernel<true>, grid, block, smem, stream, p.pdl != 0, p)
                  : launch_kernel(reroute_kernel<false>, grid, block, smem, stream, p.pdl != 0, p);
}

cudaError_t configure_reroute(size_t smem) {
  cudaError_t e = cudaFuncSetAttribute(reroute_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(reroute_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(reroute_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

}  // namespace topoep
