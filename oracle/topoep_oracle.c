/*
 * CPU oracle of the TopoEP planning step.  TEST INFRASTRUCTURE ONLY: it exists
 * to check the CUDA library and to be timed as a CPU baseline; no product code
 * may call it, and it shares no code, header, table or helper with the CUDA
 * path.
 *
 * Plain C, int64 arithmetic, dense x[E][R] and q[R][E][R], one nested loop per
 * sentence of the paper's "Two-Stage GPU-Native Solver"; no blocking, fusion
 * or reordering.  The method is a heuristic (the paper does not solve its
 * MILP), so the oracle is the algorithm step by step, in the paper's order
 * and notation:
 *
 *   O1 routing matrix Omega                      ("System Model", Eq. Omega)
 *   O2 domain demand D_{d,e}                     ("System Model", Eq. D)
 *   O3 inter-node placement with b_{d,e}         ("Inter-node placement", Eq. b; C3-C5)
 *   O4 routing construction q                    ("Inter-node placement", 2nd paragraph; C1, C2)
 *   O5 loads U_{e,r}, L_r                        (same paragraph; "Load metric")
 *   O6 intra-node refinement                     ("Intra-node refinement", Eq. delta)
 *   O7 per-token instance assignment             ("System Design": token-routing decisions
 *                                                 drive dispatch; reading stated below)
 *   O8 dispatch layout                           ("DeepEP dispatch and combine": receive
 *                                                 counts derived from the routing)
 *   O9 summaries                                 (objective terms T_comp, T_token, T_replica;
 *                                                 max/mean load ratio; inter-node and
 *                                                 replica-served fractions)
 *   O10 dispatch permutation                     (the step after the path; layout defined at
 *                                                 the function, pinned to numpy.lexsort)
 *   O11 replica parameter pull, O12 replica      ("Device-initiated replica transfers" with the
 *       gradient return                           three buffers of the same subsection; pinned by
 *                                                 hand-written byte fixtures and an identity code)
 *
 * Where the paper is silent the readings are (all listed in the design notes
 * of the repository, none of them pinned by the paper itself):
 *   - dom(r) = r / G.
 *   - C4 is strict: a cross-domain replica needs 2*D*S_tok - W > 0.
 *   - candidates of a domain are ordered by (b descending, e ascending); at
 *     most one replica per (domain, expert) in stage 1; experts whose main is
 *     in the domain are never candidates there.
 *   - "least occupied rank with a free slot" = fewest used replica slots,
 *     ties to the lowest rank id; stage 1 fills until candidates or slots end.
 *   - "approximately evenly": omega = base*n + rem; the rem instances starting
 *     at index (s+e) mod n of the ascending-rank selection get base+1.
 *   - refinement: busiest rank ties to the lowest id; candidates are all
 *     instances on it with U>0; a candidate needs delta >= min_delta; ranking
 *     is lexicographic (delta larger, target load smaller, replica-creation
 *     cost smaller, e smaller, r_t smaller); creation cost is 0 when the target
 *     hosts e already, else c(main(e), r_t)*W; moved units are taken from
 *     source r_t first, then the other sources ascending, source r_b last;
 *     replicas are never freed; a hard iteration cap per domain is an input.
 *   - per-token: within a (source, expert) group assignments are ranked by
 *     flat index t*k+j and dealt to the instances in ascending rank order,
 *     instance r taking q[s][e][r] of them.
 *   - ids outside [0,E) are ignored everywhere and map to -1.
 *   - the paper does not say whether inter-node placement leaves slots for the refinement; by
 *     default it does not (its slot-count experiment reports no gain from refinement with one
 *     slot per rank).  reserve_slots > 0 is a policy variant of ours: stage 1 fills at most
 *     N_slot - reserve_slots slots of a rank.
 *   - "least occupied" could also be read as least token-loaded; stage1_rank = 1 is that reading
 *     as a policy variant (LPT), with the load estimated before any routing exists: the demand on
 *     the rank's main instances plus the domain demand of the replicas it already got.
 *
 * Parity status: O1, O8 are pinned to library routines (bincount, cumsum);
 * O3-O6 are pinned by the paper's worked two-domain example, hand-derived
 * fixtures for each tie-break, constraints C1-C5, per-iteration half-gap
 * invariants, and exact MILP optima on tiny instances; O7 is pinned by
 * brute-force counting; O9 by the paper's 64 MiB / 27 MiB cost example and
 * the (M-1)/M closed form.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int32_t nodes;            /* M */
  int32_t gpus_per_node;    /* G */
  int32_t experts;          /* E */
  int32_t slots_per_rank;   /* N_slot */
  int32_t top_k;            /* k */
  int32_t c_intra;          /* c_{s,r}, same domain, s != r */
  int32_t c_inter;          /* c_{s,r}, different domains   */
  int32_t max_refine_iters; /* <= 0 -> 256 */
  int32_t min_delta;        /* <= 0 -> 1   */
  int32_t stages;           /* bit 0: run inter-node placement; bit 1: run refinement */
  int32_t reserve_slots;    /* non-default policy: slots per rank that inter-node placement
                               must leave free for the refinement (0 = the paper's behaviour) */
  int32_t stage1_rank;      /* non-default policy: 0 = a candidate goes to the rank with the
                               fewest used slots (the paper's wording), 1 = to the rank with the
                               smallest estimated token load (LPT) */
  int64_t token_bytes;      /* S_tok */
  int64_t expert_bytes;     /* ||W|| */
  int64_t t_ffn;            /* t_FFN */
} oracle_config;

typedef struct {
  int64_t assignments, l_max, cross_assignments, replica_served;
  int64_t replicas_inter, replicas_intra;
  int64_t t_comp, t_token, t_replica, cross_token_bytes, refine_iters, reserved;
  double imbalance, cross_fraction, replica_fraction;
} oracle_summary;

#define ORACLE_FLAG_BAD_ID 1u
#define ORACLE_FLAG_REFINE_CAP 2u
#define ORACLE_TRACE_COLS 9

static int dom_of(const oracle_config* c, int r) { return r / c->gpus_per_node; }

/* c_{s,r}: 0 on the diagonal, c_intra inside a domain, c_inter across. */
static int64_t comm_cost(const oracle_config* c, int s, int r) {
  if (s == r) return 0;
  return dom_of(c, s) == dom_of(c, r) ? c->c_intra : c->c_inter;
}

/* E_loc: the largest number of experts sharing one main rank. */
int oracle_e_loc(const oracle_config* c, const int32_t* main_rank) {
  const int R = c->nodes * c->gpus_per_node;
  int best = 0;
  for (int r = 0; r < R; ++r) {
    int n = 0;
    for (int e = 0; e < c->experts; ++e) n += (main_rank[e] == r);
    if (n > best) best = n;
  }
  return best;
}

/*
 * Physical instance id of expert e on rank r, or -1 if r does not host it.
 * l < E_loc: position of e among the experts whose main is r (ascending e);
 * l = E_loc + j: replica slot j.
 */
static int64_t instance_id(const oracle_config* c, const int32_t* main_rank,
                           const int32_t* slotmap, int e_loc, int e, int r) {
  const int s_phys = e_loc + c->slots_per_rank;
  if (main_rank[e] == r) {
    int l = 0;
    for (int e2 = 0; e2 < e; ++e2) l += (main_rank[e2] == r);
    return (int64_t)r * s_phys + l;
  }
  for (int j = 0; j < c->slots_per_rank; ++j)
    if (slotmap[(size_t)r * c->slots_per_rank + j] == e) return (int64_t)r * s_phys + e_loc + j;
  return -1;
}

/* O1 -- omega[s][e] = number of assignments of source rank s that select e. */
void oracle_histogram(const oracle_config* c, const int32_t* ids /*[R][T][k]*/, int T,
                      int64_t* omega /*[R][E]*/, uint32_t* flags) {
  const int R = c->nodes * c->gpus_per_node, E = c->experts, k = c->top_k;
  memset(omega, 0, sizeof(int64_t) * (size_t)R * E);
  for (int s = 0; s < R; ++s)
    for (int t = 0; t < T; ++t)
      for (int j = 0; j < k; ++j) {
        const int32_t e = ids[((size_t)s * T + t) * k + j];
        if (e >= 0 && e < E) omega[(size_t)s * E + e] += 1;
        else if (e != -1) *flags |= ORACLE_FLAG_BAD_ID;
      }
}

/* O2 -- D[d][e] = sum of omega[s][e] over the source ranks s of domain d. */
static void domain_demand(const oracle_config* c, const int64_t* omega, int64_t* D /*[M][E]*/) {
  const int R = c->nodes * c->gpus_per_node, E = c->experts;
  memset(D, 0, sizeof(int64_t) * (size_t)c->nodes * E);
  for (int s = 0; s < R; ++s)
    for (int e = 0; e < E; ++e) D[(size_t)dom_of(c, s) * E + e] += omega[(size_t)s * E + e];
}

/*
 * O3 -- inter-node placement.  Every domain, on its own: the experts whose
 * main lies outside it and whose benefit b = 2*D*S_tok - W is positive, taken
 * in descending order of b, each put on the rank of the domain that has a free
 * slot and the fewest used slots.  A single domain has nothing to evaluate.
 */
static void inter_node_placement(const oracle_config* c, const int32_t* main_rank,
                                 const int64_t* D, int8_t* x, int32_t* slotmap, int32_t* used) {
  const int M = c->nodes, G = c->gpus_per_node, E = c->experts, R = M * G, N = c->slots_per_rank;
  /* slots this stage may fill on a rank: all of them unless the reservation policy is on */
  int cap = N - (c->reserve_slots > 0 ? c->reserve_slots : 0);
  if (cap < 0) cap = 0;
  if (M == 1) return;
  int8_t* taken = (int8_t*)malloc((size_t)E);
  /* LPT variant: estimated load of a rank = what its main instances receive from all sources
     (sum over the domains of D) plus the demand D[d][e] of the replicas placed on it so far */
  int64_t* est = (int64_t*)calloc((size_t)R, sizeof(int64_t));
  for (int e = 0; e < E; ++e)
    for (int d = 0; d < M; ++d) est[main_rank[e]] += D[(size_t)d * E + e];
  for (int d = 0; d < M; ++d) {
    memset(taken, 0, (size_t)E);
    for (;;) {
      /* next candidate: largest b, then smallest e, among those not taken yet */
      int best_e = -1;
      int64_t best_b = 0;
      for (int e = 0; e < E; ++e) {
        if (taken[e] || dom_of(c, main_rank[e]) == d) continue;
        const int64_t b = 2 * D[(size_t)d * E + e] * c->token_bytes - c->expert_bytes;
        if (b <= 0) continue;
        if (best_e < 0 || b > best_b) { best_e = e; best_b = b; }
      }
      if (best_e < 0) break;
      /* the rank of d that takes it, among those with a free slot: the least occupied one, or
         (LPT variant) the one with the smallest estimated load; ties to the lowest rank */
      int best_r = -1;
      for (int r = d * G; r < (d + 1) * G; ++r) {
        if (used[r] >= cap) continue;
        if (best_r < 0) { best_r = r; continue; }
        if (c->stage1_rank == 1 ? est[r] < est[best_r] : used[r] < used[best_r]) best_r = r;
      }
      if (best_r < 0) break;
      slotmap[(size_t)best_r * N + used[best_r]] = best_e;
      x[(size_t)best_e * R + best_r] = 1;
      used[best_r] += 1;
      est[best_r] += D[(size_t)d * E + best_e];
      taken[best_e] = 1;
    }
  }
  free(est);
  free(taken);
}

/*
 * O4 -- routing construction.  For each (s,e): the instances inside dom(s) if
 * there are any, else all instances, in ascending rank order; omega[s][e] is
 * divided evenly, the remainder going one each to consecutive instances
 * starting at index (s+e) mod n.
 */
static void routing_construction(const oracle_config* c, const int64_t* omega, const int8_t* x,
                                 int64_t* q /*[R][E][R]*/) {
  const int R = c->nodes * c->gpus_per_node, E = c->experts;
  int* sel = (int*)malloc(sizeof(int) * (size_t)R);
  memset(q, 0, sizeof(int64_t) * (size_t)R * E * R);
  for (int s = 0; s < R; ++s)
    for (int e = 0; e < E; ++e) {
      const int64_t w = omega[(size_t)s * E + e];
      if (w == 0) continue;
      int n = 0;
      for (int r = 0; r < R; ++r)
        if (x[(size_t)e * R + r] && dom_of(c, r) == dom_of(c, s)) sel[n++] = r;
      if (n == 0)
        for (int r = 0; r < R; ++r)
          if (x[(size_t)e * R + r]) sel[n++] = r;
      const int64_t base = w / n, rem = w % n;
      const int start = (s + e) % n;
      for (int i = 0; i < n; ++i) {
        const int shifted = ((i - start) % n + n) % n;
        q[((size_t)s * E + e) * R + sel[i]] = base + (shifted < rem ? 1 : 0);
      }
    }
  free(sel);
}

/* O5 -- U[e][r] = sum_s q[s][e][r]; L[r] = sum_e U[e][r]. */
static void compute_loads(const oracle_config* c, const int64_t* q, int64_t* U, int64_t* L) {
  const int R = c->nodes * c->gpus_per_node, E = c->experts;
  memset(U, 0, sizeof(int64_t) * (size_t)E * R);
  memset(L, 0, sizeof(int64_t) * (size_t)R);
  for (int s = 0; s < R; ++s)
    for (int e = 0; e < E; ++e)
      for (int r = 0; r < R; ++r) U[(size_t)e * R + r] += q[((size_t)s * E + e) * R + r];
  for (int e = 0; e < E; ++e)
    for (int r = 0; r < R; ++r) L[r] += U[(size_t)e * R + r];
}

/*
 * O6 -- intra-node refinement of one domain.  Each iteration: busiest rank
 * r_b; for every expert loading it and every other rank r_t of the domain that
 * hosts the expert or has a free slot, delta = min(U[e][r_b], (L_b - L_t)/2);
 * the best candidate by (delta, target load, cost) is committed: a replica is
 * created if needed and delta units of q move from r_b to r_t.
 */
static void refine_domain(const oracle_config* c, const int32_t* main_rank, int d, int8_t* x,
                          int32_t* slotmap, int32_t* used, int64_t* q, int64_t* U, int64_t* L,
                          int32_t* iters_out, uint32_t* flags, int64_t* trace, int64_t trace_cap,
                          int64_t* n_trace) {
  const int G = c->gpus_per_node, E = c->experts, R = c->nodes * G, N = c->slots_per_rank;
  const int cap = c->max_refine_iters > 0 ? c->max_refine_iters : 256;
  const int64_t min_delta = c->min_delta > 0 ? c->min_delta : 1;
  int it = 0;
  for (;;) {
    int rb = d * G;
    for (int r = d * G; r < (d + 1) * G; ++r)
      if (L[r] > L[rb]) rb = r;
    int have = 0, be = 0, brt = 0;
    int64_t bdelta = 0, bload = 0, bcost = 0;
    for (int e = 0; e < E; ++e) {
      if (U[(size_t)e * R + rb] <= 0) continue;
      for (int rt = d * G; rt < (d + 1) * G; ++rt) {
        if (rt == rb) continue;
        const int hosts = x[(size_t)e * R + rt];
        if (!hosts && used[rt] >= N) continue;
        int64_t delta = (L[rb] - L[rt]) / 2;
        if (U[(size_t)e * R + rb] < delta) delta = U[(size_t)e * R + rb];
        if (delta < min_delta) continue;
        const int64_t cost = hosts ? 0 : comm_cost(c, main_rank[e], rt) * c->expert_bytes;
        int better;
        if (!have) better = 1;
        else if (delta != bdelta) better = delta > bdelta;
        else if (L[rt] != bload) better = L[rt] < bload;
        else if (cost != bcost) better = cost < bcost;
        else if (e != be) better = e < be;
        else better = rt < brt;
        if (better) { have = 1; be = e; brt = rt; bdelta = delta; bload = L[rt]; bcost = cost; }
      }
    }
    if (!have) break;
    if (it >= cap) { *flags |= ORACLE_FLAG_REFINE_CAP; break; }
    int created = 0;
    if (!x[(size_t)be * R + brt]) {
      slotmap[(size_t)brt * N + used[brt]] = be;
      x[(size_t)be * R + brt] = 1;
      used[brt] += 1;
      created = 1;
    }
    if (trace && *n_trace < trace_cap) {
      int64_t* row = trace + (*n_trace) * ORACLE_TRACE_COLS;
      row[0] = d; row[1] = it; row[2] = be; row[3] = rb; row[4] = brt; row[5] = bdelta;
      row[6] = L[rb]; row[7] = L[brt]; row[8] = created;
    }
    if (trace) *n_trace += 1;
    /* move bdelta units of q: source r_t first, then the others ascending, source r_b last */
    int64_t left = bdelta;
    for (int pass = 0; pass < 3 && left > 0; ++pass)
      for (int s = 0; s < R && left > 0; ++s) {
        const int cls = (s == brt) ? 0 : (s == rb) ? 2 : 1;
        if (cls != pass) continue;
        int64_t* from = &q[((size_t)s * E + be) * R + rb];
        int64_t take = *from < left ? *from : left;
        *from -= take;
        q[((size_t)s * E + be) * R + brt] += take;
        left -= take;
      }
    U[(size_t)be * R + rb] -= bdelta;
    U[(size_t)be * R + brt] += bdelta;
    L[rb] -= bdelta;
    L[brt] += bdelta;
    it += 1;
  }
  iters_out[d] = it;
}

/*
 * O2..O6 from a given routing matrix.  x, slotmap, q, U, L, iters are outputs.
 * trace (optional): one row per refinement commit,
 * (d, iteration, e, r_b, r_t, delta, L_b before, L_t before, replica created).
 */
void oracle_solve(const oracle_config* c, const int32_t* main_rank, const int64_t* omega,
                  int8_t* x /*[E][R]*/, int32_t* slotmap /*[R][N_slot]*/, int64_t* q /*[R][E][R]*/,
                  int64_t* U /*[E][R]*/, int64_t* L /*[R]*/, int64_t* D /*[M][E]*/,
                  int32_t* iters /*[M]*/, uint32_t* flags, int64_t* trace, int64_t trace_cap,
                  int64_t* n_trace) {
  const int M = c->nodes, R = M * c->gpus_per_node, E = c->experts, N = c->slots_per_rank;
  int32_t* used = (int32_t*)calloc((size_t)R, sizeof(int32_t));
  memset(x, 0, (size_t)E * R);
  for (int e = 0; e < E; ++e) x[(size_t)e * R + main_rank[e]] = 1; /* C5 */
  for (size_t i = 0; i < (size_t)R * N; ++i) slotmap[i] = -1;
  for (int d = 0; d < M; ++d) iters[d] = 0;
  if (n_trace) *n_trace = 0;
  domain_demand(c, omega, D);
  if (c->stages & 1) inter_node_placement(c, main_rank, D, x, slotmap, used);
  routing_construction(c, omega, x, q);
  compute_loads(c, q, U, L);
  if (c->stages & 2)
    for (int d = 0; d < M; ++d)
      refine_domain(c, main_rank, d, x, slotmap, used, q, U, L, iters, flags, trace, trace_cap,
                    n_trace);
  free(used);
}

/*
 * O7 -- per-token instance.  Walk the assignments of source s in flat order;
 * rho = how many earlier assignments of s chose the same expert; the ranks
 * with q[s][e][r] > 0, ascending, each cover q[s][e][r] consecutive values of
 * rho; the assignment goes to the instance of e on the covering rank.
 */
void oracle_assign_tokens(const oracle_config* c, const int32_t* main_rank, const int32_t* slotmap,
                          const int32_t* ids /*[R][T][k]*/, int T, const int64_t* q,
                          int32_t* token_replica /*[R][T][k]*/) {
  const int R = c->nodes * c->gpus_per_node, E = c->experts, k = c->top_k;
  const int e_loc = oracle_e_loc(c, main_rank);
  int64_t* seen = (int64_t*)malloc(sizeof(int64_t) * (size_t)E);
  int64_t* inst = (int64_t*)malloc(sizeof(int64_t) * (size_t)E * R);
  for (int e = 0; e < E; ++e)
    for (int r = 0; r < R; ++r)
      inst[(size_t)e * R + r] = instance_id(c, main_rank, slotmap, e_loc, e, r);
  for (int s = 0; s < R; ++s) {
    memset(seen, 0, sizeof(int64_t) * (size_t)E);
    for (int64_t f = 0; f < (int64_t)T * k; ++f) {
      const int32_t e = ids[(size_t)s * T * k + f];
      int32_t out = -1;
      if (e >= 0 && e < E) {
        const int64_t rho = seen[e]++;
        int64_t cum = 0;
        for (int r = 0; r < R; ++r) {
          cum += q[((size_t)s * E + e) * R + r];
          if (rho < cum) { out = (int32_t)inst[(size_t)e * R + r]; break; }
        }
      }
      token_replica[(size_t)s * T * k + f] = out;
    }
  }
  free(seen);
  free(inst);
}

/*
 * O8 -- dispatch layout: counts[s][r] = sum_e q[s][e][r]; send offsets = the
 * exclusive scan of a row over r, receive offsets = the exclusive scan of a
 * column over s, both with the total appended; instance_counts[p] = U of the
 * instance (0 for an unused instance).
 */
void oracle_layout(const oracle_config* c, const int32_t* main_rank, const int32_t* slotmap,
                   const int64_t* q, const int64_t* U, int32_t* counts /*[R][R]*/,
                   int32_t* offsets /*[2][R][R+1]*/, int32_t* instance_counts /*[P]*/) {
  const int R = c->nodes * c->gpus_per_node, E = c->experts;
  const int e_loc = oracle_e_loc(c, main_rank), s_phys = e_loc + c->slots_per_rank;
  for (int s = 0; s < R; ++s)
    for (int r = 0; r < R; ++r) {
      int64_t n = 0;
      for (int e = 0; e < E; ++e) n += q[((size_t)s * E + e) * R + r];
      counts[(size_t)s * R + r] = (int32_t)n;
    }
  int32_t* send = offsets;
  int32_t* recv = offsets + (size_t)R * (R + 1);
  for (int s = 0; s < R; ++s) {
    int64_t acc = 0;
    for (int r = 0; r < R; ++r) { send[(size_t)s * (R + 1) + r] = (int32_t)acc; acc += counts[(size_t)s * R + r]; }
    send[(size_t)s * (R + 1) + R] = (int32_t)acc;
  }
  for (int r = 0; r < R; ++r) {
    int64_t acc = 0;
    for (int s = 0; s < R; ++s) { recv[(size_t)r * (R + 1) + s] = (int32_t)acc; acc += counts[(size_t)s * R + r]; }
    recv[(size_t)r * (R + 1) + R] = (int32_t)acc;
  }
  if (instance_counts) {
    for (size_t p = 0; p < (size_t)R * s_phys; ++p) instance_counts[p] = 0;
    for (int e = 0; e < E; ++e)
      for (int r = 0; r < R; ++r) {
        const int64_t p = instance_id(c, main_rank, slotmap, e_loc, e, r);
        if (p >= 0) instance_counts[p] = (int32_t)U[(size_t)e * R + r];
      }
  }
}

/* O9 -- derived figures of one plan. */
void oracle_summary_of(const oracle_config* c, const int32_t* main_rank, const int8_t* x,
                       const int64_t* q, const int64_t* L, const int32_t* iters,
                       oracle_summary* out) {
  const int M = c->nodes, R = M * c->gpus_per_node, E = c->experts;
  memset(out, 0, sizeof(*out));
  for (int r = 0; r < R; ++r) {
    out->assignments += L[r];
    if (L[r] > out->l_max) out->l_max = L[r];
  }
  int64_t weighted = 0;
  for (int s = 0; s < R; ++s)
    for (int e = 0; e < E; ++e)
      for (int r = 0; r < R; ++r) {
        const int64_t v = q[((size_t)s * E + e) * R + r];
        if (dom_of(c, s) != dom_of(c, r)) out->cross_assignments += v;
        if (r != main_rank[e]) out->replica_served += v;
        weighted += comm_cost(c, s, r) * v;
      }
  for (int e = 0; e < E; ++e)
    for (int r = 0; r < R; ++r) {
      if (!x[(size_t)e * R + r] || r == main_rank[e]) continue;
      if (dom_of(c, r) != dom_of(c, main_rank[e])) out->replicas_inter += 1;
      else out->replicas_intra += 1;
      out->t_replica += comm_cost(c, main_rank[e], r) * c->expert_bytes;
    }
  for (int d = 0; d < M; ++d) out->refine_iters += iters[d];
  out->t_comp = c->t_ffn * out->l_max;
  out->t_token = 2 * c->token_bytes * weighted;
  out->cross_token_bytes = 2 * c->token_bytes * out->cross_assignments;
  if (out->assignments > 0) {
    out->imbalance = (double)(out->l_max * R) / (double)out->assignments;
    out->cross_fraction = (double)out->cross_assignments / (double)out->assignments;
    out->replica_fraction = (double)out->replica_served / (double)out->assignments;
  }
}

/*
 * Whole path for a batch of B independent plans, outputs laid out like the
 * library's.  Optional outputs may be NULL.  Returns 0, or -1 when a scratch
 * allocation fails.
 */
int oracle_plan(const oracle_config* c, const int32_t* main_rank, const int32_t* ids /*[B][R][T][k]*/,
                int T, int B, int32_t* replica_map /*[B][R][N]*/, int32_t* token_replica,
                int32_t* counts /*[B][R][R]*/, int32_t* offsets /*[B][2][R][R+1]*/,
                int32_t* instance_counts /*[B][P]*/, int32_t* omega32 /*[B][R][E]*/,
                int32_t* rank_load /*[B][R]*/, int32_t* refine_iters /*[B][M]*/,
                int32_t* q_instances /*[B][R][P]: q(s, instance), 0 for unused instances*/,
                oracle_summary* summaries /*[B]*/, uint32_t* flags) {
  const int M = c->nodes, R = M * c->gpus_per_node, E = c->experts, N = c->slots_per_rank;
  const int k = c->top_k;
  const int s_phys = oracle_e_loc(c, main_rank) + N;
  int64_t* omega = (int64_t*)malloc(sizeof(int64_t) * (size_t)R * E);
  int8_t* x = (int8_t*)malloc((size_t)E * R);
  int32_t* slotmap = (int32_t*)malloc(sizeof(int32_t) * ((size_t)R * N + 1));
  int64_t* q = (int64_t*)malloc(sizeof(int64_t) * (size_t)R * E * R);
  int64_t* U = (int64_t*)malloc(sizeof(int64_t) * (size_t)E * R);
  int64_t* L = (int64_t*)malloc(sizeof(int64_t) * (size_t)R);
  int64_t* D = (int64_t*)malloc(sizeof(int64_t) * (size_t)M * E);
  int32_t* iters = (int32_t*)malloc(sizeof(int32_t) * (size_t)M);
  int32_t* cnt_tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)R * R);
  int32_t* off_tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)2 * R * (R + 1));
  if (!omega || !x || !slotmap || !q || !U || !L || !D || !iters || !cnt_tmp || !off_tmp) return -1;
  for (int b = 0; b < B; ++b) {
    const int32_t* ids_b = ids + (size_t)b * R * T * k;
    oracle_histogram(c, ids_b, T, omega, flags);
    oracle_solve(c, main_rank, omega, x, slotmap, q, U, L, D, iters, flags, NULL, 0, NULL);
    if (token_replica)
      oracle_assign_tokens(c, main_rank, slotmap, ids_b, T, q, token_replica + (size_t)b * R * T * k);
    oracle_layout(c, main_rank, slotmap, q, U, counts ? counts + (size_t)b * R * R : cnt_tmp,
                  offsets ? offsets + (size_t)b * 2 * R * (R + 1) : off_tmp,
                  instance_counts ? instance_counts + (size_t)b * R * s_phys : NULL);
    if (replica_map) memcpy(replica_map + (size_t)b * R * N, slotmap, sizeof(int32_t) * (size_t)R * N);
    if (omega32)
      for (size_t i = 0; i < (size_t)R * E; ++i) omega32[(size_t)b * R * E + i] = (int32_t)omega[i];
    if (rank_load)
      for (int r = 0; r < R; ++r) rank_load[(size_t)b * R + r] = (int32_t)L[r];
    if (refine_iters) memcpy(refine_iters + (size_t)b * M, iters, sizeof(int32_t) * (size_t)M);
    if (q_instances) {
      const int e_loc = s_phys - N;
      int32_t* qi = q_instances + (size_t)b * R * R * s_phys;
      memset(qi, 0, sizeof(int32_t) * (size_t)R * R * s_phys);
      for (int e = 0; e < E; ++e)
        for (int r = 0; r < R; ++r) {
          const int64_t p = instance_id(c, main_rank, slotmap, e_loc, e, r);
          if (p < 0) continue;
          for (int s = 0; s < R; ++s)
            qi[(size_t)s * R * s_phys + p] = (int32_t)q[((size_t)s * E + e) * R + r];
        }
    }
    if (summaries) oracle_summary_of(c, main_rank, x, q, L, iters, summaries + b);
  }
  free(omega); free(x); free(slotmap); free(q); free(U); free(L); free(D); free(iters);
  free(cnt_tmp); free(off_tmp);
  return 0;
}

/*
 * O10 -- dispatch permutation (the step right after the planning path; the paper leaves the
 * buffer layout to its dispatch library, so this is a definition of ours, stated here):
 *   send_pos: index of an assignment in its source rank's send buffer, which is ordered by
 *             (destination rank, physical instance, flat index t*k+j);
 *   recv_pos: index in its destination rank's receive buffer, which is ordered by
 *             (physical instance, source rank, flat index) -- every instance's tokens contiguous,
 *             ready for a grouped GEMM;
 *   instance_offsets[r][l]: start of instance l's segment in rank r's receive buffer
 *             (entry S_phys = L_r).
 * Written as counting walks, one buffer slot at a time; ignored ids get -1.
 */
void oracle_dispatch_positions(const oracle_config* c, const int32_t* main_rank, int T,
                               const int32_t* token_replica /*[R][T][k]*/, int32_t* send_pos,
                               int32_t* recv_pos, int32_t* instance_offsets /*[R][S_phys+1]*/) {
  const int R = c->nodes * c->gpus_per_node, k = c->top_k;
  const int s_phys = oracle_e_loc(c, main_rank) + c->slots_per_rank;
  const int64_t n = (int64_t)T * k;
  /* send side: for each source, walk the instances in ascending id (= ascending rank, then
     instance) and hand out consecutive slots in flat order */
  for (int s = 0; s < R; ++s) {
    int64_t next = 0;
    for (int p = 0; p < R * s_phys; ++p)
      for (int64_t f = 0; f < n; ++f)
        if (token_replica[(size_t)s * n + f] == p) send_pos[(size_t)s * n + f] = (int32_t)next++;
    for (int64_t f = 0; f < n; ++f)
      if (token_replica[(size_t)s * n + f] < 0) send_pos[(size_t)s * n + f] = -1;
  }
  /* receive side: for each rank, instance by instance, source by source, in flat order */
  for (int r = 0; r < R; ++r) {
    int64_t next = 0;
    for (int l = 0; l < s_phys; ++l) {
      instance_offsets[(size_t)r * (s_phys + 1) + l] = (int32_t)next;
      const int p = r * s_phys + l;
      for (int s = 0; s < R; ++s)
        for (int64_t f = 0; f < n; ++f)
          if (token_replica[(size_t)s * n + f] == p) recv_pos[(size_t)s * n + f] = (int32_t)next++;
    }
    instance_offsets[(size_t)r * (s_phys + 1) + s_phys] = (int32_t)next;
  }
  for (int s = 0; s < R; ++s)
    for (int64_t f = 0; f < n; ++f)
      if (token_replica[(size_t)s * n + f] < 0) recv_pos[(size_t)s * n + f] = -1;
}


/* l(e): position of e among the experts whose main rank is main_rank[e], ascending e. */
static int main_local_index(const int32_t* main_rank, int e) {
  int l = 0;
  for (int e2 = 0; e2 < e; ++e2) l += (main_rank[e2] == main_rank[e]);
  return l;
}

/*
 * O11 -- replica parameter pull ("Device-initiated replica transfers", forward direction).
 * Buffers as the subsection lists them, for all ranks of the simulated group side by side:
 *   main_params [R][E_loc][W]  rank m's main instances, by local index l(e);
 *   replica_buf [R][N_slot][W] rank r's replica slots.
 * For every occupied slot j of rank r (slotmap[r][j] = e >= 0) the slot receives the W bytes of
 * e's main instance; an empty slot keeps its bytes.
 */
void oracle_replica_pull(const oracle_config* c, const int32_t* main_rank, const int32_t* slotmap,
                         int64_t W, const uint8_t* main_params, uint8_t* replica_buf) {
  const int R = c->nodes * c->gpus_per_node, N = c->slots_per_rank;
  const int e_loc = oracle_e_loc(c, main_rank);
  for (int r = 0; r < R; ++r)
    for (int j = 0; j < N; ++j) {
      const int e = slotmap[(size_t)r * N + j];
      if (e < 0) continue;
      const uint8_t* src = main_params + ((size_t)main_rank[e] * e_loc + main_local_index(main_rank, e)) * W;
      uint8_t* dst = replica_buf + ((size_t)r * N + j) * W;
      for (int64_t i = 0; i < W; ++i) dst[i] = src[i];
    }
}

/*
 * O12 -- replica gradient return (same subsection, backward direction).  The slot that held the
 * parameters now holds the replica's gradient; it goes to the gradient-accumulation buffer of
 * the expert's main rank, which is partitioned by SOURCE rank into R regions of E_loc blocks:
 *   grad_acc [R main][R source][E_loc][W];  grad_acc[main(e)][r][l(e)] = replica_buf[r][j].
 * Everything else in grad_acc keeps its bytes (the copy does not accumulate: each region has
 * exactly one writer, and the main rank sums its regions later).
 */
void oracle_replica_grad_return(const oracle_config* c, const int32_t* main_rank,
                                const int32_t* slotmap, int64_t W, const uint8_t* replica_buf,
                                uint8_t* grad_acc) {
  const int R = c->nodes * c->gpus_per_node, N = c->slots_per_rank;
  const int e_loc = oracle_e_loc(c, main_rank);
  for (int r = 0; r < R; ++r)
    for (int j = 0; j < N; ++j) {
      const int e = slotmap[(size_t)r * N + j];
      if (e < 0) continue;
      const uint8_t* src = replica_buf + ((size_t)r * N + j) * W;
      uint8_t* dst = grad_acc + (((size_t)main_rank[e] * R + r) * e_loc + main_local_index(main_rank, e)) * W;
      for (int64_t i = 0; i < W; ++i) dst[i] = src[i];
    }
}
