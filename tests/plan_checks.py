"""Independent numpy checks of a plan in the library's output layout.

Used on the oracle's output (CPU tests) and on the CUDA library's output (GPU
tests, at any size).  Written from the paper's constraints C1-C5 and the
output contract; imports neither the oracle nor the CUDA binding.
"""
from __future__ import annotations

import numpy as np


def instance_tables(nodes, gpus_per_node, experts, slots, main_rank, replica_map):
    """(e_loc, s_phys, expert_of_instance [P]) for one plan's replica_map [R][N_slot]."""
    R = nodes * gpus_per_node
    main_rank = np.asarray(main_rank)
    e_loc = int(np.bincount(main_rank, minlength=R).max())
    s_phys = e_loc + slots
    inst_expert = np.full(R * s_phys, -1, np.int64)
    nxt = np.zeros(R, np.int64)
    for e in range(experts):              # ascending e -> local index in order
        r = main_rank[e]
        inst_expert[r * s_phys + nxt[r]] = e
        nxt[r] += 1
    for r in range(R):
        for j in range(slots):
            inst_expert[r * s_phys + e_loc + j] = replica_map[r][j]
    return e_loc, s_phys, inst_expert


def check_plan(nodes, gpus_per_node, experts, slots, top_k, main_rank, token_bytes, expert_bytes,
               ids, replica_map, token_replica, counts, offsets, instance_counts,
               rank_load=None):
    """Assert every structural property of ONE plan.  ids/token_replica: [R][T][k]."""
    M, G, E, N = nodes, gpus_per_node, experts, slots
    R = M * G
    main_rank = np.asarray(main_rank, np.int64)
    ids = np.asarray(ids).reshape(R, -1)
    tr = np.asarray(token_replica).reshape(R, -1)
    replica_map = np.asarray(replica_map).reshape(R, N)
    counts = np.asarray(counts, np.int64).reshape(R, R)
    offsets = np.asarray(offsets, np.int64).reshape(2, R, R + 1)
    e_loc, s_phys, inst_expert = instance_tables(M, G, E, N, main_rank, replica_map)
    P = R * s_phys
    instance_counts = np.asarray(instance_counts, np.int64).reshape(P)

    # C3 / C5 and slot hygiene: slots fill from 0, no expert twice on a rank, no replica of an
    # expert on its own main rank.
    for r in range(R):
        row = replica_map[r]
        filled = row >= 0
        assert (row[filled] < E).all()
        if N:
            assert not (np.diff(filled.astype(int)) > 0).any(), "replica slots must fill from slot 0"
        assert len(set(row[filled].tolist())) == filled.sum(), "expert twice on one rank"
        assert (main_rank[row[filled]] != r).all(), "replica on the expert's main rank"

    valid = (ids >= 0) & (ids < E)
    # every assignment keeps its logical expert and lands on an instance hosting it (C2)
    assert (tr[~valid] == -1).all()
    assert (tr[valid] >= 0).all() and (tr[valid] < P).all()
    assert (inst_expert[tr[valid]] == ids[valid]).all(), "assigned instance does not host the expert"

    # instance histogram of the outputs == U
    hist_p = np.bincount(tr[valid], minlength=P)
    assert (hist_p == instance_counts).all(), "instance_counts differ from the per-token output"

    # C1: per expert, instance loads sum to the histogram of the ids
    omega_e = np.bincount(ids[valid], minlength=E)
    per_expert = np.bincount(inst_expert[inst_expert >= 0], weights=instance_counts[inst_expert >= 0],
                             minlength=E).astype(np.int64)
    assert (per_expert == omega_e).all()

    # dispatch counts recounted from the per-token output
    src = np.broadcast_to(np.arange(R)[:, None], tr.shape)
    dst_rank = tr[valid] // s_phys
    recount = np.bincount(src[valid] * R + dst_rank, minlength=R * R).reshape(R, R)
    assert (recount == counts).all(), "dispatch_counts differ from the per-token output"
    # offsets are the exclusive scans with the total appended
    send = np.concatenate([np.zeros((R, 1), np.int64), np.cumsum(counts, axis=1)], axis=1)
    recv = np.concatenate([np.zeros((R, 1), np.int64), np.cumsum(counts.T, axis=1)], axis=1)
    assert (offsets[0] == send).all() and (offsets[1] == recv).all()
    # rank loads, recomputed three ways
    L = recount.sum(axis=0)
    assert (L == instance_counts.reshape(R, s_phys).sum(axis=1)).all()
    assert L.sum() == valid.sum()
    if rank_load is not None:
        assert (np.asarray(rank_load, np.int64).reshape(R) == L).all()

    # C4: a replica outside its main's domain needs 2*D*S_tok > W in ITS domain
    omega = np.stack([np.bincount(ids[s][valid[s]], minlength=E) for s in range(R)])
    D = omega.reshape(M, G, E).sum(axis=1)
    for r in range(R):
        for e in replica_map[r][replica_map[r] >= 0]:
            if main_rank[e] // G != r // G:
                assert 2 * int(D[r // G, e]) * token_bytes > expert_bytes, "C4 violated"

    # deterministic deal: inside a (source, expert) group the executing rank never decreases
    # along the flat index, and each instance's share is one contiguous run.
    for s in range(R):
        v = valid[s]
        e_s = ids[s][v]
        p_s = tr[s][v]
        order = np.argsort(e_s, kind="stable")
        e_sorted, p_sorted = e_s[order], p_s[order]
        same = e_sorted[1:] == e_sorted[:-1]
        assert (p_sorted[1:][same] >= p_sorted[:-1][same]).all(), "deal order is not ascending"
    return dict(e_loc=e_loc, s_phys=s_phys, L=L, omega=omega, D=D, inst_expert=inst_expert)


def objective(nodes, gpus_per_node, main_rank, token_bytes, expert_bytes, c_intra, c_inter, t_ffn,
              x, q):
    """Eq. (formulation): t_FFN*L_max + 2*S_tok*sum c q + sum c(main,r) W x, from dense x, q."""
    G = gpus_per_node
    R = nodes * G
    x = np.asarray(x, np.int64)
    q = np.asarray(q, np.int64)
    E = x.shape[0]
    dom = np.arange(R) // G
    C = np.where(dom[:, None] == dom[None, :], c_intra, c_inter).astype(np.int64)
    np.fill_diagonal(C, 0)
    L = q.sum(axis=(0, 1))
    t_comp = t_ffn * int(L.max())
    t_token = 2 * token_bytes * int((C[:, None, :] * q).sum())
    t_replica = 0
    for e in range(E):
        for r in range(R):
            if x[e, r] and r != main_rank[e]:
                t_replica += int(C[main_rank[e], r]) * expert_bytes
    return t_comp, t_token, t_replica


def dispatch_positions_by_sorting(ranks, s_phys, token_replica):
    """Independent definition of the dispatch permutation with numpy.lexsort.

    send buffer of a source: ordered by (instance id, flat index) -- instance ids ascend with
    (rank, instance); receive buffer of a rank: ordered by (instance, source, flat index).
    Returns (send_pos, recv_pos, instance_offsets) for one plan; ignored ids (-1) get -1.
    """
    tr = np.asarray(token_replica, np.int64).reshape(ranks, -1)
    n = tr.shape[1]
    send = np.full(tr.shape, -1, np.int64)
    flat = np.arange(n)
    for s in range(ranks):
        ok = tr[s] >= 0
        order = np.lexsort((flat[ok], tr[s][ok]))
        pos = np.empty(order.size, np.int64)
        pos[order] = np.arange(order.size)
        send[s][ok] = pos
    recv = np.full(tr.shape, -1, np.int64)
    src = np.broadcast_to(np.arange(ranks)[:, None], tr.shape)
    fl = np.broadcast_to(flat[None, :], tr.shape)
    inst_off = np.zeros((ranks, s_phys + 1), np.int64)
    for r in range(ranks):
        sel = (tr >= 0) & (tr // s_phys == r)
        p, s_, f_ = tr[sel], src[sel], fl[sel]
        order = np.lexsort((f_, s_, p))
        pos = np.empty(order.size, np.int64)
        pos[order] = np.arange(order.size)
        recv[sel] = pos
        counts = np.bincount(p - r * s_phys, minlength=s_phys)
        inst_off[r, 1:] = np.cumsum(counts)
    return send, recv, inst_off
