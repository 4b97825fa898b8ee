"""Plain Python restatement of the frontend's graph partitioning (Section IV: Eq. 1, Definitions 1-3, Algorithm 1).

TEST INFRASTRUCTURE ONLY: imported by tests/ (and by nothing in the product path).

Follows the algorithm's steps in the paper's order with sets and dicts, recomputing everything from
scratch after each merge. Choices the paper leaves open are read as the C library documents them:
affix candidates are the nodes adjacent to v in the current quotient graph; ties go to the smaller
smallest-member id.
"""
from __future__ import annotations

import math


def op_weight(loop_extents, c=1.0, b=0.0):
    """Eq. 1: w_v = c * prod_l log(s_l) + b."""
    prod = 1.0
    for s in loop_extents:
        prod *= math.log(s)
    return c * prod + b


def topological_stage(nodes, edges):
    """Definition 2: length of the longest path from a root to v, roots at stage 1."""
    preds = {v: [u for (u, w) in edges if w == v] for v in nodes}
    memo = {}

    def ts(v):
        if v not in memo:
            memo[v] = 1 if not preds[v] else 1 + max(ts(u) for u in preds[v])
        return memo[v]

    return {v: ts(v) for v in nodes}


def affix_set(v, nodes, edges, ts):
    """Definition 3: nodes connected to v whose stage is ts_v + 1 or ts_v - 1."""
    adjacent = {w for (u, w) in edges if u == v} | {u for (u, w) in edges if w == v}
    return {u for u in adjacent if abs(ts[u] - ts[v]) == 1}


def cluster(weights, edges, threshold):
    """Algorithm 1. Returns a list: subgraph index of every node, subgraphs numbered by smallest member."""
    groups = {i: frozenset([i]) for i in range(len(weights))}      # hyper node id -> members
    w = {i: float(weights[i]) for i in range(len(weights))}
    node_edges = set((int(a), int(b)) for a, b in edges)
    cand = set(groups)

    def quotient_edges():
        owner = {m: g for g, ms in groups.items() for m in ms}
        return {(owner[a], owner[b]) for (a, b) in node_edges if owner[a] != owner[b]}

    while cand:
        q = quotient_edges()
        ts = topological_stage(list(groups), q)
        v = min(cand, key=lambda g: (-w[g], min(groups[g])))                 # heaviest
        aff = affix_set(v, list(groups), q, ts)
        u = min(aff, key=lambda g: (w[g], min(groups[g]))) if aff else None  # lightest of the affix set
        if u is not None and w[v] + w[u] < threshold:
            groups[v] = groups[v] | groups[u]
            w[v] += w[u]
            del groups[u], w[u]
            cand.discard(u)
        else:
            cand.discard(v)
    order = sorted(groups, key=lambda g: min(groups[g]))
    out = [0] * len(weights)
    for idx, g in enumerate(order):
        for m in groups[g]:
            out[m] = idx
    return out


def is_acyclic_partition(assign, edges):
    """Definition 1, checked directly: no two parts with paths in both directions between them."""
    n = len(assign)
    reach = [[False] * n for _ in range(n)]
    for a, b in edges:
        reach[a][b] = True
    for k in range(n):
        for i in range(n):
            if reach[i][k]:
                for j in range(n):
                    if reach[k][j]:
                        reach[i][j] = True
    parts = sorted(set(assign))
    for i in parts:
        for j in parts:
            if i >= j:
                continue
            fwd = any(reach[u][v] for u in range(n) for v in range(n) if assign[u] == i and assign[v] == j)
            bwd = any(reach[v][u] for u in range(n) for v in range(n) if assign[u] == i and assign[v] == j)
            if fwd and bwd:
                return False
    return True
