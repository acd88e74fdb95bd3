"""CPU oracle for the batch-wide utility allocation (verification-budget selector).

TEST INFRASTRUCTURE ONLY (see tree_oracle.py): numpy, imported only by tests, the smoke check and
the benchmark's CPU-baseline leg.

What it computes (Section V-A, "Batch-wide utility allocation").  Every request b brings a
candidate tree of Tc nodes (parent map pi_b, node 0 is the tree's root, parent -1) and the
drafter's conditional probability p(u | pi(u)) of every node.  The utility of node v is the
drafter's probability of reaching it along its whole path,

    rho(v) = prod_{u in P(v)} p(u | pi(u)),          i.e. rho(v) = rho(pi(v)) * p(v | pi(v)),

the root of every tree is kept, and the remaining capacity (`budget` nodes in total over the
batch) is filled with the highest-rho nodes of the whole batch.  Since rho cannot grow along a
path, the kept nodes of a request form a prefix-closed subtree.  A count per request gives its
budget q_b; the kept nodes are packed request by request, in their original order, into one flat
forest (Section V-B), with parents renumbered locally.

Precision and ties (the paper is silent; fixed here): rho is computed in float32 by the
recurrence above (one rounding per edge, parent before child), which is what decides the
selection; equal rho are ordered by (request, node) index, lower first.  Roots rank above
everything.  A non-root child of the virtual root (parent -1 at index > 0) is a sibling tree of
the same request and is scored like any node (rho = its own p).
"""
from __future__ import annotations

import numpy as np


def rho_f32(parent, p):
    """rho [Tc] float32 for one request: rho_i = rho_parent * p_i in float32, rho_root = p_0."""
    parent = np.asarray(parent, dtype=np.int64)
    p = np.asarray(p, dtype=np.float32)
    rho = np.zeros(len(parent), dtype=np.float32)
    for i in range(len(parent)):
        j = int(parent[i])
        if not -1 <= j < i:
            raise ValueError("parent[i] must be in [-1, i)")
        rho[i] = p[i] if j < 0 else np.float32(rho[j] * p[i])
    return rho


def select(parents, probs, budget):
    """parents int [B, Tc], probs float32 [B, Tc], budget >= B  ->  dict with
    rho f32 [B,Tc], keep bool [B,Tc], counts [B], offsets [B+1], parent_packed [B,Tc] (local
    indices, -1 = root child or padding), node_id [budget] (b*Tc + i of each packed row, -1 past
    the forest)."""
    parents = np.asarray(parents, dtype=np.int64)
    B, Tc = parents.shape
    budget = min(int(budget), B * Tc)
    if budget < B:
        raise ValueError("the budget must keep the root of every tree")
    rho = np.stack([rho_f32(parents[b], probs[b]) for b in range(B)])
    order = []  # (is_root first, rho descending, global index ascending)
    for b in range(B):
        for i in range(Tc):
            order.append((0 if i == 0 else 1, -float(rho[b, i]), b * Tc + i))
    order.sort()
    keep = np.zeros((B, Tc), dtype=bool)
    for _, _, g in order[:budget]:
        keep[g // Tc, g % Tc] = True
    counts = keep.sum(axis=1).astype(np.int32)
    offsets = np.zeros(B + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    parent_packed = np.full((B, Tc), -1, dtype=np.int32)
    node_id = np.full(budget, -1, dtype=np.int32)
    for b in range(B):
        new = -np.ones(Tc, dtype=np.int64)
        new[keep[b]] = np.arange(counts[b])
        for i in np.nonzero(keep[b])[0]:
            j = parents[b, i]
            parent_packed[b, new[i]] = -1 if j < 0 else new[j]
            node_id[offsets[b] + new[i]] = b * Tc + i
    return {"rho": rho, "keep": keep, "counts": counts, "offsets": offsets,
            "parent_packed": parent_packed, "node_id": node_id}
