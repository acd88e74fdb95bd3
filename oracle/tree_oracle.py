"""CPU fp64 oracle for tree verification of gated (delta-rule) linear attention.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product path never does, and
this module imports nothing from the product package.  numpy only, float64
throughout, no blocking, fusion or reordering beyond what the cited passage
states.

Notation is the paper's (Section II-B Eq. 1, Section IV-A Table II):
one state head keeps ``S`` of shape ``[dk, dv]``; node ``i`` of the proposal
tree has parent ``pi(i)``; ``parent[i] == -1`` marks a child of the virtual
root whose state is the committed ``S_pre`` (Table II gives a root child the
parent index 0 and defines the state of index 0 as S_pre).  Nodes are indexed parent before child (Section IV-A,
text after Theorem 1).  Row ``i`` of ``Q, K`` is ``q_i, k_i`` (``[T, dk]``),
row ``i`` of ``V, U, O`` is ``v_i, u_i, o_i`` (``[T, dv]``); ``gamma`` is the
decay gate and ``beta`` the write gate (``[T]``).

Two update rules are covered:

* ``"delta"``  -- Eq. 1 / Table II "Sequential rule":
      S~_i = gamma_i S_pi(i);  u_i = beta_i (v_i - S~_i^T k_i);
      S_i  = S~_i + k_i u_i^T;  o_i = S_i^T q_i
* ``"gated"``  -- the same rule with the correction replaced by the value,
      u_i = v_i  (gated linear attention S_i = gamma_i S_pi(i) + k_i v_i^T;
      in Theorem 1 this is G = 0, U = V).

Pins (tests/test_oracle_pins.py): a hand-worked example, Theorem 1 evaluated
densely, Eq. 4, Lemma 3, Eq. 10, the masked linear-attention special case,
delta-rule retrieval, beta = 0, chain = sequential decoding, sibling
independence, brute force over every tree of up to five nodes, and, for the
batch wrappers at the end of this file, the hand examples laid out in the
library's transposed state layout with dk != dv and per-request trees.
"""
from __future__ import annotations

import numpy as np

GATED = "gated"
DELTA = "delta"


# --------------------------------------------------------------------------
# Tree metadata (Section IV-A Table II: Anc(i), d, M^-, M^+; Section IV-C
# "Round-level topology preprocessing").
# --------------------------------------------------------------------------
def check_parent(parent) -> np.ndarray:
    """Validate parent-before-child indexing: -1 <= parent[i] < i."""
    parent = np.asarray(parent, dtype=np.int64)
    if parent.ndim != 1:
        raise ValueError("parent must be one-dimensional")
    for i, p in enumerate(parent):
        if p < -1 or p >= i:
            raise ValueError(f"parent[{i}]={p} violates -1 <= parent[i] < i")
    return parent


def strict_ancestors(parent, i: int) -> list[int]:
    """Anc(i): the strict draft ancestors of node i, root side first."""
    chain = []
    p = int(parent[i])
    while p >= 0:
        chain.append(p)
        p = int(parent[p])
    chain.reverse()
    return chain


def path_to(parent, i: int) -> list[int]:
    """P(i) = Anc(i) + {i} in topological order (Section IV-D, accepted path)."""
    return strict_ancestors(parent, i) + [int(i)]


def tree_metadata(parent):
    """Strict-ancestor sets as 128-bit masks, depths and the maximum depth.

    Returns ``(anc, depth, d)``: ``anc`` is uint64 ``[T, 2]`` with bit
    ``j & 63`` of word ``j >> 6`` set iff ``j in Anc(i)`` (row ``i`` of M^-);
    ``depth[i] = |Anc(i)|`` (0 for a root child); ``d = max_i depth[i]``
    (Table II).  T <= 128.
    """
    parent = check_parent(parent)
    T = len(parent)
    if T > 128:
        raise ValueError("T <= 128")
    anc = np.zeros((T, 2), dtype=np.uint64)
    depth = np.zeros(T, dtype=np.int32)
    for i in range(T):
        A = strict_ancestors(parent, i)
        depth[i] = len(A)
        for j in A:
            anc[i, j >> 6] |= np.uint64(1) << np.uint64(j & 63)
    d = int(depth.max()) if T else 0
    return anc, depth, d


def ancestor_masks(parent):
    """Dense M^- and M^+ = M^- + I as float64 ``[T, T]`` (Table II)."""
    parent = check_parent(parent)
    T = len(parent)
    Mm = np.zeros((T, T))
    for i in range(T):
        for j in strict_ancestors(parent, i):
            Mm[i, j] = 1.0
    return Mm, Mm + np.eye(T)


def accepted_path(parent, a: int):
    """Accepted-path indices for terminal node ``a`` (Section IV-D).

    ``a == -1`` means that no draft token was accepted: empty path.
    """
    if a < 0:
        return []
    return path_to(parent, a)


# --------------------------------------------------------------------------
# Sequential rule on one root-to-node path (Eq. 1 with S_{t-1} -> S_pi(i)).
# --------------------------------------------------------------------------
def _step(S, k, v, gamma, beta, rule):
    """One application of the sequential rule; returns (S_i, u_i)."""
    S_tilde = gamma * S
    if rule == DELTA:
        u = beta * (v - S_tilde.T @ k)
    elif rule == GATED:
        u = v.copy()
    else:
        raise ValueError(rule)
    return S_tilde + np.outer(k, u), u


def walk_node(S_pre, Q, K, V, gamma, beta, parent, i, rule):
    """Walk the root-to-node path of node i from S_pre, step by step.

    Returns ``(o_i, u_i, S_i)``.  Touches only rows on the path.
    """
    S = np.array(S_pre, dtype=np.float64)
    u = None
    for r in path_to(parent, i):
        b = 0.0 if beta is None else float(beta[r])
        S, u = _step(S, K[r], V[r], float(gamma[r]), b, rule)
    return S.T @ Q[i], u, S


def verify_walk(S_pre, Q, K, V, gamma, beta, parent, rule):
    """Outputs and corrections of every node, each by its own path walk.

    Returns ``(O [T, dv], U [T, dv])``.
    """
    T, dv = V.shape
    O = np.zeros((T, dv))
    U = np.zeros((T, dv))
    for i in range(T):
        O[i], U[i], _ = walk_node(S_pre, Q, K, V, gamma, beta, parent, i, rule)
    return O, U


def verify_memo(S_pre, Q, K, V, gamma, beta, parent, rule):
    """Same results as :func:`verify_walk`, keeping each node's state.

    Node i starts from the stored state of its parent, which is the state the
    path walk reaches after the same operations in the same order, so the
    results are bit-identical to the per-node walk.  Used where the per-node
    walk is too slow (timing, large parity cases).
    """
    T, dv = V.shape
    S_pre = np.array(S_pre, dtype=np.float64)
    states = [None] * T
    O = np.zeros((T, dv))
    U = np.zeros((T, dv))
    for i in range(T):
        p = int(parent[i])
        S_par = S_pre if p < 0 else states[p]
        b = 0.0 if beta is None else float(beta[i])
        states[i], U[i] = _step(S_par, K[i], V[i], float(gamma[i]), b, rule)
        O[i] = states[i].T @ Q[i]
    return O, U, states


def commit_walk(S_pre, K, V, gamma, beta, parent, a, rule):
    """State that must persist after accepting terminal node ``a``.

    The state reached at the end of the accepted path (Section IV-D: Lemma 1
    "reconstructs the only state that must persist"); ``a == -1`` keeps S_pre.
    """
    S = np.array(S_pre, dtype=np.float64)
    for r in accepted_path(parent, a):
        b = 0.0 if beta is None else float(beta[r])
        S, _ = _step(S, K[r], V[r], float(gamma[r]), b, rule)
    return S


# --------------------------------------------------------------------------
# The closed form, written out densely (Theorem 1, Eq. 2; Table II).
# A second formulation used to pin the walk; not used for parity.
# --------------------------------------------------------------------------
def path_decay(gamma, parent):
    """P_i = prod_{r in Anc(i) + {i}} gamma_r (Table II)."""
    T = len(parent)
    P = np.zeros(T)
    for i in range(T):
        P[i] = np.prod([gamma[r] for r in path_to(parent, i)])
    return P


def closed_form_factors(Q, K, gamma, beta, parent):
    """(P, G, C) of Table II with D_P^{-1} written literally."""
    P = path_decay(gamma, parent)
    Mm, Mp = ancestor_masks(parent)
    DP = np.diag(P)
    DPinv = np.diag(1.0 / P)
    G = np.diag(beta) @ DP @ ((K @ K.T) * Mm) @ DPinv
    C = DP @ ((Q @ K.T) * Mp) @ DPinv
    return P, G, C


def verify_closed_form(S_pre, Q, K, V, gamma, beta, parent, rule):
    """O and U from Theorem 1 (Eq. 2) and Lemma 2 (Eq. 5), dense solve."""
    T = len(parent)
    if rule == GATED:
        P = path_decay(gamma, parent)
        _, Mp = ancestor_masks(parent)
        C = np.diag(P) @ ((Q @ K.T) * Mp) @ np.diag(1.0 / P)
        U = V.copy()
    else:
        P, G, C = closed_form_factors(Q, K, gamma, beta, parent)
        R = np.diag(beta) @ (V - np.diag(P) @ K @ S_pre)
        U = np.linalg.solve(np.eye(T) + G, R)
    O = np.diag(P) @ Q @ S_pre + C @ U
    return O, U


def neumann_solve(G, R, d):
    """U = sum_{m=0}^{d} (-G)^m R by the rounds of Eq. 8 (Lemma 3)."""
    Z = R.copy()
    U = R.copy()
    for _ in range(d):
        Z = -G @ Z
        U = U + Z
    return U


def commit_factored(S_pre, K, U, gamma, parent, a):
    """S_new = P_a S_pre + (D_a K_a)^T U_a  (Eq. 10)."""
    if a < 0:
        return np.array(S_pre, dtype=np.float64)
    path = accepted_path(parent, a)
    P = path_decay(gamma, parent)
    Da = np.diag([P[a] / P[j] for j in path])
    Ka = K[path]
    Ua = U[path]
    return P[a] * S_pre + (Da @ Ka).T @ Ua


# --------------------------------------------------------------------------
# Batched drivers in the library's memory layout.
#
# The library keeps the state transposed, S^ = S^T with shape [dv, dk] (the
# serving cache layout "[H, dv, dk]" of Section IV-D) and tensors stacked as
# [B, H, ...].  These wrappers only reshape, transpose and loop.
# --------------------------------------------------------------------------
def _tree_of(parents, b):
    parents = np.asarray(parents)
    return parents[0] if parents.shape[0] == 1 else parents[b]


def verify_batch(S_hat, q, k, v, gamma, beta, parents, rule, memo=True,
                 items=None):
    """Run the walk for every (b, h) (or the listed ``items``).

    ``S_hat [B,H,dv,dk]``, ``q,k [B,H,T,dk]``, ``v [B,H,T,dv]``,
    ``gamma, beta [B,H,T]`` (beta may be None for ``"gated"``),
    ``parents [n_trees,T]`` with n_trees in {1, B}.  Returns dict
    ``(b,h) -> (O, U)``.
    """
    B, H = q.shape[:2]
    out = {}
    todo = items if items is not None else [(b, h) for b in range(B) for h in range(H)]
    for (b, h) in todo:
        par = _tree_of(parents, b)
        S = np.asarray(S_hat[b, h], dtype=np.float64).T
        bt = None if beta is None else np.asarray(beta[b, h], dtype=np.float64)
        args = (S, np.asarray(q[b, h], np.float64), np.asarray(k[b, h], np.float64),
                np.asarray(v[b, h], np.float64), np.asarray(gamma[b, h], np.float64),
                bt, par, rule)
        if memo:
            O, U, _ = verify_memo(*args)
        else:
            O, U = verify_walk(*args)
        out[(b, h)] = (O, U)
    return out


def commit_batch(S_hat, k, v, gamma, beta, parents, accepted, rule, items=None):
    """Committed states in the library layout: dict ``(b,h) -> S^_new [dv,dk]``."""
    B, H = k.shape[:2]
    out = {}
    todo = items if items is not None else [(b, h) for b in range(B) for h in range(H)]
    for (b, h) in todo:
        par = _tree_of(parents, b)
        S = np.asarray(S_hat[b, h], dtype=np.float64).T
        bt = None if beta is None else np.asarray(beta[b, h], dtype=np.float64)
        Sn = commit_walk(S, np.asarray(k[b, h], np.float64), np.asarray(v[b, h], np.float64),
                         np.asarray(gamma[b, h], np.float64), bt, par, int(accepted[b]), rule)
        out[(b, h)] = Sn.T.copy()
    return out
