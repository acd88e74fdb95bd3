"""Seeded synthetic workloads: proposal trees, accepted nodes and layer tensors.

This module only draws inputs.  It holds none of the method's arithmetic and is
the one module that both the CPU oracle's tests and the CUDA path's tests and
benchmark read, so that both sides see the same values.

The five workloads mirror the shapes the paper serves (Section VI-A: draft
trees from an MTP/EAGLE drafter with top-k 4 and depth up to 8, 32-128 nodes,
32 state heads of 128x128 fp32 state):

=====  ====  ===  ====  =====  ======  =====  ================================
name   B     H    T     dk=dv  rule    dtype  tree
=====  ====  ===  ====  =====  ======  =====  ================================
c1     1     4    15    64     gated   f32    full binary tree of depth 3
c2     1     16   63    128    gated   bf16   frontier growth, depth <= 8
c3     32    32   64    128    gated   bf16   level widths <= 10, depth 6
c4     16    32   64    128    delta   bf16   frontier growth, depth <= 8
c5     128   32   128   128    gated   bf16   spine to depth 8 + growth, L=48
=====  ====  ===  ====  =====  ======  =====  ================================

Distributions (second parameter of N(.,.) is the standard deviation):
q, v ~ N(0,1)/8; k ~ N(0,1) (c1: /8, not normalised; bf16 workloads:
L2-normalised in fp32 and then rounded to bf16); alpha = sigmoid(N(3,0.5)) for
c1 and sigmoid(N(4,1)) otherwise; beta = sigmoid(N(0,1)) (delta rule only);
S_pre ~ N(0,0.1) for c1 and N(0,0.05) otherwise.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

GATED = 0
DELTA = 1
F32 = 0
BF16 = 1


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    T: int
    dk: int
    dv: int
    rule: int          # GATED / DELTA
    qkv_dtype: int     # F32 / BF16
    L: int             # recurrent layers stacked back to back
    tol: float         # max relative L2 error allowed against the oracle
    seed: int
    alpha_mu: float
    alpha_sd: float
    s_sd: float
    tree: str          # generator name

    @property
    def rule_name(self) -> str:
        return "delta" if self.rule == DELTA else "gated"

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.qkv_dtype == BF16 else torch.float32


WORKLOADS = {
    "c1": Workload("c1", 1, 4, 15, 64, 64, GATED, F32, 1, 1e-5, 0, 3.0, 0.5, 0.1, "binary"),
    "c2": Workload("c2", 1, 16, 63, 128, 128, GATED, BF16, 1, 2e-3, 1, 4.0, 1.0, 0.05, "frontier"),
    "c3": Workload("c3", 32, 32, 64, 128, 128, GATED, BF16, 1, 2e-3, 2, 4.0, 1.0, 0.05, "levels"),
    "c4": Workload("c4", 16, 32, 64, 128, 128, DELTA, BF16, 1, 2e-3, 3, 4.0, 1.0, 0.05, "frontier"),
    "c5": Workload("c5", 128, 32, 128, 128, 128, GATED, BF16, 48, 2e-3, 4, 4.0, 1.0, 0.05, "spine"),
}


def workload(name: str, **overrides) -> Workload:
    """Look a workload up by name; keyword overrides shrink it for tests."""
    return replace(WORKLOADS[name], **overrides)


# --------------------------------------------------------------------------
# Trees.  Every generator returns int32 parent[T] with -1 <= parent[i] < i.
# --------------------------------------------------------------------------
def tree_binary(T: int) -> np.ndarray:
    """Heap-ordered binary tree: parent[i] = (i-1)//2, one root."""
    par = np.array([(i - 1) // 2 for i in range(T)], dtype=np.int32)
    par[0] = -1
    return par


def tree_chain(T: int) -> np.ndarray:
    return np.arange(-1, T - 1, dtype=np.int32)


def tree_frontier(T: int, rng: np.random.Generator, max_depth: int = 8,
                  spine: int = 0) -> np.ndarray:
    """Frontier growth with 1-4 children per expanded node, depth <= max_depth.

    Start from one root (or a spine of ``spine`` nodes at depths 0..spine-1);
    pop a uniformly random unexpanded node of depth < max_depth, append
    c ~ U{1..4} children (index = creation order, so parent < child), until T
    nodes exist.
    """
    par = [-1]
    depth = [0]
    for s in range(1, min(spine, T)):
        par.append(s - 1)
        depth.append(s)
    frontier = [i for i in range(len(par)) if depth[i] < max_depth]
    while len(par) < T:
        if not frontier:
            frontier = [i for i in range(len(par)) if depth[i] < max_depth]
        p = frontier.pop(int(rng.integers(len(frontier))))
        c = int(rng.integers(1, 5))
        for _ in range(c):
            if len(par) >= T:
                break
            par.append(p)
            depth.append(depth[p] + 1)
            if depth[-1] < max_depth:
                frontier.append(len(par) - 1)
    return np.array(par, dtype=np.int32)


def tree_levels(T: int, rng: np.random.Generator, n_levels: int = 7,
                max_width: int = 10) -> np.ndarray:
    """Draft-style top-k forest: levels 0..n_levels-1 of width <= max_width.

    Level 0 nodes are root children.  The children of level l are dealt to the
    level l-1 nodes cyclically, c ~ Geometric(0.5) on {0,1,2,...} at a time.
    """
    widths = [max_width] * n_levels
    excess = sum(widths) - T
    if excess < 0:
        raise ValueError("T too large for the level budget")
    while excess > 0:
        l = int(rng.integers(n_levels))
        if widths[l] > 1:
            widths[l] -= 1
            excess -= 1
    par = [-1] * widths[0]
    prev = list(range(widths[0]))
    for l in range(1, n_levels):
        cur = []
        pi = 0
        while len(cur) < widths[l]:
            c = int(rng.geometric(0.5)) - 1
            for _ in range(c):
                if len(cur) >= widths[l]:
                    break
                par.append(prev[pi % len(prev)])
                cur.append(len(par) - 1)
            pi += 1
        prev = cur
    return np.array(par, dtype=np.int32)


def node_depths(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int32)
    for i, p in enumerate(parent):
        d[i] = 0 if p < 0 else d[p] + 1
    return d


def accepted_walk(parent: np.ndarray, rng: np.random.Generator) -> int:
    """Random root-to-leaf walk: uniform root child, then uniform child."""
    T = len(parent)
    kids = [[] for _ in range(T)]
    roots = []
    for i, p in enumerate(parent):
        (roots if p < 0 else kids[p]).append(i)
    a = roots[int(rng.integers(len(roots)))]
    while kids[a]:
        a = kids[a][int(rng.integers(len(kids[a])))]
    return a


def accepted_prefix(parent: np.ndarray, rng: np.random.Generator, max_len: int) -> int:
    """Accepted prefix length L ~ U{0..max_len}; L = 0 -> -1, else a uniformly
    random node of depth L-1 (falls back to the deepest level that exists)."""
    L = int(rng.integers(0, max_len + 1))
    if L == 0:
        return -1
    d = node_depths(parent)
    want = min(L - 1, int(d.max()))
    cand = np.nonzero(d == want)[0]
    return int(cand[int(rng.integers(len(cand)))])


def make_trees(wl: Workload, per_request: bool = True):
    """Return ``(parents int32 [n_trees, T], accepted int32 [B])``."""
    rng = np.random.Generator(np.random.Philox(key=wl.seed + 1000))
    n_trees = wl.B if per_request else 1
    parents = np.zeros((n_trees, wl.T), dtype=np.int32)
    for t in range(n_trees):
        if wl.tree == "binary":
            parents[t] = tree_binary(wl.T)
        elif wl.tree == "chain":
            parents[t] = tree_chain(wl.T)
        elif wl.tree == "frontier":
            parents[t] = tree_frontier(wl.T, rng)
        elif wl.tree == "spine":
            parents[t] = tree_frontier(wl.T, rng, spine=min(9, wl.T))
        elif wl.tree == "levels":
            parents[t] = tree_levels(wl.T, rng)
        else:
            raise ValueError(wl.tree)
    accepted = np.zeros(wl.B, dtype=np.int32)
    for b in range(wl.B):
        par = parents[b if per_request else 0]
        if wl.tree == "levels":
            accepted[b] = accepted_prefix(par, rng, 6)
        else:
            accepted[b] = accepted_walk(par, rng)
    return parents, accepted


def tree_stats(parents: np.ndarray, accepted: np.ndarray) -> dict:
    """Shape statistics printed beside benchmark numbers."""
    depths = np.stack([node_depths(p) for p in parents])
    T = parents.shape[1]
    acc_len = []
    for b, a in enumerate(accepted):
        d = depths[b if parents.shape[0] > 1 else 0]
        acc_len.append(0 if a < 0 else int(d[a]) + 1)
    return {
        "max_depth": int(depths.max()),
        "mean_ancestors": float(depths.mean()),
        "mask_density": float((depths + 1).sum() / (parents.shape[0] * T * T)),
        "mean_accepted_len": float(np.mean(acc_len)),
        "accepted_none": int(sum(1 for a in accepted if a < 0)),
    }


# --------------------------------------------------------------------------
# Tensors.
# --------------------------------------------------------------------------
def make_tensors(wl: Workload, layer: int = 0, device: str = "cpu") -> dict:
    """Draw one layer's tensors in the library layout.

    ``S_pre`` f32 [B,H,dv,dk]; ``q,k`` [B,H,T,dk]; ``v`` [B,H,T,dv] in the
    workload's dtype; ``alpha`` f32 [B,H,T]; ``beta`` f32 [B,H,T] or None.
    Values depend on (workload seed, layer, device type): the CPU and CUDA
    generators are different streams of the same distributions.
    """
    g = torch.Generator(device=device)
    g.manual_seed(wl.seed * 1000003 + layer * 7919 + 17)
    B, H, T, dk, dv = wl.B, wl.H, wl.T, wl.dk, wl.dv

    def randn(*shape):
        return torch.randn(*shape, generator=g, device=device, dtype=torch.float32)

    dt = wl.torch_dtype
    S_pre = randn(B, H, dv, dk) * wl.s_sd
    q = (randn(B, H, T, dk) / 8).to(dt)
    k = randn(B, H, T, dk)
    if wl.qkv_dtype == BF16:
        k = k / k.norm(dim=-1, keepdim=True)
    else:
        k = k / 8
    k = k.to(dt)
    v = (randn(B, H, T, dv) / 8).to(dt)
    alpha = torch.sigmoid(wl.alpha_mu + wl.alpha_sd * randn(B, H, T))
    beta = torch.sigmoid(randn(B, H, T)) if wl.rule == DELTA else None
    return {"S_pre": S_pre.contiguous(), "q": q.contiguous(), "k": k.contiguous(),
            "v": v.contiguous(), "alpha": alpha.contiguous(),
            "beta": None if beta is None else beta.contiguous()}


def make_conv_inputs(wl: Workload, layer: int = 0, device: str = "cpu", W: int = 4) -> dict:
    """Draw one layer's front-end inputs: projected activations ``x`` [B,T,C] and context rows
    ``ctx`` [B,W-1,C] in the workload's dtype (C = H(2dk+dv), channel order q|k|v), a depthwise
    filter ``weight`` f32 [C,W] and ``bias`` f32 [C], gate pre-activations ``gate_a``, ``gate_b``
    [B,T,H] in the workload's dtype, and the per-head gate parameters ``A_log``, ``dt_bias`` f32 [H]
    drawn so that the decay lands in the same range as ``make_tensors`` draws it directly."""
    g = torch.Generator(device=device)
    g.manual_seed(wl.seed * 1000003 + layer * 7919 + 4241)
    B, H, T, dk, dv = wl.B, wl.H, wl.T, wl.dk, wl.dv
    C = H * (2 * dk + dv)

    def randn(*shape):
        return torch.randn(*shape, generator=g, device=device, dtype=torch.float32)

    def rand(*shape):
        return torch.rand(*shape, generator=g, device=device, dtype=torch.float32)

    dt = wl.torch_dtype
    return {"x": randn(B, T, C).to(dt).contiguous(), "ctx": randn(B, W - 1, C).to(dt).contiguous(),
            "weight": (randn(C, W) / W ** 0.5).contiguous(), "bias": (0.1 * randn(C)).contiguous(),
            "gate_a": randn(B, T, H).to(dt).contiguous(), "gate_b": randn(B, T, H).to(dt).contiguous(),
            "A_log": (-2.0 + 2.5 * rand(H)).contiguous(), "dt_bias": (-3.0 + 2.0 * rand(H)).contiguous()}


def to_f64(t):
    """Widen exactly the values the GPU receives to float64 numpy."""
    if t is None:
        return None
    return t.detach().to("cpu").to(torch.float64).numpy()
