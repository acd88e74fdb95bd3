"""Pins for the budget-selector oracle (batch-wide utility allocation, Section V-A)."""
import itertools

import numpy as np

from oracle import budget_oracle as bo


def rand_trees(B, Tc, rng):
    par = np.zeros((B, Tc), dtype=np.int64)
    for b in range(B):
        par[b, 0] = -1
        for i in range(1, Tc):
            par[b, i] = rng.integers(0, i)
    return par


def test_rho_is_the_product_along_the_path():
    rng = np.random.default_rng(0)
    par = rand_trees(1, 12, rng)[0]
    p = rng.uniform(0.05, 1.0, size=12).astype(np.float32)
    rho = bo.rho_f32(par, p)
    for i in range(12):
        prod, j = 1.0, i
        while j >= 0:
            prod *= float(p[j]); j = par[j]
        assert np.isclose(rho[i], prod, rtol=1e-6)
    # hand example in exact binary fractions: a chain 0-1-2 and a sibling 3 of node 1
    rho = bo.rho_f32([-1, 0, 1, 0], np.array([1.0, 0.5, 0.25, 0.75], dtype=np.float32))
    assert rho.tolist() == [1.0, 0.5, 0.125, 0.75]


def prefix_closed(par, keep):
    return all(par[i] < 0 or keep[par[i]] for i in np.nonzero(keep)[0])


def test_selection_is_prefix_closed_keeps_roots_and_fills_the_budget():
    rng = np.random.default_rng(1)
    for B, Tc, budget in ((3, 7, 9), (5, 16, 40), (4, 9, 4), (2, 5, 10), (2, 5, 99)):
        par = rand_trees(B, Tc, rng)
        p = rng.uniform(0.0, 1.0, size=(B, Tc)).astype(np.float32)
        r = bo.select(par, p, budget)
        K = min(budget, B * Tc)
        assert r["keep"].sum() == K and r["counts"].sum() == K and r["offsets"][-1] == K
        assert r["keep"][:, 0].all()
        for b in range(B):
            assert prefix_closed(par[b], r["keep"][b])
        # threshold property: every kept non-root scores at least as high as every dropped node
        nonroot = np.ones((B, Tc), bool); nonroot[:, 0] = False
        kept, dropped = r["rho"][r["keep"] & nonroot], r["rho"][~r["keep"]]
        if kept.size and dropped.size:
            assert kept.min() >= dropped.max()


def test_selection_maximises_the_retained_mass_brute_force():
    """Among all root-containing prefix-closed node sets of the budget's size, the selected set
    has the largest total rho (the paper's optimality claim), checked by enumeration."""
    rng = np.random.default_rng(2)
    for trial in range(6):
        B, Tc, budget = 2, 5, 6
        par = rand_trees(B, Tc, rng)
        p = rng.uniform(0.1, 0.95, size=(B, Tc)).astype(np.float32)
        r = bo.select(par, p, budget)
        rho = r["rho"].astype(np.float64).reshape(-1)
        flatpar = [(-1 if par[b, i] < 0 else b * Tc + par[b, i]) for b in range(B) for i in range(Tc)]
        roots = [b * Tc for b in range(B)]
        rest = [g for g in range(B * Tc) if g not in roots]
        best = -1.0
        for extra in itertools.combinations(rest, budget - B):
            s = set(roots) | set(extra)
            if all(flatpar[g] < 0 or flatpar[g] in s for g in s):
                best = max(best, sum(rho[g] for g in s))
        got = rho[r["keep"].reshape(-1)].sum()
        assert np.isclose(got, best, rtol=1e-12), (trial, got, best)


def test_ties_go_to_the_lower_index_and_packing_renumbers_parents():
    par = np.array([[-1, 0, 0, 1], [-1, 0, 1, 2]])
    p = np.array([[1.0, 0.5, 0.5, 1.0], [1.0, 0.5, 1.0, 1.0]], dtype=np.float32)
    # rho: request 0 = [1, .5, .5, .5]; request 1 = [1, .5, .5, .5]: six nodes tie at 0.5
    r = bo.select(par, p, 5)
    assert r["keep"].tolist() == [[True, True, True, True], [True, False, False, False]]
    assert r["counts"].tolist() == [4, 1] and r["offsets"].tolist() == [0, 4, 5]
    assert r["node_id"].tolist() == [0, 1, 2, 3, 4]
    r = bo.select(par, p, 7)
    assert r["keep"].tolist() == [[True, True, True, True], [True, True, True, False]]
    assert r["parent_packed"][1].tolist() == [-1, 0, 1, -1]
    # packing keeps the original order and maps parents through the renumbering
    par2 = np.array([[-1, 0, 0, 2, 2]])
    p2 = np.array([[1.0, 0.1, 0.9, 0.9, 0.2]], dtype=np.float32)
    r = bo.select(par2, p2, 3)
    assert r["keep"][0].tolist() == [True, False, True, True, False]
    assert r["parent_packed"][0].tolist() == [-1, 0, 1, -1, -1]
    assert r["node_id"].tolist() == [0, 2, 3]


def test_packed_forest_is_a_valid_forest_with_the_same_ancestry():
    rng = np.random.default_rng(3)
    B, Tc = 4, 20
    par = rand_trees(B, Tc, rng)
    p = rng.uniform(0.2, 1.0, size=(B, Tc)).astype(np.float32)
    r = bo.select(par, p, 37)
    for b in range(B):
        n = r["counts"][b]
        pp = r["parent_packed"][b]
        assert all(-1 <= pp[i] < i for i in range(n)) and (pp[n:] == -1).all()
        ids = r["node_id"][r["offsets"][b]:r["offsets"][b + 1]] - b * Tc
        assert (np.diff(ids) > 0).all()
        for i in range(n):   # the packed parent is the packed image of the original parent
            assert (pp[i] < 0 and par[b, ids[i]] < 0) or ids[pp[i]] == par[b, ids[i]]
