"""Pins for the CPU oracle: what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible mistake in the oracle (a dropped decay, a wrong sign, pre- instead
of post-update readout, a transposed state, a sibling leaking in) fails it.
"""
import itertools
import json
import os

import numpy as np
import pytest

from oracle import tree_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rand_tree(T, rng, max_children=3):
    par = np.full(T, -1, dtype=np.int64)
    for i in range(1, T):
        par[i] = rng.integers(-1, i)
    return par


def rand_problem(T, dk, dv, rng, unit_keys=False):
    S = rng.normal(size=(dk, dv))
    Q = rng.normal(size=(T, dk))
    K = rng.normal(size=(T, dk))
    if unit_keys:
        K /= np.linalg.norm(K, axis=1, keepdims=True)
    V = rng.normal(size=(T, dv))
    gamma = rng.uniform(0.3, 1.0, size=T)
    beta = rng.uniform(0.0, 1.0, size=T)
    return S, Q, K, V, gamma, beta


# ---- worked example (Eq. 1 / Table II sequential rule, by hand) ------------
def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLD, "hand_example.json")))
    par = np.array(g["parent"])
    S = np.array(g["S_pre"]); Q = np.array(g["Q"]); K = np.array(g["K"]); V = np.array(g["V"])
    gamma = np.array(g["gamma"]); beta = np.array(g["beta"])
    for rule in ("delta", "gated"):
        O, U = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
        O2, U2, states = orc.verify_memo(S, Q, K, V, gamma, beta, par, rule)
        assert np.array_equal(O, np.array(g[rule]["O"]))
        assert np.array_equal(O2, O) and np.array_equal(U2, U)
        if rule == "delta":
            assert np.array_equal(U, np.array(g[rule]["U"]))
        else:
            assert np.array_equal(U, V)
        for i in range(3):
            assert np.array_equal(states[i], np.array(g[rule][f"S_{i}"]))
            assert np.array_equal(orc.commit_walk(S, K, V, gamma, beta, par, i, rule),
                                  np.array(g[rule][f"S_{i}"]))
        assert np.array_equal(orc.commit_walk(S, K, V, gamma, beta, par, -1, rule), S)


# ---- Theorem 1 (Eq. 2) written densely equals the walk ---------------------
@pytest.mark.parametrize("rule", ["gated", "delta"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_closed_form_equals_walk(rule, seed):
    rng = np.random.default_rng(seed)
    T, dk, dv = 40, 16, 12
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, beta = rand_problem(T, dk, dv, rng, unit_keys=True)
    O, U = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
    Oc, Uc = orc.verify_closed_form(S, Q, K, V, gamma, beta, par, rule)
    assert np.abs(O - Oc).max() <= 1e-11 * max(1.0, np.abs(O).max())
    assert np.abs(U - Uc).max() <= 1e-11 * max(1.0, np.abs(U).max())
    Om, Um, _ = orc.verify_memo(S, Q, K, V, gamma, beta, par, rule)
    assert np.array_equal(O, Om) and np.array_equal(U, Um)


# ---- Eq. 4: factorised readout, gated rule as an explicit ancestor sum -----
def test_gated_explicit_ancestor_sum():
    rng = np.random.default_rng(5)
    T, dk, dv = 23, 8, 6
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, _ = rand_problem(T, dk, dv, rng)
    O, _ = orc.verify_walk(S, Q, K, V, gamma, None, par, "gated")
    for i in range(T):
        # ancestors found by following parent links here, not by the oracle
        chain, p = [i], par[i]
        while p >= 0:
            chain.append(p); p = par[p]
        Pi = np.prod(gamma[chain])
        o = Pi * (S.T @ Q[i])
        for j in chain:
            sub, p = [], i
            while p != j:          # gates strictly after j on the path
                sub.append(p); p = par[p]
            o = o + np.prod(gamma[sub]) * (Q[i] @ K[j]) * V[j]
        assert np.allclose(O[i], o, rtol=1e-12, atol=1e-13)


# ---- Lemma 3: G strictly lower triangular, nilpotent of order d+1 ----------
def test_nilpotency_and_neumann():
    rng = np.random.default_rng(7)
    T, dk, dv = 30, 8, 5
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, beta = rand_problem(T, dk, dv, rng)
    beta = beta + 0.1
    anc, depth, d = orc.tree_metadata(par)
    P, G, C = orc.closed_form_factors(Q, K, gamma, beta, par)
    assert np.array_equal(np.triu(G), np.zeros_like(G))
    assert abs(np.linalg.det(np.eye(T) + G) - 1.0) < 1e-12
    assert np.array_equal(np.linalg.matrix_power(G, d + 1), np.zeros_like(G))
    assert np.abs(np.linalg.matrix_power(G, d)).max() > 0
    R = np.diag(beta) @ (V - np.diag(P) @ K @ S)
    Un = orc.neumann_solve(G, R, d)
    Us = np.linalg.solve(np.eye(T) + G, R)
    assert np.allclose(Un, Us, rtol=1e-12, atol=1e-13)
    _, Uw = orc.verify_walk(S, Q, K, V, gamma, beta, par, "delta")
    assert np.allclose(Un, Uw, rtol=1e-11, atol=1e-12)


# ---- Eq. 10: factored commit reconstructs the walked state -----------------
@pytest.mark.parametrize("rule", ["gated", "delta"])
def test_commit_factored_equals_walk(rule):
    rng = np.random.default_rng(11)
    T, dk, dv = 25, 10, 7
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, beta = rand_problem(T, dk, dv, rng)
    _, U = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
    for a in [-1, 0, 7, T - 1]:
        Sw = orc.commit_walk(S, K, V, gamma, beta, par, a, rule)
        Sf = orc.commit_factored(S, K, U, gamma, par, a)
        assert np.allclose(Sw, Sf, rtol=1e-12, atol=1e-13)
    assert np.array_equal(orc.commit_walk(S, K, V, gamma, beta, par, -1, rule), S)


# ---- textbook special cases -------------------------------------------------
def test_masked_linear_attention_special_case():
    """gamma = 1, S_pre = 0, gated  =>  O = ((Q K^T) * M+) V, mask by brute force."""
    rng = np.random.default_rng(13)
    T, dk, dv = 31, 9, 4
    par = rand_tree(T, rng)
    _, Q, K, V, _, _ = rand_problem(T, dk, dv, rng)
    A = np.zeros((T, T), dtype=np.int64)        # adjacency child -> parent
    for i, p in enumerate(par):
        if p >= 0:
            A[i, p] = 1
    reach = np.zeros_like(A)
    Pw = np.eye(T, dtype=np.int64)
    for _ in range(T):                           # transitive closure by powers
        Pw = Pw @ A
        reach += Pw
    Mp = (reach > 0).astype(float) + np.eye(T)
    O, _ = orc.verify_walk(np.zeros((dk, dv)), Q, K, V, np.ones(T), None, par, "gated")
    assert np.allclose(O, ((Q @ K.T) * Mp) @ V, rtol=1e-12, atol=1e-13)
    Mm, Mp2 = orc.ancestor_masks(par)
    assert np.array_equal(Mp2, Mp) and np.array_equal(Mm, Mp - np.eye(T))


def test_delta_retrieval():
    """beta = 1, |k| = 1, q = k  =>  o_i = v_i exactly, for every node of any tree."""
    rng = np.random.default_rng(17)
    T, dk, dv = 20, 12, 6
    par = rand_tree(T, rng)
    S, _, K, V, gamma, _ = rand_problem(T, dk, dv, rng, unit_keys=True)
    O, _ = orc.verify_walk(S, K, K, V, gamma, np.ones(T), par, "delta")
    assert np.allclose(O, V, rtol=0, atol=1e-12)


def test_beta_zero_is_pure_decay():
    rng = np.random.default_rng(19)
    T, dk, dv = 18, 7, 5
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, _ = rand_problem(T, dk, dv, rng)
    O, U = orc.verify_walk(S, Q, K, V, gamma, np.zeros(T), par, "delta")
    assert np.array_equal(U, np.zeros_like(U))
    for i in range(T):
        Pi, p = gamma[i], par[i]
        while p >= 0:
            Pi *= gamma[p]; p = par[p]
        assert np.allclose(O[i], Pi * (S.T @ Q[i]), rtol=1e-12, atol=1e-14)


# ---- chain tree = ordinary sequential decoding (Eq. 1) ---------------------
@pytest.mark.parametrize("rule", ["gated", "delta"])
def test_chain_is_sequential_decode(rule):
    rng = np.random.default_rng(23)
    T, dk, dv = 12, 6, 5
    S, Q, K, V, gamma, beta = rand_problem(T, dk, dv, rng)
    par = np.arange(-1, T - 1)
    O, U = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
    St = S.copy()
    for t in range(T):                       # Eq. 1 in token order, one state
        St = gamma[t] * St
        u = beta[t] * (V[t] - K[t] @ St) if rule == "delta" else V[t]
        St = St + K[t][:, None] * u[None, :]
        assert np.allclose(O[t], Q[t] @ St, rtol=1e-12, atol=1e-13)
    assert np.allclose(orc.commit_walk(S, K, V, gamma, beta, par, T - 1, rule), St,
                       rtol=1e-12, atol=1e-13)


def test_single_node_is_one_decode_step():
    rng = np.random.default_rng(29)
    S, Q, K, V, gamma, beta = rand_problem(1, 5, 4, rng)
    O, U = orc.verify_walk(S, Q, K, V, gamma, beta, np.array([-1]), "delta")
    St = gamma[0] * S
    u = beta[0] * (V[0] - St.T @ K[0])
    assert np.allclose(U[0], u) and np.allclose(O[0], (St + np.outer(K[0], u)).T @ Q[0])


# ---- independence of siblings and non-ancestors -----------------------------
@pytest.mark.parametrize("rule", ["gated", "delta"])
def test_sibling_and_non_ancestor_independence(rule):
    rng = np.random.default_rng(31)
    T, dk, dv = 24, 6, 5
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, beta = rand_problem(T, dk, dv, rng)
    O, U = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
    for i in [3, 11, T - 1]:
        keep = set(orc.path_to(par, i))
        K2, V2, Q2, g2, b2 = K.copy(), V.copy(), Q.copy(), gamma.copy(), beta.copy()
        for j in range(T):
            if j not in keep:
                K2[j] = rng.normal(size=dk) * 1e3; V2[j] = np.inf; Q2[j] = np.nan
                g2[j] = 7.0; b2[j] = -3.0
        o, u, _ = orc.walk_node(S, Q2, K2, V2, g2, b2, par, i, rule)
        assert np.array_equal(o, O[i]) and np.array_equal(u, U[i])


# ---- brute force over every tree with up to five nodes ----------------------
def all_parent_arrays(T):
    return itertools.product(*[range(-1, i) for i in range(T)])


@pytest.mark.parametrize("rule", ["gated", "delta"])
def test_brute_force_all_small_trees(rule):
    rng = np.random.default_rng(37)
    count = 0
    for T in range(1, 6):
        S, Q, K, V, gamma, beta = rand_problem(T, 3, 2, rng)
        for par in all_parent_arrays(T):
            par = np.array(par)
            O, U = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
            Oc, Uc = orc.verify_closed_form(S, Q, K, V, gamma, beta, par, rule)
            assert np.allclose(O, Oc, rtol=1e-11, atol=1e-12)
            assert np.allclose(U, Uc, rtol=1e-11, atol=1e-12)
            count += 1
    assert count == 1 + 2 + 6 + 24 + 120


# ---- verify/commit consistency (Lemma 1) ------------------------------------
@pytest.mark.parametrize("rule", ["gated", "delta"])
def test_commit_then_verify_subtree(rule):
    rng = np.random.default_rng(41)
    T, dk, dv = 26, 6, 4
    par = rand_tree(T, rng)
    S, Q, K, V, gamma, beta = rand_problem(T, dk, dv, rng)
    O, _ = orc.verify_walk(S, Q, K, V, gamma, beta, par, rule)
    a = 2
    Sa = orc.commit_walk(S, K, V, gamma, beta, par, a, rule)
    desc = [i for i in range(T) if a in orc.strict_ancestors(par, i)]
    assert desc, "pick a node with descendants"
    remap = {a: -1}
    sub = []
    for i in desc:
        remap[i] = len(sub); sub.append(i)
    par2 = np.array([remap[par[i]] for i in sub])
    O2, _ = orc.verify_walk(Sa, Q[sub], K[sub], V[sub], gamma[sub], beta[sub], par2, rule)
    assert np.allclose(O2, O[sub], rtol=1e-11, atol=1e-12)


# ---- metadata ---------------------------------------------------------------
def test_metadata_invariants():
    rng = np.random.default_rng(43)
    for T in [1, 2, 15, 64, 65, 128]:
        par = rand_tree(T, rng)
        anc, depth, d = orc.tree_metadata(par)
        assert anc.dtype == np.uint64 and anc.shape == (T, 2)
        for i in range(T):
            bits = [j for j in range(128) if (int(anc[i, j >> 6]) >> (j & 63)) & 1]
            assert len(bits) == depth[i]
            assert all(j < i for j in bits)
            if par[i] >= 0:
                p = par[i]
                pb = [j for j in range(128) if (int(anc[p, j >> 6]) >> (j & 63)) & 1]
                assert sorted(pb + [int(p)]) == bits
            else:
                assert bits == []
            assert orc.accepted_path(par, i) == bits + [i]
        assert d == depth.max()
    assert orc.accepted_path(np.array([-1, 0]), -1) == []
    with pytest.raises(ValueError):
        orc.tree_metadata(np.array([-1, 1]))
    with pytest.raises(ValueError):
        orc.tree_metadata(np.array([-2]))


def test_binary_tree_depth_three():
    par = np.array([-1] + [(i - 1) // 2 for i in range(1, 15)])
    anc, depth, d = orc.tree_metadata(par)
    assert d == 3 and list(depth) == [0, 1, 1, 2, 2, 2, 2] + [3] * 8
    assert int(anc[14, 0]) == (1 << 0) | (1 << 2) | (1 << 6)


# ---- size arithmetic the paper prints (Table I; Eq. 9) ----------------------
def test_state_and_factor_sizes_match_table_one():
    layers, H, dk, dv, T = 24, 32, 128, 128, 100
    state = layers * H * dk * dv * 4
    assert state == 48 * 2 ** 20                      # "48 MB" linear state
    snapshots = T * state
    assert abs(snapshots / 1e9 - 4.7) < 0.4           # "4.7 GB" of snapshots
    # printed per-node reduction "82-99x": 4.7 GB / 57 MB and 14.1 GB / 142 MB
    assert 82 <= 4.7e9 / 57e6 < 83 and 99 <= 14.1e9 / 142e6 < 100
    # Eq. 9: one factorised node costs Theta(H (dk+dv+1)) elements, a snapshot H dk dv
    assert (H * dk * dv) / (H * (dk + dv + 1)) > 60


# ---- the batch wrappers: library layout S^ = S^T [B,H,dv,dk], tree pick per request ----------
def _hand_batch(rule, per_request_trees):
    """The hand-worked examples laid out as the library stores them, with dk = 2 != dv = 3.

    Every value channel of the recurrence evolves on its own and linearly in (its column of
    S_pre, its column of V) (Sec. IV-B: value channels are independent), so a third channel
    2*c0 - c1 must come out as 2*out0 - out1, and head 1 (S_pre and V scaled by -1/2) as -1/2
    of head 0.  Request 1 uses either the same tree or the root-child variant of the second
    golden file, whose node 1 differs.  All expected values trace back to the hand examples.
    """
    g = json.load(open(os.path.join(GOLD, "hand_example.json")))
    g2 = json.load(open(os.path.join(GOLD, "hand_example_root_child.json")))
    widen = lambda rows: [[r[0], r[1], 2 * r[0] - r[1]] for r in rows]        # [.., 2] -> [.., 3]
    S3, V3 = widen(g["S_pre"]), widen(g["V"])                                  # [dk][3], [T][3]
    B, H, T, dk, dv = 2, 2, 3, 2, 3
    scale = [1.0, -0.5]
    S_hat = np.zeros((B, H, dv, dk)); q = np.zeros((B, H, T, dk)); k = np.zeros((B, H, T, dk))
    v = np.zeros((B, H, T, dv)); gamma = np.zeros((B, H, T)); beta = np.zeros((B, H, T))
    for b in range(B):
        for h in range(H):
            for c in range(dv):
                for kk in range(dk):
                    S_hat[b, h, c, kk] = scale[h] * S3[kk][c]      # transposed by hand
            for i in range(T):
                for kk in range(dk):
                    q[b, h, i, kk] = g["Q"][i][kk]
                    k[b, h, i, kk] = g["K"][i][kk]
                for c in range(dv):
                    v[b, h, i, c] = scale[h] * V3[i][c]
                gamma[b, h, i] = g["gamma"][i]
                beta[b, h, i] = g["beta"][i]
    parents = np.array([g["parent"], g2["parent"]]) if per_request_trees else np.array([g["parent"]])
    # expected per request: rows of O, U and the per-node states [dk][dv], widened to 3 channels
    exp = []
    for b in range(B):
        O = [list(r) for r in g[rule]["O"]]
        U = [list(r) for r in (g[rule]["U"] if rule == "delta" else g["V"])]
        St = [g[rule][f"S_{i}"] for i in range(T)]
        if per_request_trees and b == 1:
            O[1] = list(g2[rule]["O_1"])
            if rule == "delta":
                U[1] = list(g2[rule]["U_1"])
            St[1] = g2[rule]["S_1"]
        exp.append((widen(O), widen(U), [widen(s) for s in St]))
    return (S_hat, q, k, v, gamma, beta, parents), exp, scale, widen(g["S_pre"])


@pytest.mark.parametrize("rule", ["gated", "delta"])
@pytest.mark.parametrize("per_request_trees", [False, True])
@pytest.mark.parametrize("memo", [True, False])
def test_verify_batch_layout_and_tree_pick(rule, per_request_trees, memo):
    (S_hat, q, k, v, gamma, beta, parents), exp, scale, _ = _hand_batch(rule, per_request_trees)
    out = orc.verify_batch(S_hat, q, k, v, gamma, None if rule == "gated" else beta, parents, rule, memo=memo)
    assert sorted(out) == [(b, h) for b in range(2) for h in range(2)]
    for (b, h), (O, U) in out.items():
        Oe, Ue, _ = exp[b]
        assert O.shape == (3, 3) and U.shape == (3, 3)
        assert np.array_equal(O, scale[h] * np.array(Oe)), (b, h)
        assert np.array_equal(U, scale[h] * np.array(Ue)), (b, h)
    # the item list restricts the work and keeps the indexing
    one = orc.verify_batch(S_hat, q, k, v, gamma, beta, parents, rule, memo=memo, items=[(1, 1)])
    assert list(one) == [(1, 1)] and np.array_equal(one[(1, 1)][0], out[(1, 1)][0])


@pytest.mark.parametrize("rule", ["gated", "delta"])
@pytest.mark.parametrize("per_request_trees", [False, True])
def test_commit_batch_layout_and_tree_pick(rule, per_request_trees):
    (S_hat, q, k, v, gamma, beta, parents), exp, scale, S3 = _hand_batch(rule, per_request_trees)
    for accepted in ([2, 1], [1, -1], [-1, 0]):
        out = orc.commit_batch(S_hat, k, v, gamma, None if rule == "gated" else beta, parents, accepted, rule)
        for (b, h), Sn in out.items():
            a = accepted[b]
            S_paper = S3 if a < 0 else exp[b][2][a]                  # [dk][dv]
            want = np.zeros((3, 2))
            for c in range(3):
                for kk in range(2):
                    want[c, kk] = scale[h] * S_paper[kk][c]          # library layout [dv][dk]
            assert Sn.shape == (3, 2)
            assert np.array_equal(Sn, want), (accepted, b, h)
