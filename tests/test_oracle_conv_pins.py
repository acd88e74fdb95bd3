"""Pins for the Stage-1 oracle (tree-parallel causal convolution + bias + SiLU)."""
import numpy as np

from oracle import tree_conv_oracle as cv


def rand_tree(T, rng):
    return np.array([-1] + [rng.integers(-1, i) for i in range(1, T)])


def test_hand_worked_example():
    """Two channels, width 3, by hand: node 0 root child, nodes 1 and 2 children of 0."""
    x = np.array([[1.0, 2.0], [3.0, -1.0], [0.5, 4.0]])
    ctx = np.array([[10.0, 20.0], [-2.0, 0.25]])          # oldest first; ctx[1] is the last token
    w = np.array([[0.5, -1.0, 2.0], [1.0, 0.0, -0.5]])     # w[c][2] multiplies the current token
    bias = np.array([0.25, -1.0])
    par = np.array([-1, 0, 0])
    y = cv.tree_conv(x, ctx, w, bias, par)
    # node 0: inputs (x0, ctx[1], ctx[0]);  node 1: (x1, x0, ctx[1]);  node 2: (x2, x0, ctx[1])
    z = np.array([
        [0.25 + 2.0 * 1.0 + (-1.0) * (-2.0) + 0.5 * 10.0, -1.0 + (-0.5) * 2.0 + 0.0 * 0.25 + 1.0 * 20.0],
        [0.25 + 2.0 * 3.0 + (-1.0) * 1.0 + 0.5 * (-2.0), -1.0 + (-0.5) * (-1.0) + 0.0 * 2.0 + 1.0 * 0.25],
        [0.25 + 2.0 * 0.5 + (-1.0) * 1.0 + 0.5 * (-2.0), -1.0 + (-0.5) * 4.0 + 0.0 * 2.0 + 1.0 * 0.25],
    ])
    assert np.array_equal(z, np.array([[9.25, 18.0], [4.25, -0.25], [-0.75, -2.75]]))
    assert np.allclose(y, z / (1.0 + np.exp(-z)), rtol=1e-15)


def test_chain_equals_library_causal_convolution():
    """On a chain the operator is the ordinary causal depthwise convolution of the sequence
    [context, tokens]: numpy.convolve per channel."""
    rng = np.random.default_rng(1)
    T, C, W = 17, 5, 4
    x = rng.normal(size=(T, C)); ctx = rng.normal(size=(W - 1, C))
    w = rng.normal(size=(C, W)); bias = rng.normal(size=C)
    y = cv.tree_conv(x, ctx, w, bias, np.arange(-1, T - 1))
    seq = np.concatenate([ctx, x])
    for c in range(C):
        full = np.convolve(seq[:, c], w[c, ::-1])          # correlation with w = convolution with reversed w
        z = full[W - 1:W - 1 + T] + bias[c]
        assert np.allclose(y[:, c], z / (1 + np.exp(-z)), rtol=1e-12, atol=1e-13)


def test_width_one_is_pointwise_and_no_bias_is_zero_bias():
    rng = np.random.default_rng(2)
    T, C = 9, 4
    x = rng.normal(size=(T, C)); w = rng.normal(size=(C, 1)); par = rand_tree(T, rng)
    y = cv.tree_conv(x, np.zeros((0, C)), w, None, par)
    z = x * w[:, 0]
    assert np.allclose(y, z / (1 + np.exp(-z)), rtol=1e-14)
    y0 = cv.tree_conv(x, np.zeros((0, C)), w, np.zeros(C), par)
    assert np.array_equal(y, y0)


def test_node_depends_only_on_its_path_and_the_context():
    rng = np.random.default_rng(3)
    T, C, W = 20, 3, 4
    par = rand_tree(T, rng)
    x = rng.normal(size=(T, C)); ctx = rng.normal(size=(W - 1, C))
    w = rng.normal(size=(C, W)); bias = rng.normal(size=C)
    y = cv.tree_conv(x, ctx, w, bias, par)
    for i in (4, 11, T - 1):
        keep, j = set(), i
        while j >= 0:
            keep.add(j); j = par[j]
        x2 = x.copy()
        for j in range(T):
            if j not in keep:
                x2[j] = np.nan
        assert np.array_equal(cv.tree_conv(x2, ctx, w, bias, par)[i], y[i])
    # every node at depth >= W-1 ignores the context altogether
    depth = np.zeros(T, dtype=int)
    for i in range(T):
        depth[i] = 0 if par[i] < 0 else depth[par[i]] + 1
    yc = cv.tree_conv(x, ctx * 0 + 99.0, w, bias, par)
    for i in range(T):
        assert np.array_equal(yc[i], y[i]) == (depth[i] >= W - 1)


def test_siblings_share_the_parent_window():
    """Two children of the same parent with equal inputs get equal outputs (their windows
    coincide), whatever sits between them in the flattened order."""
    rng = np.random.default_rng(4)
    C, W = 6, 4
    par = np.array([-1, 0, 1, 1, 0, 1])
    x = rng.normal(size=(6, C)); x[5] = x[2]
    ctx = rng.normal(size=(W - 1, C)); w = rng.normal(size=(C, W))
    y = cv.tree_conv(x, ctx, w, None, par)
    assert np.array_equal(y[5], y[2]) and not np.array_equal(y[3], y[2])


def test_head_split_and_normalisation():
    rng = np.random.default_rng(5)
    T, H, dk, dv = 3, 2, 4, 3
    y = rng.normal(size=(T, H * (2 * dk + dv)))
    q, k, v = cv.split_heads(y, H, dk, dv)
    assert q.shape == (H, T, dk) and v.shape == (H, T, dv)
    assert np.array_equal(q[1, 2], y[2, dk:2 * dk])
    assert np.array_equal(k[0, 1], y[1, H * dk:H * dk + dk])
    assert np.array_equal(v[1, 0], y[0, 2 * H * dk + dv:2 * H * dk + 2 * dv])
    qn, kn, vn = cv.split_heads(y, H, dk, dv, normalize_qk=True, eps=0.0)
    assert np.allclose(np.linalg.norm(qn, axis=-1), 1.0) and np.allclose(np.linalg.norm(kn, axis=-1), 1.0)
    assert np.array_equal(vn, v)
    assert np.allclose(qn * np.linalg.norm(q, axis=-1, keepdims=True), q)


def test_gate_prep_closed_forms_and_library():
    import torch
    rng = np.random.default_rng(6)
    T, H = 7, 3
    a = rng.normal(size=(T, H)) * 3; b = rng.normal(size=(T, H)) * 3
    A_log = rng.uniform(-1, 2, size=H); dt_bias = rng.uniform(-4, 1, size=H)
    gamma, beta = cv.gate_prep(a, b, A_log, dt_bias)
    assert gamma.shape == (H, T) and beta.shape == (H, T)
    sp = torch.nn.functional.softplus(torch.tensor(a + dt_bias), threshold=1e9).numpy()
    assert np.allclose(gamma.T, np.exp(-np.exp(A_log) * sp), rtol=1e-13)
    assert np.allclose(beta.T, torch.sigmoid(torch.tensor(b)).numpy(), rtol=1e-13)
    # closed forms: softplus(0) = ln 2, sigmoid(0) = 1/2, sigmoid(x) + sigmoid(-x) = 1
    g0, b0 = cv.gate_prep(np.zeros((1, 1)), np.zeros((1, 1)), np.array([0.0]), np.array([0.0]))
    assert np.isclose(g0[0, 0], 0.5, rtol=1e-15) and b0[0, 0] == 0.5      # exp(-ln 2)
    _, bm = cv.gate_prep(a, -b, A_log, dt_bias)
    assert np.allclose(beta + bm, 1.0, rtol=1e-14)
    # large arguments: softplus(z) -> z, no overflow
    g1, _ = cv.gate_prep(np.full((1, 1), 800.0), np.zeros((1, 1)), np.array([-3.0]), np.array([0.0]))
    assert np.isclose(g1[0, 0], np.exp(-np.exp(-3.0) * 800.0), rtol=1e-13)
    assert np.all(gamma > 0) and np.all(gamma <= 1)


def test_conv_commit_continues_the_linear_sequence():
    """After committing a path, a follow-up chain convolved with the new context equals the
    library convolution over [old context, accepted tokens, new tokens]."""
    rng = np.random.default_rng(7)
    T, C, W = 12, 4, 4
    par = rand_tree(T, rng)
    x = rng.normal(size=(T, C)); ctx = rng.normal(size=(W - 1, C))
    w = rng.normal(size=(C, W)); bias = rng.normal(size=C)
    depth = np.zeros(T, dtype=int)
    for i in range(T):
        depth[i] = 0 if par[i] < 0 else depth[par[i]] + 1
    for acc in (-1, int(np.argmin(depth)), int(np.argmax(depth)), T - 1):
        new_ctx = cv.conv_commit(x, ctx, par, acc)
        assert new_ctx.shape == ctx.shape
        path = []
        j = acc
        while j >= 0:
            path.append(j); j = par[j]
        path.reverse()
        x2 = rng.normal(size=(5, C))
        y2 = cv.tree_conv(x2, new_ctx, w, bias, np.arange(-1, 4))
        seq = np.concatenate([ctx, x[path], x2])
        for c in range(C):
            z = np.convolve(seq[:, c], w[c, ::-1])[len(seq) - 5:len(seq)] + bias[c]
            assert np.allclose(y2[:, c], z / (1 + np.exp(-z)), rtol=1e-12, atol=1e-13)
    assert np.array_equal(cv.conv_commit(x, ctx, par, -1), ctx)
    # a path shorter than the window keeps the newest old rows
    root_child = int(np.argmin(depth))
    nc = cv.conv_commit(x, ctx, par, root_child)
    assert np.array_equal(nc[-1], x[root_child]) and np.array_equal(nc[:-1], ctx[1:])
