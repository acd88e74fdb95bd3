"""Packed forest (Section V-B): requests with different node counts share flat tensors; every
request is checked against the oracle run on its own tree, and against the dense call on the
same request."""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from oracle import tree_oracle as orc
from tests.parity_util import rel_l2_rows, rel_fro

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_forest(B, n_max, seed, kind="frontier"):
    """Per-request trees of 1..n_max nodes (the first has n_max, the second one node)."""
    rng = np.random.Generator(np.random.Philox(key=seed))
    sizes = [n_max, 1] + [int(rng.integers(1, n_max + 1)) for _ in range(max(0, B - 2))]
    sizes = sizes[:B]
    parents = []
    for n in sizes:
        if kind == "chain":
            parents.append(inputs.tree_chain(n))
        else:
            parents.append(inputs.tree_frontier(n, rng) if n > 1 else np.array([-1], dtype=np.int32))
    accepted = np.array([inputs.accepted_walk(p, rng) for p in parents], dtype=np.int32)
    accepted[-1] = -1
    return parents, accepted


def packed_tensors(wl, parents, capacity, Hk, L=1):
    """Draw dense per-request tensors with the workload's generator, then pack the real rows."""
    B, H = wl.B, wl.H
    G = H // Hk
    dt = wl.torch_dtype
    off = np.concatenate([[0], np.cumsum([len(p) for p in parents])]).astype(np.int64)
    layers = [inputs.make_tensors(wl, layer=l) for l in range(L)]
    fill = lambda *shape: torch.full(shape, float("nan"))   # rows past the forest: whatever is read there must not matter
    P = {"q": fill(L, Hk, capacity, wl.dk).to(dt), "k": fill(L, Hk, capacity, wl.dk).to(dt),
         "v": fill(L, H, capacity, wl.dv).to(dt), "alpha": fill(L, H, capacity),
         "beta": fill(L, H, capacity) if layers[0]["beta"] is not None else None,
         "S_pre": torch.stack([x["S_pre"] for x in layers])}
    for l, t in enumerate(layers):
        for b, par in enumerate(parents):
            n = len(par)
            rows = slice(int(off[b]), int(off[b]) + n)
            P["q"][l, :, rows] = t["q"][b, ::G, :n]
            P["k"][l, :, rows] = t["k"][b, ::G, :n]
            P["v"][l, :, rows] = t["v"][b, :, :n]
            P["alpha"][l, :, rows] = t["alpha"][b, :, :n]
            if P["beta"] is not None:
                P["beta"][l, :, rows] = t["beta"][b, :, :n]
    return P, off


def oracle_request(wl, P, off, parents, accepted, l, b, h, Hk):
    G = wl.H // Hk
    n = len(parents[b])
    rows = slice(int(off[b]), int(off[b]) + n)
    f = lambda t: inputs.to_f64(t)
    S = f(P["S_pre"][l, b, h]).T            # paper orientation [dk][dv]
    q, k, v = f(P["q"][l, h // G, rows]), f(P["k"][l, h // G, rows]), f(P["v"][l, h, rows])
    al = f(P["alpha"][l, h, rows])
    be = None if P["beta"] is None else f(P["beta"][l, h, rows])
    O, U, _ = orc.verify_memo(S, q, k, v, al, be, parents[b], wl.rule_name)
    Sn = orc.commit_walk(S, k, v, al, be, parents[b], int(accepted[b]), wl.rule_name)
    return O, U, Sn.T


CASES = [  # B, H, Hk, n_max, dk, dv, L
    (5, 4, 4, 64, 128, 128, 1),
    (4, 4, 2, 128, 128, 128, 2),
    (6, 2, 1, 33, 64, 128, 1),
    (3, 2, 2, 17, 64, 64, 1),
    (9, 2, 2, 8, 128, 128, 1),
    (40, 2, 2, 70, 128, 128, 1),
]


@pytest.mark.parametrize("impl", [tv.IMPL_AUTO, tv.IMPL_SIMT])
@pytest.mark.parametrize("rule", [inputs.GATED, inputs.DELTA])
@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("case", CASES)
def test_forest_matches_oracle_per_request(case, dtype, rule, impl):
    B, H, Hk, n_max, dk, dv, L = case
    wl = inputs.workload("c2", B=B, H=H, T=n_max, dk=dk, dv=dv, rule=rule, qkv_dtype=dtype, seed=400 + n_max)
    parents, accepted = make_forest(B, n_max, seed=n_max + B)
    total = sum(len(p) for p in parents)
    capacity = total + 37                      # spare rows at the end of every plane
    P, off = packed_tensors(wl, parents, capacity, Hk, L)
    g = {n: (None if t is None else t.to(DEV)) for n, t in P.items()}
    forest = tv.forest_build(parents, n_max=n_max, capacity=capacity).upload()
    O = torch.full((L, H, capacity, dv), 7.0, device=DEV)
    U = torch.full((L, H, capacity, dv), 7.0, device=DEV)
    tv.tree_verify(forest, g["S_pre"], g["q"], g["k"], g["v"], g["alpha"], g["beta"], rule=rule, O=O, U=U,
                   impl=impl)
    acc = torch.from_numpy(accepted).to(DEV)
    outs = []
    for with_U in (False, True):
        Sn = torch.empty_like(g["S_pre"])
        tv.commit_path(forest, acc, g["S_pre"], g["k"], g["v"], g["alpha"], g["beta"], rule=rule,
                       U=U if with_U else None, S_new=Sn)
        outs.append(Sn.cpu().double().numpy())
    torch.cuda.synchronize()
    forest.device_status()          # raises if a bounded device wait ran out
    assert torch.equal(g["S_pre"].cpu(), P["S_pre"])
    On, Un = O.cpu().double().numpy(), U.cpu().double().numpy()
    assert (On[:, :, total:] == 7.0).all() and (Un[:, :, total:] == 7.0).all()   # spare rows untouched
    tol = 1e-5 if dtype == inputs.F32 else 2e-3
    for l in range(L):
        for b in range(B):
            n = len(parents[b])
            rows = slice(int(off[b]), int(off[b]) + n)
            for h in range(H):
                Or, Ur, Sr = oracle_request(wl, P, off, parents, accepted, l, b, h, Hk)
                assert rel_l2_rows(On[l, h, rows], Or) <= tol
                assert rel_l2_rows(Un[l, h, rows], Ur) <= tol
                for Sn in outs:
                    assert rel_fro(Sn[l, b, h], Sr) <= tol


@pytest.mark.parametrize("n_max", [64, 128])
@pytest.mark.parametrize("rule", [inputs.GATED, inputs.DELTA])
def test_forest_takes_the_tensor_core_kernels(rule, n_max):
    """bf16, dk = dv = 128: IMPL_TC must accept a packed forest for both rules and both tree-size
    classes (no silent fallback) and agree with the general kernel."""
    wl = inputs.workload("c2", B=5, H=2, T=n_max, rule=rule, seed=11)
    parents, _ = make_forest(5, n_max, seed=12)
    cap = sum(len(p) for p in parents) + 3
    P, _ = packed_tensors(wl, parents, cap, 2)
    g = {n: (None if t is None else t.to(DEV)) for n, t in P.items()}
    forest = tv.forest_build(parents, n_max=n_max, capacity=cap).upload()
    outs = []
    for impl in (tv.IMPL_TC, tv.IMPL_SIMT):
        O = torch.zeros(1, 2, cap, 128, device=DEV)
        U = torch.zeros_like(O)
        tv.tree_verify(forest, g["S_pre"], g["q"], g["k"], g["v"], g["alpha"], g["beta"], rule=rule, O=O, U=U,
                       impl=impl)
        torch.cuda.synchronize()
        outs.append((O.cpu().double().numpy(), U.cpu().double().numpy()))
    forest.device_status()
    assert rel_fro(outs[0][0], outs[1][0]) < 2e-3 and rel_fro(outs[0][1], outs[1][1]) < 2e-3
    # deeper than the tensor-core delta kernel's path tables: declined, not faked
    if rule == inputs.DELTA and n_max == 64:
        deep = tv.forest_build([inputs.tree_chain(40)], n_max=64, capacity=64).upload()
        one = {n: (None if t is None else t[:, :1].contiguous() if n == "S_pre" else t) for n, t in g.items()}
        with pytest.raises(tv.TreeVerifyError) as e:
            tv.tree_verify(deep, one["S_pre"], g["q"][:, :, :64].contiguous(), g["k"][:, :, :64].contiguous(),
                           g["v"][:, :, :64].contiguous(), g["alpha"][:, :, :64].contiguous(),
                           g["beta"][:, :, :64].contiguous(), rule=rule, impl=tv.IMPL_TC)
        assert e.value.status == -3


def test_forest_metadata_and_rebuild():
    parents, accepted = make_forest(5, 40, seed=3)
    forest = tv.forest_build(parents, n_max=40, capacity=300).upload()
    anc, depth, max_depth = forest.meta()
    dev_anc, dev_depth = forest.meta_device()
    assert np.array_equal(anc, dev_anc) and np.array_equal(depth, dev_depth)
    for b, par in enumerate(parents):
        ref_anc, ref_depth, ref_md = orc.tree_metadata(par)
        n = len(par)
        assert np.array_equal(anc[b, :n], ref_anc) and np.array_equal(depth[b, :n], ref_depth)
        assert max_depth[b] == ref_md
        assert not anc[b, n:].any() and not depth[b, n:].any()
    # new topology with other sizes in the same buffers
    parents2, _ = make_forest(5, 40, seed=4, kind="chain")
    forest.rebuild_forest(parents2).upload()
    anc2, depth2, _ = forest.meta()
    dev_anc2, dev_depth2 = forest.meta_device()
    assert np.array_equal(anc2, dev_anc2) and np.array_equal(depth2, dev_depth2)
    assert depth2[0, 39] == 39


def test_forest_argument_errors():
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.forest_build([np.array([-1, 0]), np.array([-1])], n_max=1)
    assert e.value.status == -1
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.forest_build([np.array([-1, 0]), np.array([-1])], n_max=2, capacity=2)
    assert e.value.status == -8
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.forest_build([np.array([-1, 1])], n_max=2)
    assert e.value.status == -2
    dense = tv.tree_build(np.array([[-1, 0]], dtype=np.int32))
    with pytest.raises(tv.TreeVerifyError):
        dense.rebuild_forest([np.array([-1, 0])])


@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("W", [2, 4])
def test_forest_stage1_conv_and_context_commit(dtype, W):
    """Stage 1 on a packed forest: x rows packed, outputs in the planes the verify kernels read."""
    from oracle import tree_conv_oracle as cv
    H, dk, dv, n_max = 3, 64, 40, 48
    parents, accepted = make_forest(6, n_max, seed=21 + W)
    B = len(parents)
    total = sum(len(p) for p in parents)
    cap = total + 5
    C = H * (2 * dk + dv)
    dt = torch.bfloat16 if dtype == inputs.BF16 else torch.float32
    gen = torch.Generator().manual_seed(7 + W)
    x = torch.full((cap, C), float("nan")).to(dt)
    x[:total] = torch.randn(total, C, generator=gen).to(dt)
    ga = torch.full((cap, H), float("nan")).to(dt)
    gb = torch.full((cap, H), float("nan")).to(dt)
    ga[:total] = torch.randn(total, H, generator=gen).to(dt)
    gb[:total] = torch.randn(total, H, generator=gen).to(dt)
    ctx = torch.randn(B, W - 1, C, generator=gen).to(dt)
    weight = torch.randn(C, W, generator=gen) / W ** 0.5
    bias = 0.1 * torch.randn(C, generator=gen)
    A_log = -2 + 2.5 * torch.rand(H, generator=gen)
    dt_bias = -3 + 2 * torch.rand(H, generator=gen)
    forest = tv.forest_build(parents, n_max=n_max, capacity=cap).upload()
    out = {n: torch.full((H, cap, d), 9.0, device=DEV, dtype=dt) for n, d in (("q", dk), ("k", dk), ("v", dv))}
    al = torch.full((H, cap), 9.0, device=DEV)
    be = torch.full((H, cap), 9.0, device=DEV)
    tv.tree_conv(forest, x.to(DEV), ctx.to(DEV), weight.to(DEV), bias.to(DEV), H=H, dk=dk, dv=dv,
                 gate_a=ga.to(DEV), gate_b=gb.to(DEV), A_log=A_log.to(DEV), dt_bias=dt_bias.to(DEV),
                 normalize_qk=True, q=out["q"], k=out["k"], v=out["v"], alpha=al, beta=be)
    ctx_new = tv.conv_commit(forest, torch.from_numpy(accepted).to(DEV), x.to(DEV), ctx.to(DEV).clone(),
                             H=H, dk=dk, dv=dv)
    torch.cuda.synchronize()
    rtol, atol = (2.0 ** -8, 2e-6) if dtype == inputs.BF16 else (1e-5, 1e-6)
    f = inputs.to_f64
    off = 0
    for b, par in enumerate(parents):
        n = len(par)
        rows = slice(off, off + n)
        y = cv.tree_conv(f(x[rows]), f(ctx[b]), f(weight), f(bias), par)
        for name, ref in zip(("q", "k", "v"), cv.split_heads(y, H, dk, dv, normalize_qk=True, eps=1e-6)):
            got = out[name][:, rows].cpu().double().numpy()
            assert (np.abs(got - ref) <= rtol * np.abs(ref) + atol).all(), (name, b)
        ra, rb = cv.gate_prep(f(ga[rows]), f(gb[rows]), f(A_log), f(dt_bias))
        assert np.allclose(al[:, rows].cpu().double().numpy(), ra, rtol=5e-6)
        assert np.allclose(be[:, rows].cpu().double().numpy(), rb, rtol=5e-6)
        ref_ctx = cv.conv_commit(f(x[rows]), f(ctx[b]), par, int(accepted[b]))
        assert np.array_equal(ctx_new[b].cpu().double().numpy(), ref_ctx)
        off += n
    for t in list(out.values()) + [al, be]:
        assert bool((t[:, total:] == 9.0).all())      # rows past the forest untouched


@pytest.mark.parametrize("n_trees,n", [(200, 100), (129, 128), (16, 128)])
def test_metadata_upload_paths_agree_with_the_host(n_trees, n):
    """Small tree sets ride in the kernel parameters, large ones are staged through pinned memory:
    both must reproduce the host-built masks and depths bit for bit (and survive a rebuild)."""
    rng = np.random.Generator(np.random.Philox(key=n_trees))
    for trial in range(3):
        par = np.stack([inputs.tree_frontier(n, rng) for _ in range(n_trees)]).astype(np.int32)
        tree = tv.tree_build(par) if trial == 0 else tree.rebuild(par)
        tree.upload()
        anc, depth, _ = tree.meta()
        danc, ddepth = tree.meta_device()
        assert np.array_equal(anc, danc) and np.array_equal(depth, ddepth)


def test_commit_right_behind_a_forest_upload():
    """tv_commit_path directly behind tv_forest_rebuild + tv_tree_upload on the same stream, with
    no verify call in between: the commit grid may be scheduled while the metadata kernel still
    runs, and must not read the request offsets (or anything else that kernel writes) before that
    kernel is complete.  The handle first holds another forest, so stale offsets would put every
    request's rows in the wrong place."""
    B, H, n_max = 48, 8, 64
    wl = inputs.workload("c2", B=B, H=H, T=n_max, seed=77)
    first, _ = make_forest(B, n_max, seed=5)
    first = first[::-1]                                   # other sizes per request than `parents`
    parents, accepted = make_forest(B, n_max, seed=6)
    accepted = np.array([len(p) - 1 for p in parents], dtype=np.int32)   # last node: needs the right row count
    cap = B * n_max
    P, off = packed_tensors(wl, parents, cap, H)
    g = {n: (None if t is None else t.to(DEV)) for n, t in P.items()}
    acc = torch.from_numpy(accepted).to(DEV)
    forest = tv.forest_build(first, n_max=n_max, capacity=cap).upload()
    torch.cuda.synchronize()
    for _ in range(3):
        forest.rebuild_forest(first).upload()
        torch.cuda.synchronize()
        Sn = torch.empty_like(g["S_pre"])
        forest.rebuild_forest(parents).upload()
        tv.commit_path(forest, acc, g["S_pre"], g["k"], g["v"], g["alpha"], None, S_new=Sn)
        torch.cuda.synchronize()
        Snn = Sn.cpu().double().numpy()
        for b in range(0, B, 5):
            for h in (0, H - 1):
                Sr = oracle_request(wl, P, off, parents, accepted, 0, b, h, H)[2]
                assert rel_fro(Snn[0, b, h], Sr) <= 2e-3, (b, h)
