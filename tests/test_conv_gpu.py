"""GPU parity of Stage 1 (tv_tree_conv, tv_conv_commit) against the fp64 oracle, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from oracle import tree_conv_oracle as cv

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# Elementwise bounds.  bf16 outputs: one rounding to 8 significant bits (2^-9 relative) on top of
# fp32 arithmetic -> 2^-8 relative + 2e-6 absolute.  f32: ex2/rcp approximations and fp32 sums of
# at most 8 products -> 1e-5 relative + 1e-6 absolute.  Gates use the accurate fp32 functions.
TOL = {torch.bfloat16: (2.0 ** -8, 2e-6), torch.float32: (1e-5, 1e-6)}
GATE_RTOL = 5e-6


def canary(shape, dtype):
    n = int(np.prod(shape))
    buf = torch.full((n + 128,), 77.0, device=DEV, dtype=dtype)
    return buf, buf[64:64 + n].view(*shape)


def canary_ok(buf, n):
    return bool((buf[:64] == 77.0).all() and (buf[64 + n:] == 77.0).all())


def close(got, ref, dtype, what, scale=1.0):
    """`scale` widens the absolute term with the size of the summed products (cancellation in the
    fp32 sum loses absolute, not relative, accuracy)."""
    rtol, atol = TOL[dtype]
    atol *= scale
    got = got.detach().cpu().double().numpy()
    err = np.abs(got - ref) - (rtol * np.abs(ref) + atol)
    assert np.isfinite(got).all(), what
    assert err.max() <= 0, f"{what}: worst excess {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"


def run_case(wl, parents, W=4, normalize=False, gates=True, gate_b=True, bias=True, scale=1.0, requests=None,
             impl=tv.IMPL_AUTO):
    ci = inputs.make_conv_inputs(wl, layer=0, device="cpu", W=W)
    if scale != 1.0:
        ci["x"] = (ci["x"].float() * scale).to(ci["x"].dtype)
    dt = ci["x"].dtype
    g = {k: v.to(DEV) for k, v in ci.items()}
    tree = tv.tree_build(parents).upload()
    B, H, T, dk, dv = wl.B, wl.H, wl.T, wl.dk, wl.dv
    qb, q = canary((B, H, T, dk), dt)
    kb, k = canary((B, H, T, dk), dt)
    vb, v = canary((B, H, T, dv), dt)
    ab, al = canary((B, H, T), torch.float32)
    bb, be = canary((B, H, T), torch.float32)
    x0 = g["x"].clone()
    tv.tree_conv(tree, g["x"], g["ctx"] if W > 1 else None, g["weight"], g["bias"] if bias else None,
                 H=H, dk=dk, dv=dv, gate_a=g["gate_a"] if gates else None,
                 gate_b=g["gate_b"] if gates and gate_b else None, A_log=g["A_log"], dt_bias=g["dt_bias"],
                 normalize_qk=normalize, eps=1e-6, q=q, k=k, v=v, alpha=al if gates else None,
                 beta=be if gates and gate_b else None, impl=impl)
    torch.cuda.synchronize()
    assert torch.equal(g["x"], x0)
    for buf, t in ((qb, q), (kb, k), (vb, v), (ab, al), (bb, be)):
        assert canary_ok(buf, t.numel())
    if not gates:
        assert bool((al == 77.0).all())
    if not (gates and gate_b):
        assert bool((be == 77.0).all())
    f = {k_: inputs.to_f64(v_) for k_, v_ in ci.items()}
    sel = range(B) if requests is None else requests
    par = np.asarray(parents)
    for b in sel:
        pb = par[0] if par.shape[0] == 1 else par[b]
        y = cv.tree_conv(f["x"][b], f["ctx"][b] if W > 1 else np.zeros((0, f["x"].shape[2])), f["weight"],
                         f["bias"] if bias else None, pb)
        rq, rk, rv = cv.split_heads(y, H, dk, dv, normalize_qk=normalize, eps=1e-6)
        close(q[b], rq, dt, f"q[{b}]", scale)
        close(k[b], rk, dt, f"k[{b}]", scale)
        close(v[b], rv, dt, f"v[{b}]", scale)
        if gates:
            ga, gb = cv.gate_prep(f["gate_a"][b], f["gate_b"][b], f["A_log"], f["dt_bias"])
            assert np.allclose(al[b].cpu().double().numpy(), ga, rtol=GATE_RTOL, atol=1e-30)
            if gate_b:
                assert np.allclose(be[b].cpu().double().numpy(), gb, rtol=GATE_RTOL, atol=0)
    return g, tree


@pytest.mark.parametrize("impl", [tv.IMPL_AUTO, tv.IMPL_SIMT])
@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_workloads(name, impl):
    wl = inputs.workload(name)
    parents, _ = inputs.make_trees(wl)
    run_case(wl, parents, W=4, normalize=(name in ("c2", "c4")), impl=impl)


@pytest.mark.parametrize("T", [1, 7, 16, 17, 63, 64, 65, 100, 128])
@pytest.mark.parametrize("W", [1, 2, 3, 4])
def test_bf16_head128_tile_edges(T, W):
    """bf16, 128-channel heads, W <= 4 (the shape of the workloads) over tile-edge node counts."""
    wl = dataclasses.replace(inputs.workload("c2"), B=3, H=2, T=T, seed=900 + T + W)
    parents, _ = inputs.make_trees(wl)
    run_case(wl, parents, W=W, normalize=bool(T & 1), gate_b=bool(W & 1), bias=W != 3)


def test_no_tensor_core_form():
    """IMPL_TC is refused: the operator has no tensor-core kernel and never falls back silently."""
    wl = dataclasses.replace(inputs.workload("c2"), B=1, H=2, T=16)
    parents, _ = inputs.make_trees(wl)
    with pytest.raises(tv.TreeVerifyError) as e:
        run_case(wl, parents, W=4, impl=tv.IMPL_TC)
    assert e.value.status == -3


def test_c5_sampled_requests():
    wl = inputs.workload("c5")
    parents, _ = inputs.make_trees(wl)
    run_case(wl, parents, W=4, normalize=True, requests=[0, 37, 127])


SHAPES = [  # B, H, T, dk, dv
    (1, 1, 1, 8, 8), (2, 3, 5, 64, 128), (3, 2, 33, 128, 64), (2, 2, 128, 128, 128),
    (2, 1, 65, 192, 256), (1, 2, 127, 256, 200), (5, 4, 64, 32, 40),
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("W", [1, 2, 4, 8])
def test_shapes(shape, dtype, W):
    B, H, T, dk, dv = shape
    if dtype == inputs.F32 and (dk % 4 or dv % 4):
        pytest.skip("not a float shape")
    wl = dataclasses.replace(inputs.workload("c2"), B=B, H=H, T=T, dk=dk, dv=dv, qkv_dtype=dtype,
                             seed=B * 1000 + T * 10 + W)
    parents, _ = inputs.make_trees(wl)
    run_case(wl, parents, W=W, normalize=bool(W & 2), gates=True, gate_b=bool(W & 4), bias=W != 2)


@pytest.mark.parametrize("B,H", [(1, 160), (2, 100), (3, 70)])
def test_many_slices_per_cta(B, H):
    """More (slice, request) items than CTAs with one to three requests per slice: every CTA walks
    several items whose filter changes with (almost) every item, through all of its slots."""
    wl = dataclasses.replace(inputs.workload("c2"), B=B, H=H, T=12, dk=16, dv=8, seed=4000 + B)
    parents, _ = inputs.make_trees(wl)
    run_case(wl, parents, W=4, normalize=True, gates=True, gate_b=True)


@pytest.mark.parametrize("kind", ["chain", "star", "shared"])
def test_tree_kinds(kind):
    wl = dataclasses.replace(inputs.workload("c2"), B=3, H=2, T=40)
    if kind == "chain":
        parents = np.tile(inputs.tree_chain(wl.T), (wl.B, 1))
    elif kind == "star":
        parents = np.full((wl.B, wl.T), -1, dtype=np.int32)
    else:
        parents = inputs.tree_binary(wl.T)[None, :]
    run_case(wl, parents, W=4, normalize=True)


@pytest.mark.filterwarnings("ignore:overflow encountered in exp")
def test_large_activations_saturate_cleanly():
    """|z| of a few hundred: e^-z overflows in fp32; outputs must be z or (minus) zero, not NaN."""
    wl = dataclasses.replace(inputs.workload("c2"), B=1, H=2, T=31, qkv_dtype=inputs.F32)
    parents, _ = inputs.make_trees(wl)
    run_case(wl, parents, W=4, scale=300.0, gates=False)


@pytest.mark.parametrize("W", [2, 3, 4, 8])
@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("in_place", [False, True])
def test_conv_commit_bit_exact(W, dtype, in_place):
    wl = dataclasses.replace(inputs.workload("c4"), B=6, H=3, T=50, dk=64, dv=40, qkv_dtype=dtype, seed=50 + W)
    parents, accepted = inputs.make_trees(wl)
    accepted = accepted.copy()
    accepted[0] = -1                      # nothing accepted: context unchanged
    accepted[1] = int(np.argmax(inputs.node_depths(parents[1])))   # the deepest path
    accepted[2] = 0                       # a single token: W-2 old rows survive
    ci = inputs.make_conv_inputs(wl, W=W)
    x, ctx = ci["x"].to(DEV), ci["ctx"].to(DEV)
    tree = tv.tree_build(parents).upload()
    acc = torch.from_numpy(accepted).to(DEV)
    buf, out = canary(tuple(ctx.shape), ctx.dtype)
    if in_place:
        out.copy_(ctx)
        tv.conv_commit(tree, acc, x, out, H=wl.H, dk=wl.dk, dv=wl.dv)
    else:
        ctx0 = ctx.clone()
        tv.conv_commit(tree, acc, x, ctx, H=wl.H, dk=wl.dk, dv=wl.dv, ctx_new=out)
        torch.cuda.synchronize()
        assert torch.equal(ctx, ctx0)
    torch.cuda.synchronize()
    assert canary_ok(buf, out.numel())
    xf, cf = inputs.to_f64(ci["x"]), inputs.to_f64(ci["ctx"])
    for b in range(wl.B):
        ref = cv.conv_commit(xf[b], cf[b], parents[b], int(accepted[b]))
        assert np.array_equal(out[b].cpu().double().numpy(), ref), b


def test_conv_then_commit_then_conv_matches_linear_sequence():
    """Two rounds on the GPU: the second round's outputs for a chain equal the oracle run over the
    committed linear sequence (context, accepted tokens, new tokens)."""
    wl = dataclasses.replace(inputs.workload("c2"), B=2, H=2, T=24, seed=9)
    parents, accepted = inputs.make_trees(wl)
    W = 4
    c1 = inputs.make_conv_inputs(wl, layer=0, W=W)
    c2 = inputs.make_conv_inputs(wl, layer=1, W=W)
    tree = tv.tree_build(parents).upload()
    ctx = c1["ctx"].to(DEV).clone()
    tv.conv_commit(tree, torch.from_numpy(accepted).to(DEV), c1["x"].to(DEV), ctx, H=wl.H, dk=wl.dk, dv=wl.dv)
    chain = np.tile(inputs.tree_chain(wl.T), (wl.B, 1))
    tree2 = tv.tree_build(chain).upload()
    q, k, v = tv.tree_conv(tree2, c2["x"].to(DEV), ctx, c1["weight"].to(DEV), c1["bias"].to(DEV),
                           H=wl.H, dk=wl.dk, dv=wl.dv)
    torch.cuda.synchronize()
    f1 = {n: inputs.to_f64(t) for n, t in c1.items()}
    x2 = inputs.to_f64(c2["x"])
    for b in range(wl.B):
        path = []
        j = int(accepted[b])
        while j >= 0:
            path.append(j); j = int(parents[b][j])
        path.reverse()
        seq = np.concatenate([f1["ctx"][b], f1["x"][b][path], x2[b]])
        n = seq.shape[0]
        y = cv.tree_conv(seq[W - 1:], seq[:W - 1], f1["weight"], f1["bias"], np.arange(-1, n - W))
        rq, rk, rv = cv.split_heads(y[n - (W - 1) - wl.T:], wl.H, wl.dk, wl.dv)
        close(q[b], rq, torch.bfloat16, "q")
        close(k[b], rk, torch.bfloat16, "k")
        close(v[b], rv, torch.bfloat16, "v")


def test_argument_errors():
    wl = dataclasses.replace(inputs.workload("c2"), B=2, H=2, T=16)
    parents, _ = inputs.make_trees(wl)
    ci = {n: t.to(DEV) for n, t in inputs.make_conv_inputs(wl, W=4).items()}
    kw = dict(H=wl.H, dk=wl.dk, dv=wl.dv)
    tree = tv.tree_build(parents)
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.tree_conv(tree, ci["x"], ci["ctx"], ci["weight"], **kw)
    assert e.value.status == -5
    tree.upload()
    # misaligned x
    flat = torch.zeros(ci["x"].numel() + 8, device=DEV, dtype=ci["x"].dtype)
    xm = flat[1:1 + ci["x"].numel()].view_as(ci["x"])
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_conv(tree, xm, ci["ctx"], ci["weight"], **kw)
    # aliased outputs
    q = torch.empty(wl.B, wl.H, wl.T, wl.dk, device=DEV, dtype=ci["x"].dtype)
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_conv(tree, ci["x"], ci["ctx"], ci["weight"], q=q, k=q, v=torch.empty_like(q), **kw)
    # tree of another size
    other = tv.tree_build(parents[:, :8].copy()).upload()
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_conv(other, ci["x"], ci["ctx"], ci["weight"], **kw)
    # too many taps, unsupported head width
    w9 = torch.zeros(ci["x"].shape[2], 9, device=DEV)
    c9 = torch.zeros(wl.B, 8, ci["x"].shape[2], device=DEV, dtype=ci["x"].dtype)
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_conv(tree, ci["x"], c9, w9, **kw)
    x12 = torch.zeros(wl.B, wl.T, 2 * 36, device=DEV, dtype=torch.bfloat16)
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_conv(tree, x12, torch.zeros(wl.B, 3, 72, device=DEV, dtype=torch.bfloat16),
                     torch.zeros(72, 4, device=DEV), H=2, dk=12, dv=12)
    # gates without their parameters
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_conv(tree, ci["x"], ci["ctx"], ci["weight"], gate_a=ci["gate_a"], **kw)
    torch.cuda.synchronize()
