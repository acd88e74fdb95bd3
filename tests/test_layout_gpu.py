"""Strided layouts (tv_dims strides) and per-layer pointer tables (tv_commit_path_layers).

Section IV-C folds "layout conversion" into the stages: a caller whose projections are
token-major [B, T, H, d], or slices of one fused projection [B, T, C], hands them over as they
are.  Section IV-D / V-B: all recurrent layers are committed by one launch even when every layer
owns its tensors.  Each case is checked against the oracle and, bit for bit, against the dense
head-major call on the same values (the kernels do the same arithmetic in the same order).
"""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def token_major(x):
    """A [B, H, T, ...] tensor re-laid as [B, T, H, ...] in memory, returned as a [B, H, T, ...] view."""
    return x.transpose(1, 2).contiguous().transpose(1, 2)


def dense_round(wl, tree, t, acc, impl):
    O = torch.empty(wl.B, wl.H, wl.T, wl.dv, device=DEV)
    U = torch.empty_like(O)
    tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], t["beta"], rule=wl.rule, O=O, U=U, impl=impl)
    Sn = torch.empty_like(t["S_pre"])
    tv.commit_path(tree, acc, t["S_pre"], t["k"], t["v"], t["alpha"], t["beta"], rule=wl.rule, U=U, S_new=Sn)
    return O, U, Sn


CASES = [  # name, B, H, T, rule, dtype, impl
    ("c3", 6, 4, 64, inputs.GATED, inputs.BF16, tv.IMPL_TC),
    ("c5", 3, 4, 128, inputs.GATED, inputs.BF16, tv.IMPL_TC),
    ("c5", 2, 3, 100, inputs.GATED, inputs.BF16, tv.IMPL_TC),
    ("c3", 3, 4, 37, inputs.GATED, inputs.BF16, tv.IMPL_SIMT),
    ("c4", 3, 4, 64, inputs.DELTA, inputs.BF16, tv.IMPL_AUTO),
    ("c4", 3, 4, 64, inputs.DELTA, inputs.BF16, tv.IMPL_TC),
    ("c4", 2, 3, 33, inputs.DELTA, inputs.BF16, tv.IMPL_TC),
    ("c4", 2, 2, 100, inputs.DELTA, inputs.BF16, tv.IMPL_TC),       # the kernel for 65..128 nodes
    ("c4", 2, 3, 128, inputs.DELTA, inputs.BF16, tv.IMPL_TC),
    ("c1", 2, 4, 15, inputs.GATED, inputs.F32, tv.IMPL_AUTO),
    ("c4", 2, 2, 40, inputs.DELTA, inputs.F32, tv.IMPL_AUTO),
]


@pytest.mark.parametrize("name,B,H,T,rule,dtype,impl", CASES)
def test_token_major_inputs_and_outputs(name, B, H, T, rule, dtype, impl):
    wl = inputs.workload(name, B=B, H=H, T=T, rule=rule, qkv_dtype=dtype, L=1, seed=500 + T)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    t = {k: (None if v is None else v.to(DEV)) for k, v in tens.items()}
    tree = tv.tree_build(parents).upload()
    acc = torch.from_numpy(accepted).to(DEV)
    O_d, U_d, S_d = dense_round(wl, tree, t, acc, impl)
    # the same values token-major: [B, T, H, d] in memory, handed over as strided views
    tm = {k: (None if t[k] is None else token_major(t[k])) for k in ("q", "k", "v", "alpha", "beta")}
    assert not tm["q"].is_contiguous()
    O_buf = torch.full((B, T, H, wl.dv), float("nan"), device=DEV)
    U_buf = torch.full((B, T, H, wl.dv), float("nan"), device=DEV)
    O, U = O_buf.transpose(1, 2), U_buf.transpose(1, 2)
    tv.tree_verify(tree, t["S_pre"], tm["q"], tm["k"], tm["v"], tm["alpha"], tm["beta"], rule=rule, O=O, U=U,
                   impl=impl)
    Sn = torch.empty_like(t["S_pre"])
    tv.commit_path(tree, acc, t["S_pre"], tm["k"], tm["v"], tm["alpha"], tm["beta"], rule=rule, U=U, S_new=Sn)
    Sn2 = torch.empty_like(t["S_pre"])
    tv.commit_path(tree, acc, t["S_pre"], tm["k"], tm["v"], tm["alpha"], tm["beta"], rule=rule, S_new=Sn2)
    torch.cuda.synchronize()
    tree.device_status()
    assert torch.isfinite(O_buf).all() and torch.isfinite(U_buf).all()
    # the same kernel runs on both layouts: identical bits
    assert torch.equal(O, O_d) and torch.equal(U, U_d) and torch.equal(Sn, S_d)
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    eO, eU, eS = pu.compare(wl, O.cpu().double().numpy(), U.cpu().double().numpy(), Sn.cpu().double().numpy(),
                            ver, com)
    eS2 = max(pu.rel_fro(Sn2[b, h].cpu().double().numpy(), com[(b, h)]) for (b, h) in com)
    assert max(eO, eU, eS, eS2) <= wl.tol, (eO, eU, eS, eS2)


@pytest.mark.parametrize("T,Hk", [(64, 4), (128, 2), (20, 1)])
def test_slices_of_one_fused_projection(T, Hk):
    """q, k, v read in place from one projection output [B, T, Hk*dk | Hk*dk | H*dv] (grouped key
    heads when Hk < H), gates from [B, T, 2, H]."""
    B, H, dk, dv = 3, 4, 128, 128
    wl = inputs.workload("c5", B=B, H=H, T=T, L=1, seed=900 + T)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    G = H // Hk
    q, k = tens["q"][:, ::G].contiguous(), tens["k"][:, ::G].contiguous()       # [B, Hk, T, dk]
    C = 2 * Hk * dk + H * dv
    x = torch.empty(B, T, C, dtype=torch.bfloat16)
    x[..., :Hk * dk] = q.transpose(1, 2).reshape(B, T, Hk * dk)
    x[..., Hk * dk:2 * Hk * dk] = k.transpose(1, 2).reshape(B, T, Hk * dk)
    x[..., 2 * Hk * dk:] = tens["v"].transpose(1, 2).reshape(B, T, H * dv)
    gates = torch.empty(B, T, 2, H)
    gates[:, :, 0] = tens["alpha"].transpose(1, 2)
    x, gates = x.to(DEV), gates.to(DEV)
    qv = x[..., :Hk * dk].view(B, T, Hk, dk).transpose(1, 2)
    kv = x[..., Hk * dk:2 * Hk * dk].view(B, T, Hk, dk).transpose(1, 2)
    vv = x[..., 2 * Hk * dk:].view(B, T, H, dv).transpose(1, 2)
    al = gates[:, :, 0].transpose(1, 2)
    S = tens["S_pre"].to(DEV)
    tree = tv.tree_build(parents).upload()
    O = torch.empty(B, T, H * dv, device=DEV)                  # what an output projection reads
    tv.tree_verify(tree, S, qv, kv, vv, al, O=O.view(B, T, H, dv).transpose(1, 2), impl=tv.IMPL_TC)
    acc = torch.from_numpy(accepted).to(DEV)
    Sn = torch.empty_like(S)
    tv.commit_path(tree, acc, S, kv, vv, al, S_new=Sn)
    torch.cuda.synchronize()
    tree.device_status()
    ref = dict(tens)
    ref["q"], ref["k"] = q.repeat_interleave(G, dim=1), k.repeat_interleave(G, dim=1)
    ver, com = pu.oracle_round(wl, parents, accepted, ref)
    On = O.view(B, T, H, dv).transpose(1, 2).cpu().double().numpy()
    eO, _, eS = pu.compare(wl, On, None, Sn.cpu().double().numpy(), ver, com)
    assert eO <= wl.tol and eS <= wl.tol, (eO, eS)


def test_bad_strides_are_refused():
    wl = inputs.workload("c3", B=2, H=2, T=16)
    parents, _ = inputs.make_trees(wl)
    t = {k: (None if v is None else v.to(DEV)) for k, v in inputs.make_tensors(wl).items()}
    tree = tv.tree_build(parents).upload()
    O = torch.empty(2, 2, 16, 128, device=DEV)
    # a channel-strided view cannot be described: refused by the binding
    wide = torch.zeros(2, 2, 16, 256, device=DEV, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], wide[..., ::2], t["alpha"], O=O)
    # strides that are not multiples of 16 bytes: refused by the library
    import ctypes
    d = tv._dims(t["S_pre"], t["k"], t["v"], tv.GATED, tv.IMPL_AUTO)
    d.v = tv._Strides(4096 + 4, 2048 + 4, 128 + 4)
    st = tv.lib().tv_tree_verify(tree._h, ctypes.byref(d), t["S_pre"].data_ptr(), t["q"].data_ptr(), t["k"].data_ptr(),
                                 t["v"].data_ptr(), t["alpha"].data_ptr(), None, O.data_ptr(), None, None)
    assert st == -1
    # a packed forest keeps its planes
    forest = tv.forest_build([parents[0], parents[1]], n_max=16, capacity=32).upload()
    d2 = tv._dims(t["S_pre"], t["k"], t["v"], tv.GATED, tv.IMPL_AUTO)
    d2.qk = tv._Strides(4096, 128, 256)
    st = tv.lib().tv_tree_verify(forest._h, ctypes.byref(d2), t["S_pre"].data_ptr(), t["q"].data_ptr(),
                                 t["k"].data_ptr(), t["v"].data_ptr(), t["alpha"].data_ptr(), None, O.data_ptr(), None,
                                 None)
    assert st == -3


LAYER_CASES = [  # name, L, B, H, T, rule, with_U, in_place
    ("c3", 4, 4, 4, 64, inputs.GATED, False, True),
    ("c3", 3, 4, 4, 50, inputs.GATED, False, False),
    ("c4", 4, 3, 4, 64, inputs.DELTA, True, True),
    ("c4", 2, 3, 2, 40, inputs.DELTA, False, False),      # corrections re-derived along the path
    ("c3", 4, 32, 32, 64, inputs.GATED, False, True),     # large enough for the persistent kernel
    ("c1", 3, 2, 4, 15, inputs.GATED, False, True),       # fp32, dk = 64: the general kernel
]


@pytest.mark.parametrize("name,L,B,H,T,rule,with_U,in_place", LAYER_CASES)
def test_commit_layers_equals_the_stacked_call(name, L, B, H, T, rule, with_U, in_place):
    wl = inputs.workload(name, B=B, H=H, T=T, rule=rule, L=L, seed=70 + L + T)
    parents, accepted = inputs.make_trees(wl)
    layers = [{k: (None if v is None else v.to(DEV)) for k, v in inputs.make_tensors(wl, layer=l).items()}
              for l in range(L)]
    stack = {k: (None if layers[0][k] is None else torch.stack([x[k] for x in layers])) for k in layers[0]}
    tree = tv.tree_build(parents).upload()
    acc = torch.from_numpy(accepted).to(DEV)
    U_st = None
    if with_U:
        U_st = torch.empty(L, B, H, T, wl.dv, device=DEV)
        for l in range(L):
            tv.tree_verify(tree, stack["S_pre"][l], stack["q"][l], stack["k"][l], stack["v"][l], stack["alpha"][l],
                           stack["beta"][l], rule=rule, O=torch.empty(B, H, T, wl.dv, device=DEV), U=U_st[l])
    # reference: the stacked call
    S_ref = torch.empty_like(stack["S_pre"])
    tv.commit_path(tree, acc, stack["S_pre"], stack["k"], stack["v"], stack["alpha"], stack["beta"], rule=rule,
                   U=U_st, S_new=S_ref)
    # the same layers as separately allocated tensors (with spacers in between so that nothing is adjacent)
    spacer = []
    sep = {k: [] for k in ("S_pre", "k", "v", "alpha", "beta", "U")}
    for l in range(L):
        for key in ("S_pre", "k", "v", "alpha", "beta"):
            sep[key].append(None if layers[l][key] is None else layers[l][key].clone())
            spacer.append(torch.empty(1000 + 37 * l, device=DEV))
        sep["U"].append(None if U_st is None else U_st[l].clone())
    lists = {k: (None if sep[k][0] is None else sep[k]) for k in sep}
    S0 = [s.clone() for s in sep["S_pre"]]
    if in_place:
        out = tv.commit_path_layers(tree, acc, lists["S_pre"], lists["k"], lists["v"], lists["alpha"], lists["beta"],
                                    rule=rule, U=lists["U"])
    else:
        out = [torch.empty_like(s) for s in sep["S_pre"]]
        tv.commit_path_layers(tree, acc, lists["S_pre"], lists["k"], lists["v"], lists["alpha"], lists["beta"],
                              rule=rule, U=lists["U"], S_new=out)
    torch.cuda.synchronize()
    for l in range(L):
        assert torch.equal(out[l], S_ref[l]), f"layer {l}"
        if not in_place:
            assert torch.equal(sep["S_pre"][l], S0[l])
    # and against the oracle on a sample
    f = inputs.to_f64
    for l in (0, L - 1):
        tl = {k: (None if v is None else v.cpu()) for k, v in layers[l].items()}
        items = [(0, 0), (B - 1, H - 1)]
        _, com = pu.oracle_round(wl, parents, accepted, tl, items=items)
        for (b, h) in items:
            assert pu.rel_fro(f(out[l][b, h].cpu()), com[(b, h)]) <= wl.tol


def test_commit_layers_argument_errors():
    wl = inputs.workload("c3", B=2, H=2, T=16, L=2)
    parents, accepted = inputs.make_trees(wl)
    ls = [{k: (None if v is None else v.to(DEV)) for k, v in inputs.make_tensors(wl, layer=l).items()} for l in range(2)]
    tree = tv.tree_build(parents).upload()
    acc = torch.from_numpy(accepted).to(DEV)
    S, k, v, al = ([x[key] for x in ls] for key in ("S_pre", "k", "v", "alpha"))
    with pytest.raises(ValueError):
        tv.commit_path_layers(tree, acc, S, k[:1], v, al)
    # in place for one layer, out of place for the other: refused
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.commit_path_layers(tree, acc, S, k, v, al, S_new=[S[0], torch.empty_like(S[1])])
    assert e.value.status == -1
    # an output that overlaps another layer's input: refused
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.commit_path_layers(tree, acc, S, k, v, al, S_new=[S[1], S[0]])
    assert e.value.status == -1
