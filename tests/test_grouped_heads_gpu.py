"""Grouped key heads (Section IV-D: a K factor shared by several state heads is stored once):
q and k arrive with Hk < H heads; state head h reads q/k head h / (H / Hk)."""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from tests.parity_util import gpu_round, oracle_round, compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def grouped(tens, G):
    """Keep every G-th q/k head (the shared ones) and return (grouped, expanded) tensor sets."""
    g = dict(tens)
    e = dict(tens)
    for n in ("q", "k"):
        g[n] = tens[n][:, ::G].contiguous()
        e[n] = g[n].repeat_interleave(G, dim=1).contiguous()
    return g, e


CASES = [  # T, dk, dv, B, H, Hk
    (64, 128, 128, 3, 4, 2),
    (40, 128, 128, 2, 4, 1),
    (128, 128, 128, 1, 6, 3),
    (33, 64, 128, 2, 4, 2),
    (20, 64, 64, 2, 8, 2),
]


@pytest.mark.parametrize("impl", [tv.IMPL_AUTO, tv.IMPL_SIMT])
@pytest.mark.parametrize("rule", [inputs.GATED, inputs.DELTA])
@pytest.mark.parametrize("dtype", [inputs.BF16, inputs.F32])
@pytest.mark.parametrize("case", CASES)
def test_grouped_matches_oracle_and_expanded_call(case, dtype, rule, impl):
    T, dk, dv, B, H, Hk = case
    wl = inputs.workload("c2", T=T, dk=dk, dv=dv, B=B, H=H, rule=rule, qkv_dtype=dtype, seed=300 + T + Hk)
    parents, accepted = inputs.make_trees(wl)
    accepted[0] = -1 if T % 2 else accepted[0]
    tens_g, tens_e = grouped(inputs.make_tensors(wl), H // Hk)
    tol = 1e-5 if dtype == inputs.F32 else 2e-3
    for with_U in (False, True):
        O, U, Sn, _ = gpu_round(wl, parents, accepted, tens_g, impl=impl, commit_with_U=with_U)
        ver, com = oracle_round(wl, parents, accepted, tens_e)
        eO, eU, eS = compare(wl, O, U, Sn, ver, com)
        assert eO <= tol and eU <= tol and eS <= tol, (eO, eU, eS)
        # the same arithmetic on an explicitly expanded q/k: identical bits
        O2, U2, Sn2, _ = gpu_round(wl, parents, accepted, tens_e, impl=impl, commit_with_U=with_U)
        assert np.array_equal(O, O2) and np.array_equal(U, U2) and np.array_equal(Sn, Sn2)


def test_grouped_many_layers_in_one_commit():
    wl = inputs.workload("c3", B=4, H=8, L=3, seed=77)
    parents, accepted = inputs.make_trees(wl)
    G = 4
    layers = [grouped(inputs.make_tensors(wl, layer=l), G) for l in range(wl.L)]
    stack = lambda sel, n: torch.stack([x[sel][n] for x in layers]).to(DEV)
    tree = tv.tree_build(parents).upload()
    acc = torch.from_numpy(accepted).to(DEV)
    S = stack(0, "S_pre")
    outs = []
    for sel in (0, 1):
        Sn = torch.empty_like(S)
        O = tv.tree_verify(tree, S, stack(sel, "q"), stack(sel, "k"), stack(sel, "v"), stack(sel, "alpha"))
        tv.commit_path(tree, acc, S, stack(sel, "k"), stack(sel, "v"), stack(sel, "alpha"), S_new=Sn)
        torch.cuda.synchronize()
        outs.append((O.cpu(), Sn.cpu()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])


def test_grouped_session_round():
    wl = inputs.workload("c4", B=2, H=4, T=30, seed=5)
    parents, accepted = inputs.make_trees(wl)
    tens_g, tens_e = grouped(inputs.make_tensors(wl), 2)
    host = {n: (None if t is None else t.pin_memory()) for n, t in tens_g.items()}
    O = torch.empty(wl.B, wl.H, wl.T, wl.dv).pin_memory()
    Sn = torch.empty_like(host["S_pre"]).pin_memory()
    sess = tv.Session(1, wl.B, wl.H, wl.T, wl.dk, wl.dv, rule=wl.rule, qkv_dtype=wl.qkv_dtype, Hk=2)
    sess.round(parents, accepted, host["S_pre"], host["q"], host["k"], host["v"], host["alpha"], host["beta"],
               O, Sn)
    torch.cuda.synchronize()
    sess.free()
    ver, com = oracle_round(wl, parents, accepted, tens_e)
    eO, _, eS = compare(wl, O.double().numpy(), None, Sn.double().numpy(), ver, com)
    assert eO <= 2e-3 and eS <= 2e-3, (eO, eS)


def test_bad_group_counts():
    wl = inputs.workload("c2", B=1, H=4, T=16)
    parents, _ = inputs.make_trees(wl)
    t = {n: (None if x is None else x.to(DEV)) for n, x in inputs.make_tensors(wl).items()}
    tree = tv.tree_build(parents).upload()
    with pytest.raises(ValueError):
        tv.tree_verify(tree, t["S_pre"], t["q"][:, :3].contiguous(), t["k"][:, :3].contiguous(), t["v"], t["alpha"])
    d = tv._Dims(1, 1, 4, 16, 128, 128, 0, 1, 0, 3)
    import ctypes
    O = torch.empty(1, 4, 16, 128, device=DEV)
    st = tv.lib().tv_tree_verify(tree._h, ctypes.byref(d), tv._ptr(t["S_pre"]), tv._ptr(t["q"]), tv._ptr(t["k"]),
                                 tv._ptr(t["v"]), tv._ptr(t["alpha"]), None, tv._ptr(O), None, None)
    assert st == -1
