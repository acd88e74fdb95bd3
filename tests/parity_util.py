"""Shared helpers of the GPU parity tests (test infrastructure)."""
import numpy as np
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from oracle import tree_oracle as orc


def rel_l2_rows(x, ref):
    """max over rows of |x - ref|_2 / |ref|_2 (rows = last axis vectors)."""
    num = np.linalg.norm(x - ref, axis=-1)
    den = np.linalg.norm(ref, axis=-1)
    den = np.where(den == 0, 1.0, den)
    return float((num / den).max())


def rel_fro(x, ref):
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / (den if den else 1.0))


def with_canary(shape, device, pad=64):
    """Float tensor view of `shape` inside a buffer whose borders hold a canary."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * pad,), 12345.0, device=device, dtype=torch.float32)
    return buf, buf[pad:pad + n].view(*shape)


def canary_intact(buf, n, pad=64):
    return bool((buf[:pad] == 12345.0).all() and (buf[pad + n:] == 12345.0).all())


def gpu_round(wl, parents, accepted, tens, *, impl=tv.IMPL_AUTO, want_U=True, commit_with_U=False,
              in_place=False):
    """tree_build -> tree_verify -> commit_path through the C ABI on cuda:0."""
    dev = "cuda:0"
    t = {k: (None if v is None else v.to(dev)) for k, v in tens.items()}
    tree = tv.tree_build(parents).upload()
    S0 = t["S_pre"].clone()
    shape_O = tuple(t["v"].shape[:-1]) + (wl.dv,)
    Obuf, O = with_canary(shape_O, dev)
    Ubuf, U = with_canary(shape_O, dev) if want_U else (None, None)
    tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], t["beta"], rule=wl.rule,
                   O=O, U=U, impl=impl)
    torch.cuda.synchronize()
    assert torch.equal(t["S_pre"], S0), "verify must not write S_pre"
    assert canary_intact(Obuf, O.numel())
    if want_U:
        assert canary_intact(Ubuf, U.numel())
    acc = torch.from_numpy(np.asarray(accepted, dtype=np.int32)).to(dev)
    if in_place:
        Sbuf, Sn = with_canary(tuple(S0.shape), dev)
        Sn.copy_(S0)
        tv.commit_path(tree, acc, Sn, t["k"], t["v"], t["alpha"], t["beta"], rule=wl.rule,
                       U=U if commit_with_U else None)
    else:
        Sbuf, Sn = with_canary(tuple(S0.shape), dev)
        tv.commit_path(tree, acc, t["S_pre"], t["k"], t["v"], t["alpha"], t["beta"], rule=wl.rule,
                       U=U if commit_with_U else None, S_new=Sn)
    torch.cuda.synchronize()
    assert torch.equal(t["S_pre"], S0), "out-of-place commit must not write S_pre"
    assert canary_intact(Sbuf, Sn.numel())
    return (O.cpu().double().numpy(), None if U is None else U.cpu().double().numpy(),
            Sn.cpu().double().numpy(), tree)


def oracle_round(wl, parents, accepted, tens, items=None, layer=None):
    """Oracle outputs for the listed (b, h) items on the values the GPU got."""
    f = {k: inputs.to_f64(v) for k, v in tens.items()}
    if layer is not None:
        f = {k: (None if v is None else v[layer]) for k, v in f.items()}
    ver = orc.verify_batch(f["S_pre"], f["q"], f["k"], f["v"], f["alpha"], f["beta"], parents,
                           wl.rule_name, memo=True, items=items)
    com = orc.commit_batch(f["S_pre"], f["k"], f["v"], f["alpha"], f["beta"], parents, accepted,
                           wl.rule_name, items=items)
    return ver, com


def compare(wl, O, U, Sn, ver, com, layer=None):
    """Worst per-node relative L2 of O and U, worst per-state relative Frobenius."""
    eO = eU = eS = 0.0
    for (b, h), (Or, Ur) in ver.items():
        idx = (b, h) if layer is None else (layer, b, h)
        eO = max(eO, rel_l2_rows(O[idx], Or))
        if U is not None:
            eU = max(eU, rel_l2_rows(U[idx], Ur))
        eS = max(eS, rel_fro(Sn[idx], com[(b, h)]))
    return eO, eU, eS
