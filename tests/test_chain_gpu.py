"""Whole rounds queued on one stream without any synchronisation: upload -> Stage 1 -> verify ->
commit, twice over, every kernel a dependent launch of the one in front of it.  The results must be
bit for bit those of the same calls issued one at a time with a device synchronisation after each:
a kernel that read an input before the kernel producing it had finished, or wrote a buffer that an
older kernel was still reading, would show up as a difference."""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _round_calls(wl, rule, impl):
    parents, accepted = inputs.make_trees(wl)
    tree = tv.tree_build(parents)
    acc = torch.from_numpy(np.asarray(accepted, dtype=np.int32)).to(DEV)
    B, H, T, dk, dv = wl.B, wl.H, wl.T, wl.dk, wl.dv
    ci = [{k: v.to(DEV) for k, v in inputs.make_conv_inputs(wl, layer=r, device="cpu").items()} for r in range(2)]
    S0 = inputs.make_tensors(wl)["S_pre"].to(DEV)
    delta = rule == tv.DELTA

    def run(sync):
        S = S0.clone()
        ctx = [c["ctx"].clone() for c in ci]
        outs = []
        torch.cuda.synchronize()
        pause = torch.cuda.synchronize if sync else (lambda: None)
        for r in range(2):
            c = ci[r]
            tree.upload(); pause()
            q, k, v, al, be = tv.tree_conv(tree, c["x"], ctx[r], c["weight"], c["bias"], H=H, dk=dk, dv=dv,
                                           gate_a=c["gate_a"], gate_b=c["gate_b"], A_log=c["A_log"],
                                           dt_bias=c["dt_bias"], normalize_qk=True)
            pause()
            O = torch.empty(B, H, T, dv, device=DEV)
            U = torch.empty_like(O) if delta else None
            tv.tree_verify(tree, S, q, k, v, al, be if delta else None, rule=rule, O=O, U=U, impl=impl)
            pause()
            tv.commit_path(tree, acc, S, k, v, al, be if delta else None, rule=rule, U=U)   # in place
            pause()
            tv.conv_commit(tree, acc, c["x"], ctx[r], H=H, dk=dk, dv=dv)                      # in place
            pause()
            outs.append((q, k, v, al, be, O, U))
        torch.cuda.synchronize()
        tree.device_status()
        return S, ctx, outs

    return run


@pytest.mark.parametrize("name,B,H,T,rule,impl", [
    ("c3", 32, 32, 64, tv.GATED, tv.IMPL_AUTO),
    ("c3", 6, 8, 40, tv.GATED, tv.IMPL_AUTO),
    ("c4", 16, 32, 64, tv.DELTA, tv.IMPL_AUTO),
    ("c5", 24, 16, 128, tv.GATED, tv.IMPL_AUTO),
    ("c3", 5, 4, 33, tv.GATED, tv.IMPL_SIMT),
])
def test_unsynchronised_rounds_equal_synchronised_ones(name, B, H, T, rule, impl):
    wl = inputs.workload(name, B=B, H=H, T=T, L=1, seed=1234 + T)
    run = _round_calls(wl, rule, impl)
    S_ref, ctx_ref, outs_ref = run(sync=True)
    assert torch.isfinite(S_ref).all()
    for rep in range(3):
        S, ctx, outs = run(sync=False)
        assert torch.equal(S, S_ref), f"state differs (repeat {rep})"
        for a, b in zip(ctx, ctx_ref):
            assert torch.equal(a, b), f"context rows differ (repeat {rep})"
        for r, (got, ref) in enumerate(zip(outs, outs_ref)):
            for i, (x, y) in enumerate(zip(got, ref)):
                if y is None:
                    assert x is None
                else:
                    assert torch.equal(x, y), f"round {r}, output {i} differs (repeat {rep})"
