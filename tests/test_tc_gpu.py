"""Tensor-core verify kernel: smallest cases first, then several items per CTA."""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,T", [(1, 1, 128), (1, 1, 64), (1, 2, 37), (4, 8, 128), (40, 16, 100)])
def test_tc_gated(B, H, T):
    wl = inputs.workload("c5", B=B, H=H, T=T, L=1, tree="frontier", seed=11 + T)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    O, U, Sn, tree = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=True)
    tree.device_status()
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    eO, eU, eS = pu.compare(wl, O, U, Sn, ver, com)
    print(f"TC B{B} H{H} T{T}: rel-L2 O {eO:.3e} U {eU:.3e} S {eS:.3e}")
    assert eO <= wl.tol and eU == 0.0 and eS <= wl.tol


def test_tc_error_budget_report():
    """Mean and worst per-node error of the tensor-core path on c3 (printed)."""
    wl = inputs.workload("c3", B=4)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    O, _, Sn, tree = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=False)
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    errs = []
    for (b, h), (Or, _) in ver.items():
        errs.append(np.linalg.norm(O[b, h] - Or, axis=-1) / np.linalg.norm(Or, axis=-1))
    errs = np.concatenate(errs)
    print(f"TC c3 per-node rel-L2: mean {errs.mean():.3e} max {errs.max():.3e}")
    assert errs.max() <= wl.tol


@pytest.mark.parametrize("impl", [tv.IMPL_SIMT, tv.IMPL_TC])
@pytest.mark.parametrize("tree,mu", [("chain", -2.0), ("spine", -3.0), ("frontier", 8.0)])
def test_extreme_decay(tree, mu, impl):
    """Strong decay (path products far below fp32 range) and no decay at all:
    decay ratios are only ever formed on ancestor pairs, so nothing overflows."""
    wl = inputs.workload("c5", B=2, H=2, T=128, L=1, tree=tree, seed=77, alpha_mu=mu, alpha_sd=1.0)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    O, U, Sn, _ = pu.gpu_round(wl, parents, accepted, tens, impl=impl, want_U=False)
    assert np.isfinite(O).all() and np.isfinite(Sn).all()
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    eO, _, eS = pu.compare(wl, O, None, Sn, ver, com)
    print(f"decay mu={mu} {tree} impl={impl}: rel-L2 O {eO:.3e} S {eS:.3e}")
    assert eO <= wl.tol and eS <= wl.tol
