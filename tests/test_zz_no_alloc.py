"""tv_tree_verify_static: the entry point for callers that must not allocate.

Collected last on purpose (file name): it is an addition beside the paper's path, and a run
that stops at the first failure should already have run every other test.  The new entry is
called through the C ABI and compared with the regular entry point (tv_tree_build +
tv_tree_upload + tv_tree_verify) and with the fp64 oracle on the same inputs, twice in a row,
because the fixed device array it works in keeps the previous call's contents.
"""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _regular(wl, parents, t, want_U):
    tree = tv.tree_build(parents).upload()
    out = tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], t["beta"], rule=wl.rule,
                         want_U=want_U)
    torch.cuda.synchronize()
    return out if want_U else (out, None)


def _static(wl, parents_dev, t, want_U):
    O = torch.full(tuple(t["v"].shape[:-1]) + (wl.dv,), float("nan"), device="cuda")
    U = torch.full_like(O, float("nan")) if want_U else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tv.tree_verify_static(parents_dev, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], t["beta"],
                          rule=wl.rule, O=O, U=U, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return O, U


def _close(a, b, tol):
    a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
    num = np.linalg.norm(a - b, axis=-1)
    den = np.linalg.norm(b, axis=-1)
    return float((num / np.where(den == 0, 1.0, den)).max()) <= tol


@pytest.mark.parametrize("name,B,H", [("c3", 6, 4), ("c4", 3, 4), ("c1", 1, 4)])
def test_static_matches_regular_entry_point_twice(name, B, H):
    wl = inputs.workload(name, B=B, H=H)
    dev = lambda d: {k: (None if v is None else v.cuda()) for k, v in d.items()}
    # two different rounds back to back: the second must not see anything of the first
    for round_ in range(2):
        wl_r = inputs.workload(name, B=B, H=H, seed=wl.seed + 50 * round_)
        parents, _ = inputs.make_trees(wl_r)
        t_cpu = inputs.make_tensors(wl_r)
        t = dev(t_cpu)
        want_U = wl.rule == inputs.DELTA
        O_ref, U_ref = _regular(wl_r, parents, t, want_U)
        O, U = _static(wl_r, torch.from_numpy(parents).cuda(), t, want_U)
        assert torch.isfinite(O).all()
        # both entry points run the same kernels on the same metadata: same results, and in any
        # case within the tolerance of the parity tests
        assert _close(O, O_ref, wl.tol)
        if want_U:
            assert _close(U, U_ref, wl.tol)
        if wl.rule == inputs.GATED:
            assert torch.equal(O, O_ref)
        # and directly against the oracle, on every (request, head)
        ver, _ = pu.oracle_round(wl_r, parents, np.full(B, -1), t_cpu)
        On = O.cpu().double().numpy()
        Un = None if U is None else U.cpu().double().numpy()
        for (b, h), (Or, Ur) in ver.items():
            assert pu.rel_l2_rows(On[b, h], Or) <= wl.tol
            if want_U:
                assert pu.rel_l2_rows(Un[b, h], Ur) <= wl.tol


def test_static_shared_tree_capacity_and_bad_parents():
    wl = inputs.workload("c2", B=2, H=2, T=20)
    parents, _ = inputs.make_trees(wl, per_request=False)          # one tree for the batch
    t = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(wl).items()}
    O_ref, _ = _regular(wl, parents, t, False)
    O, _ = _static(wl, torch.from_numpy(parents).cuda(), t, False)
    assert torch.equal(O, O_ref)
    # more trees than the fixed array holds: refused with its own status, nothing launched
    big = inputs.workload("c2", B=tv.STATIC_MAX_TREES + 1, H=1, T=4, dk=64, dv=64)
    tb = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(big).items()}
    par = torch.full((big.B, big.T), -1, dtype=torch.int32, device="cuda")
    Ob = torch.empty(big.B, 1, big.T, 64, device="cuda")
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.tree_verify_static(par, tb["S_pre"], tb["q"], tb["k"], tb["v"], tb["alpha"], O=Ob)
    assert e.value.status == -8
    # a malformed parent array (device data cannot be checked on the host) is flagged, not followed
    bad = torch.from_numpy(parents).cuda().clone()
    bad[0, 3] = 7
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O2 = torch.empty_like(O)
    tv.tree_verify_static(bad, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], O=O2, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -2 and torch.isfinite(O2).all()


def test_static_call_allocates_nothing():
    wl = inputs.workload("c3", B=4, H=4)
    parents, _ = inputs.make_trees(wl)
    t = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(wl).items()}
    par = torch.from_numpy(parents).cuda()
    O = torch.empty(wl.B, wl.H, wl.T, wl.dv, device="cuda")
    tv.tree_verify_static(par, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], O=O)   # loads the kernels
    torch.cuda.synchronize()
    # handles left over from earlier tests free their device memory when they are collected:
    # do that now, not between the two readings
    import gc
    gc.collect()
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0 = torch.cuda.memory_allocated()
    for _ in range(3):
        tv.tree_verify_static(par, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], O=O)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_allocated() == alloc0
