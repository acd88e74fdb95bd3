"""Host-buffer round (tv_session_round) and pre-marshalled calls against the oracle."""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,B,H,L", [("c3", 3, 4, 2), ("c4", 2, 4, 1), ("c1", 1, 4, 1)])
def test_session_round_matches_oracle(name, B, H, L):
    wl = inputs.workload(name, B=B, H=H, L=L)
    parents, accepted = inputs.make_trees(wl)
    layers = [inputs.make_tensors(wl, layer=l) for l in range(L)]
    host = {k: (None if layers[0][k] is None else torch.stack([x[k] for x in layers]).pin_memory())
            for k in layers[0]}
    O = torch.empty(L, B, H, wl.T, wl.dv).pin_memory()
    S_new = torch.empty_like(host["S_pre"]).pin_memory()
    sess = tv.Session(L, B, H, wl.T, wl.dk, wl.dv, rule=wl.rule, qkv_dtype=wl.qkv_dtype)
    S0 = host["S_pre"].clone()
    for _ in range(2):   # a session is reusable; the host state is not modified
        sess.round(parents, accepted, host["S_pre"], host["q"], host["k"], host["v"], host["alpha"],
                   host["beta"], O, S_new)
    assert torch.equal(host["S_pre"], S0)
    On, Sn = O.double().numpy(), S_new.double().numpy()
    for l in range(L):
        ver, com = pu.oracle_round(wl, parents, accepted, host, layer=l)
        eO, _, eS = pu.compare(wl, On, None, Sn, ver, com, layer=l)
        assert eO <= wl.tol and eS <= wl.tol, (l, eO, eS)
    sess.free()
    with pytest.raises(tv.TreeVerifyError):     # malformed tree is refused before any copy
        bad = parents.copy()
        bad[0, 1] = 5
        s2 = tv.Session(L, B, H, wl.T, wl.dk, wl.dv, rule=wl.rule, qkv_dtype=wl.qkv_dtype)
        s2.round(bad, accepted, host["S_pre"], host["q"], host["k"], host["v"], host["alpha"],
                 host["beta"], O, S_new)


@pytest.mark.parametrize("name,B,T", [("c4", 24, 64), ("c4", 12, 128), ("c3", 40, 64)])
def test_session_round_in_several_groups(name, B, T):
    """Enough traffic for three or more request groups (copy-in, kernel and copy-out streams chained
    per group): sampled items of every group against the oracle, all outputs finite."""
    H = 32
    wl = inputs.workload(name, B=B, H=H, T=T, L=1, seed=61 + B)
    parents, accepted = inputs.make_trees(wl)
    t = inputs.make_tensors(wl)
    host = {k: (None if v is None else v.unsqueeze(0).contiguous().pin_memory()) for k, v in t.items()}
    O = torch.full((1, B, H, T, wl.dv), float("nan")).pin_memory()
    S_new = torch.full_like(host["S_pre"], float("nan")).pin_memory()
    sess = tv.Session(1, B, H, T, wl.dk, wl.dv, rule=wl.rule, qkv_dtype=wl.qkv_dtype)
    sess.round(parents, accepted, host["S_pre"], host["q"], host["k"], host["v"], host["alpha"], host["beta"],
               O, S_new)
    sess.free()
    assert torch.isfinite(O).all() and torch.isfinite(S_new).all()     # every group wrote its rows
    rng = np.random.default_rng(B)
    items = [(int(b), int(rng.integers(H))) for b in sorted({0, B - 1, *rng.integers(0, B, 6).tolist()})]
    ver, com = pu.oracle_round(wl, parents, accepted, host, items=items, layer=0)
    eO, _, eS = pu.compare(wl, O.double().numpy(), None, S_new.double().numpy(), ver, com, layer=0)
    assert eO <= wl.tol and eS <= wl.tol, (eO, eS)


def test_prepared_calls_equal_direct_calls():
    wl = inputs.workload("c3", B=4, H=4)
    parents, accepted = inputs.make_trees(wl)
    t = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(wl).items()}
    tree = tv.tree_build(parents).upload()
    acc = torch.from_numpy(accepted).cuda()
    O1 = tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"])
    S1 = torch.empty_like(t["S_pre"])
    tv.commit_path(tree, acc, t["S_pre"], t["k"], t["v"], t["alpha"], S_new=S1)
    par = np.ascontiguousarray(parents, dtype=np.int32)
    refresh = tree.prepare_refresh(par)
    O2 = torch.empty_like(O1)
    S2 = torch.empty_like(S1)
    ver = tv.prepare_tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], O=O2)
    com = tv.prepare_commit_path(tree, acc, t["S_pre"], t["k"], t["v"], t["alpha"], S_new=S2)
    for _ in range(2):
        refresh(); ver(); com()
    torch.cuda.synchronize()
    assert torch.equal(O1, O2) and torch.equal(S1, S2)
    # the refresh re-reads the caller's parent array: a new topology changes the result
    par[:] = inputs.make_trees(inputs.workload("c3", B=4, H=4, seed=99))[0]
    refresh(); ver()
    torch.cuda.synchronize()
    assert not torch.equal(O1, O2)


def test_bounded_device_wait_reports_and_context_survives():
    """A wait that nothing satisfies runs out after its limit: the kernel reports a timeout
    status and returns; later launches on the same context work."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tv.selftest_wait_timeout(status)
    torch.cuda.synchronize()
    assert int(status.item()) == -6
    wl = inputs.workload("c2", B=1, H=2, T=20)
    parents, accepted = inputs.make_trees(wl)
    t = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(wl).items()}
    tree = tv.tree_build(parents).upload()
    O = tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"])
    tree.device_status()                      # no timeout in a real launch
    assert torch.isfinite(O).all()
