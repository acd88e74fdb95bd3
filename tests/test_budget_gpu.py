"""Budget selector on the GPU (tv_budget_select) against the oracle, bit for bit, and the
GPU-resident round it feeds: select -> forest metadata from device memory -> verify -> commit."""
import numpy as np
import pytest
import torch

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from oracle import budget_oracle as bo
from oracle import tree_oracle as orc
from tests.parity_util import rel_l2_rows, rel_fro

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def candidates(B, Tc, seed, ties=False):
    rng = np.random.Generator(np.random.Philox(key=seed))
    par = np.zeros((B, Tc), dtype=np.int32)
    for b in range(B):
        par[b] = inputs.tree_frontier(Tc, rng) if Tc > 1 else -1
        par[b, 0] = -1
    if ties:   # few distinct probabilities: many equal scores, exercises the tie order
        p = rng.choice(np.array([0.25, 0.5, 1.0], dtype=np.float32), size=(B, Tc))
    else:
        p = rng.uniform(0.02, 1.0, size=(B, Tc)).astype(np.float32)
    return par, p


CASES = [  # B, Tc, budget, ties
    (1, 1, 1, False), (3, 7, 9, False), (32, 64, 1234, False), (128, 128, 128 * 40, False),
    (16, 64, 16, False), (5, 33, 5 * 33, False), (5, 33, 10 ** 6, False),
    (8, 40, 100, True), (64, 128, 3000, True), (1024, 3, 2000, True),
]


@pytest.mark.parametrize("case", CASES)
def test_select_matches_oracle_bit_for_bit(case):
    B, Tc, budget, ties = case
    par, p = candidates(B, Tc, seed=B * 131 + Tc, ties=ties)
    budget_eff = min(budget, 4 * B * Tc)     # node_id is sized by the budget
    ref = bo.select(par, p, budget_eff)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    got = tv.budget_select(torch.from_numpy(par).to(DEV), torch.from_numpy(p).to(DEV), budget_eff, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(got["rho"].cpu().numpy().view(np.uint32), ref["rho"].view(np.uint32))
    assert np.array_equal(got["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(got["offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(got["parent_packed"].cpu().numpy(), ref["parent_packed"])
    node_id = got["node_id"].cpu().numpy()
    K = min(budget_eff, B * Tc)
    assert np.array_equal(node_id[:K], ref["node_id"][:K]) and (node_id[K:] == -1).all()


def test_invalid_parent_is_reported_not_followed():
    par, p = candidates(4, 16, seed=5)
    par[2, 7] = 9          # parent after child
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    got = tv.budget_select(torch.from_numpy(par).to(DEV), torch.from_numpy(p).to(DEV), 30, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -2
    assert int(got["offsets"][-1].item()) == 30
    with pytest.raises(tv.TreeVerifyError):
        tv.budget_select(torch.from_numpy(par).to(DEV), torch.from_numpy(p).to(DEV), 3)     # budget < roots


@pytest.mark.parametrize("rule", [inputs.GATED, inputs.DELTA])
def test_gpu_resident_round(rule):
    """Candidates and probabilities live on the GPU; the selected forest is verified and committed
    without the host touching the topology.  Checked per request against the tree oracle on the
    topology the selector oracle predicts."""
    B, H, Tc, budget = 6, 2, 64, 200
    wl = inputs.workload("c2", B=B, H=H, T=Tc, rule=rule, seed=23)
    par, p = candidates(B, Tc, seed=77)
    ref = bo.select(par, p, budget)
    sel = tv.budget_select(torch.from_numpy(par).to(DEV), torch.from_numpy(p).to(DEV), budget)
    # any forest of the same shape gives the handle; its topology is then replaced from the device
    forest = tv.forest_build([np.array([-1], dtype=np.int32)] * B, n_max=Tc, capacity=budget)
    forest.upload_device(sel["parent_packed"], sel["offsets"], max_depth_bound=8)
    with pytest.raises(tv.TreeVerifyError):
        forest.meta()                                   # the host copy is stale and says so
    # tensors of the candidates, gathered into packed planes by the selector's node ids (on the GPU)
    t = {n: (None if x is None else x.to(DEV)) for n, x in inputs.make_tensors(wl).items()}
    ids = sel["node_id"].long()

    def plane(x):        # [B,H,Tc,...] -> [H, budget, ...]
        flat = x.transpose(0, 1).reshape(H, B * Tc, *x.shape[3:])
        return flat.index_select(1, ids).contiguous()
    q, k, v, al = plane(t["q"]), plane(t["k"]), plane(t["v"]), plane(t["alpha"])
    be = None if t["beta"] is None else plane(t["beta"])
    O, U = tv.tree_verify(forest, t["S_pre"], q, k, v, al, be, rule=rule, want_U=True)
    accepted = np.array([int(c) - 1 for c in ref["counts"]], dtype=np.int32)    # last kept node of each request
    Sn = torch.empty_like(t["S_pre"])
    tv.commit_path(forest, torch.from_numpy(accepted).to(DEV), t["S_pre"], k, v, al, be, rule=rule, U=U, S_new=Sn)
    torch.cuda.synchronize()
    forest.device_status()
    f = inputs.to_f64
    On, Un, Snn = O.cpu().double().numpy(), U.cpu().double().numpy(), Sn.cpu().double().numpy()
    for b in range(B):
        n = int(ref["counts"][b])
        rows = slice(int(ref["offsets"][b]), int(ref["offsets"][b]) + n)
        keep = np.nonzero(ref["keep"][b])[0]
        pp = ref["parent_packed"][b, :n]
        for h in range(H):
            S = f(t["S_pre"][b, h].cpu()).T
            qq, kk, vv = f(t["q"][b, h].cpu())[keep], f(t["k"][b, h].cpu())[keep], f(t["v"][b, h].cpu())[keep]
            aa = f(t["alpha"][b, h].cpu())[keep]
            bb = None if t["beta"] is None else f(t["beta"][b, h].cpu())[keep]
            Or, Ur, _ = orc.verify_memo(S, qq, kk, vv, aa, bb, pp, wl.rule_name)
            Sr = orc.commit_walk(S, kk, vv, aa, bb, pp, int(accepted[b]), wl.rule_name).T
            assert rel_l2_rows(On[h, rows], Or) <= 2e-3
            assert rel_l2_rows(Un[h, rows], Ur) <= 2e-3
            assert rel_fro(Snn[b, h], Sr) <= 2e-3


def test_round_replays_from_a_cuda_graph_with_a_new_topology():
    """Section V-B: fixed addresses and kernel shapes, topology and node allocation change from
    round to round.  One round (select -> metadata -> verify -> commit) is captured once and
    replayed after the candidate trees, the probabilities and the tensors changed in place; the
    replay must equal an ordinary run on the new inputs."""
    B, H, Tc, budget = 8, 2, 64, 300
    wl = inputs.workload("c2", B=B, H=H, T=Tc, seed=31)
    forest = tv.forest_build([np.array([-1], dtype=np.int32)] * B, n_max=Tc, capacity=budget)
    par_d = torch.empty(B, Tc, dtype=torch.int32, device=DEV)
    p_d = torch.empty(B, Tc, dtype=torch.float32, device=DEV)
    planes = {"q": torch.empty(H, budget, 128, device=DEV, dtype=torch.bfloat16)}
    planes["k"] = torch.empty_like(planes["q"])
    planes["v"] = torch.empty_like(planes["q"])
    planes["alpha"] = torch.empty(H, budget, device=DEV)
    S = torch.empty(B, H, 128, 128, device=DEV)
    S_new = torch.empty_like(S)
    O = torch.empty(H, budget, 128, device=DEV)
    acc = torch.zeros(B, dtype=torch.int32, device=DEV)      # node 0 (the root) of every request
    sel = None

    def load_inputs(seed):
        par, p = candidates(B, Tc, seed=seed)
        par_d.copy_(torch.from_numpy(par)); p_d.copy_(torch.from_numpy(p))
        t = inputs.make_tensors(inputs.workload("c2", B=B, H=H, T=Tc, seed=seed))
        S.copy_(t["S_pre"])
        for n in ("q", "k", "v", "alpha"):     # candidate tensors land in the packed planes below
            planes[n].zero_()
        return par, p, t

    def round_(stream):
        nonlocal sel
        sel = tv.budget_select(par_d, p_d, budget, stream=stream, out=sel)
        forest.upload_device(sel["parent_packed"], sel["offsets"], max_depth_bound=8, stream=stream)
        tv.tree_verify(forest, S, planes["q"], planes["k"], planes["v"], planes["alpha"], O=O, stream=stream)
        tv.commit_path(forest, acc, S, planes["k"], planes["v"], planes["alpha"], S_new=S_new, stream=stream)

    def fill_planes(par, p, t):
        ref = bo.select(par, p, budget)
        ids = torch.from_numpy(ref["node_id"][:int(ref["offsets"][-1])].astype(np.int64)).to(DEV)
        n = ids.numel()
        for name in ("q", "k", "v", "alpha"):
            x = t[name].to(DEV)
            flat = x.transpose(0, 1).reshape(H, B * Tc, *x.shape[3:])
            planes[name][:, :n] = flat.index_select(1, ids)

    stream = torch.cuda.Stream()
    # warm-up outside the capture: allocations, attribute calls and tensor-map encodes happen here
    par, p, t = load_inputs(101)
    fill_planes(par, p, t)
    with torch.cuda.stream(stream):
        round_(stream)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        round_(stream)
    # new round: other trees, probabilities and tensors at the same addresses
    par, p, t = load_inputs(202)
    fill_planes(par, p, t)
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    O_graph, S_graph, off_graph = O.clone(), S_new.clone(), sel["offsets"].clone()
    O.zero_(); S_new.zero_()
    with torch.cuda.stream(stream):
        round_(stream)
    stream.synchronize()
    assert torch.equal(off_graph, sel["offsets"])
    n = int(off_graph[-1].item())
    assert torch.equal(O_graph[:, :n], O[:, :n]) and torch.equal(S_graph, S_new)
    ref = bo.select(par, p, budget)
    assert np.array_equal(off_graph.cpu().numpy(), ref["offsets"])


def test_depth_bound_is_checked_on_the_device():
    """tv_forest_upload_device is told a bound on the tree depth (it picks the kernels).  A forest
    that is deeper is reported by tv_tree_device_status and its masks are cut to the bound, so the
    delta-rule tensor-core kernel that the bound selected stays inside its tables; the next upload
    with an honest bound clears the report."""
    B, n = 3, 40
    chains = np.tile(np.arange(-1, n - 1, dtype=np.int32), (B, 1))          # depth n - 1 = 39
    offsets = torch.arange(0, (B + 1) * n, n, dtype=torch.int32, device=DEV)
    forest = tv.forest_build([np.array([-1], dtype=np.int32)] * B, n_max=n, capacity=B * n)
    par_d = torch.from_numpy(chains).to(DEV)
    forest.upload_device(par_d, offsets, max_depth_bound=8)
    anc, depth = forest.meta_device()
    assert int(depth.max()) == 8
    assert all(bin(int(anc[b, i, 0])).count("1") == min(i, 8) for b in range(B) for i in range(n))
    with pytest.raises(tv.TreeVerifyError) as e:
        forest.device_status()
    assert e.value.status == -3
    # the kernels chosen for depth <= 8 run on those masks without leaving their tables
    wl = inputs.workload("c4", B=B, H=2, T=n, seed=3)
    t = {k: (None if v is None else v.to(DEV)) for k, v in inputs.make_tensors(wl).items()}
    plane = lambda x: x.transpose(0, 1).reshape(x.shape[1], B * n, *x.shape[3:]).contiguous()
    O = torch.empty(2, B * n, 128, device=DEV)
    tv.tree_verify(forest, t["S_pre"], plane(t["q"]), plane(t["k"]), plane(t["v"]), plane(t["alpha"]),
                   plane(t["beta"]), rule=inputs.DELTA, O=O, impl=tv.IMPL_TC)
    torch.cuda.synchronize()
    assert torch.isfinite(O).all()
    # an honest bound: same handle, report gone, full masks
    forest.upload_device(par_d, offsets, max_depth_bound=n - 1)
    forest.device_status()
    anc, depth = forest.meta_device()
    assert int(depth.max()) == n - 1
    # and a host-side rebuild after a failed device upload starts clean as well
    forest.upload_device(par_d, offsets, max_depth_bound=2)
    forest.rebuild_forest([c for c in chains]).upload()
    forest.device_status()
