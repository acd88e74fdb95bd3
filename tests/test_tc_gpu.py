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


@pytest.mark.parametrize("T", [64, 100])
def test_ordinary_and_extreme_decay_items_alternate_on_one_cta(T):
    """More items than SMs, and the decay of an item depends on the pass in which a CTA meets it:
    ordinary gates in the first pass, path products far below fp32 range in the second, ordinary
    again in the third.  The two forms of the kernel (plain, and row exponents with a rescaled q
    copy) then follow each other item by item on every CTA."""
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    B, H = 8, 40
    wl = inputs.workload("c5", B=B, H=H, T=T, L=1, tree="frontier", seed=91)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    item = torch.arange(B * H).view(B, H)
    second_pass = ((item // n_sm) % 2 == 1)
    g = torch.Generator().manual_seed(5)
    harsh = torch.sigmoid(torch.randn(B, H, T, generator=g) - 14.0).clamp_min(1e-9)   # alpha ~ 1e-6: |g| > 100 from depth 5 on
    tens["alpha"] = torch.where(second_pass[:, :, None], harsh, tens["alpha"])
    O, U, Sn, _ = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=False)
    assert np.isfinite(O).all() and np.isfinite(Sn).all()
    picks = [(b, h) for b in range(B) for h in range(H) if (b * H + h) % 23 == 0]
    picks += [(int(i) // H, int(i) % H) for i in (n_sm - 1, n_sm, n_sm + 1, 2 * n_sm - 1, 2 * n_sm, B * H - 1)
              if i < B * H]
    ver, com = pu.oracle_round(wl, parents, accepted, tens, items=sorted(set(picks)))
    eO, _, eS = pu.compare(wl, O, None, Sn, ver, com)
    assert eO <= wl.tol and eS <= wl.tol, (eO, eS)


@pytest.mark.parametrize("B,H,T,tree", [(1, 1, 64, "frontier"), (1, 2, 37, "frontier"), (2, 3, 1, "chain"),
                                         (3, 4, 16, "chain"), (16, 32, 64, "frontier"), (5, 7, 50, "levels")])
def test_tc_delta(B, H, T, tree):
    """Delta rule on the tensor cores: O and the corrections U against the oracle."""
    wl = inputs.workload("c4", B=B, H=H, T=T, L=1, tree=tree, seed=23 + T)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    O, U, Sn, tree_h = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=True,
                                    commit_with_U=True, in_place=True)
    tree_h.device_status()
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    eO, eU, eS = pu.compare(wl, O, U, Sn, ver, com)
    print(f"TC delta B{B} H{H} T{T} {tree}: rel-L2 O {eO:.3e} U {eU:.3e} S {eS:.3e}")
    assert eO <= wl.tol and eU <= wl.tol and eS <= wl.tol
    O2, _, _, _ = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=False)
    assert np.array_equal(O2, O)          # asking for U does not change O


@pytest.mark.parametrize("B,H,T,tree", [(1, 1, 128, "frontier"), (1, 2, 65, "frontier"), (2, 3, 96, "binary"),
                                         (3, 2, 127, "frontier"), (8, 32, 128, "frontier"), (2, 2, 100, "spine")])
def test_tc_delta_large_trees(B, H, T, tree):
    """Delta rule, 64 < T <= 128: the two-row-block tensor-core kernel against the oracle, O and U,
    per-request trees; asking for U must not change O."""
    wl = inputs.workload("c4", B=B, H=H, T=T, L=1, tree=tree, seed=41 + T)
    parents, accepted = inputs.make_trees(wl)
    assert max(int(inputs.node_depths(par).max()) for par in parents) <= 15   # what the kernel takes
    tens = inputs.make_tensors(wl)
    O, U, Sn, tree_h = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=True,
                                    commit_with_U=True, in_place=True)
    tree_h.device_status()
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    eO, eU, eS = pu.compare(wl, O, U, Sn, ver, com)
    print(f"TC delta (large trees) B{B} H{H} T{T} {tree}: rel-L2 O {eO:.3e} U {eU:.3e} S {eS:.3e}")
    assert eO <= wl.tol and eU <= wl.tol and eS <= wl.tol
    O2, _, _, _ = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=False)
    assert np.array_equal(O2, O)          # asking for U does not change O
    O3, _, _, _ = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=True)
    assert np.array_equal(O3, O)          # run to run identical


@pytest.mark.parametrize("T", [64, 128])
def test_tc_delta_depth_15(T):
    """Trees of depth 9..15 take the deeper instantiation of the row solve (both tree sizes)."""
    B, H = 3, 2
    wl = inputs.workload("c4", B=B, H=H, T=T, L=1, seed=97 + T)
    rng = np.random.default_rng(5 + T)
    parents = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        par, dep = [-1], [0]
        for i in range(1, T):
            if i <= 15:
                p = i - 1                                   # a spine down to depth 15
            else:
                p = int(rng.choice([j for j in range(i) if dep[j] < 15]))
            par.append(p)
            dep.append(dep[p] + 1)
        assert max(dep) == 15
        parents[b] = par
    accepted = np.array([15, T - 1, -1], dtype=np.int32)
    tens = inputs.make_tensors(wl)
    O, U, Sn, tree_h = pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=True,
                                    commit_with_U=True, in_place=True)
    tree_h.device_status()
    ver, com = pu.oracle_round(wl, parents, accepted, tens)
    eO, eU, eS = pu.compare(wl, O, U, Sn, ver, com)
    print(f"TC delta depth 15, T{T}: rel-L2 O {eO:.3e} U {eU:.3e} S {eS:.3e}")
    assert eO <= wl.tol and eU <= wl.tol and eS <= wl.tol


@pytest.mark.parametrize("T", [64, 100, 128])
def test_tc_delta_run_to_run_identical(T):
    """Several items per CTA, U requested and not, repeated: O and U identical bit for bit.  (A slot
    table overwritten by a fast warp while a slow one still read it once showed up exactly here.)"""
    wl = inputs.workload("c4", B=16, H=32, T=T, L=1, tree="frontier", seed=23 + T)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    outs = [pu.gpu_round(wl, parents, accepted, tens, impl=tv.IMPL_TC, want_U=w)[:2]
            for w in (True, True, False, False, True, False)]
    for O, U in outs[1:]:
        assert np.array_equal(O, outs[0][0])
        if U is not None:
            assert np.array_equal(U, outs[0][1])


@pytest.mark.parametrize("T,B,H", [(64, 32, 32), (128, 20, 32), (40, 24, 20)])
def test_tc_gated_run_to_run_identical(T, B, H):
    """Several items per CTA, many launches back to back on the same inputs: O identical bit for
    bit every time (the roles of the kernel hand buffers to each other through barriers only; a
    buffer reused one hand-over too early shows up as a run that differs)."""
    wl = inputs.workload("c5" if T > 64 else "c3", B=B, H=H, T=T, L=1, tree="frontier", seed=31 + T)
    parents, accepted = inputs.make_trees(wl)
    t = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(wl).items()}
    tree = tv.tree_build(parents).upload()
    first = None
    for i in range(24):
        O = torch.full((B, H, T, wl.dv), float("nan"), device="cuda")
        tv.tree_verify(tree, t["S_pre"], t["q"], t["k"], t["v"], t["alpha"], O=O, impl=tv.IMPL_TC)
        if first is None:
            first = O
        else:
            assert torch.equal(O, first), f"launch {i} differs"
    torch.cuda.synchronize()
    tree.device_status()
    assert torch.isfinite(first).all()


def test_in_place_commits_with_only_an_upload_between():
    """commit (in place) -> tree upload -> commit (in place) on one stream, nothing else and no
    synchronisation in between.  Every kernel in that chain is a dependent launch, and the commit
    kernel fetches its state rows before its own wait: the second commit must not be scheduled
    while the first one still writes those rows (a kernel releases its dependents only after its
    own wait, so a dependent never runs beside anything older than the kernel in front of it)."""
    from oracle import tree_oracle as orc
    wl = inputs.workload("c3", B=32, H=32, T=64, L=1, seed=91)
    parents, accepted = inputs.make_trees(wl)
    tens = inputs.make_tensors(wl)
    t = {k: (None if v is None else v.cuda()) for k, v in tens.items()}
    acc = torch.from_numpy(np.asarray(accepted, dtype=np.int32)).cuda()
    tree = tv.tree_build(parents).upload()
    items = [(0, 0), (7, 31), (19, 5), (31, 31)]
    f = {k: inputs.to_f64(v) for k, v in tens.items()}
    once = orc.commit_batch(f["S_pre"], f["k"], f["v"], f["alpha"], None, parents, accepted, wl.rule_name, items=items)
    S1 = np.array(f["S_pre"], dtype=np.float64, copy=True)
    for (b, h), Sn in once.items():
        S1[b, h] = Sn
    twice = orc.commit_batch(S1, f["k"], f["v"], f["alpha"], None, parents, accepted, wl.rule_name, items=items)
    for rep in range(6):
        S = t["S_pre"].clone()
        torch.cuda.synchronize()
        tv.commit_path(tree, acc, S, t["k"], t["v"], t["alpha"])
        tree.upload()
        tv.commit_path(tree, acc, S, t["k"], t["v"], t["alpha"])
        torch.cuda.synchronize()
        Sh = S.cpu().double().numpy()
        for (b, h), Sr in twice.items():
            assert pu.rel_fro(Sh[b, h], Sr) <= 1e-5, (rep, b, h)


def test_tc_delta_falls_back_on_deep_trees():
    wl = inputs.workload("c4", B=1, H=2, T=40, tree="chain", seed=5)   # depth 39 > 15
    parents, accepted = inputs.make_trees(wl)
    tens = {k: (None if v is None else v.cuda()) for k, v in inputs.make_tensors(wl).items()}
    tree = tv.tree_build(parents).upload()
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.tree_verify(tree, tens["S_pre"], tens["q"], tens["k"], tens["v"], tens["alpha"], tens["beta"],
                       rule=tv.DELTA, impl=tv.IMPL_TC)
    assert e.value.status == -3
    O = tv.tree_verify(tree, tens["S_pre"], tens["q"], tens["k"], tens["v"], tens["alpha"], tens["beta"],
                       rule=tv.DELTA)            # AUTO takes the SIMT kernel
    torch.cuda.synchronize()
    assert torch.isfinite(O).all()


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c5"])
def test_device_built_metadata_bit_exact(name):
    """Masks and depths derived by the device kernel equal the host's and the oracle's."""
    from oracle import tree_oracle as orc
    wl = inputs.workload(name)
    parents, _ = inputs.make_trees(wl)
    tree = tv.tree_build(parents).upload()
    anc_d, depth_d = tree.meta_device()
    anc_h, depth_h, _ = tree.meta()
    assert anc_d.tobytes() == anc_h.tobytes() and depth_d.tobytes() == depth_h.tobytes()
    for t in (0, len(parents) - 1):
        oanc, odepth, _ = orc.tree_metadata(parents[t])
        assert anc_d[t].tobytes() == oanc.tobytes() and depth_d[t].tobytes() == odepth.tobytes()
    tree.rebuild(parents[::-1].copy()).upload()       # new topology, same buffers
    anc_d2, depth_d2 = tree.meta_device()
    anc_h2, depth_h2, _ = tree.meta()
    assert anc_d2.tobytes() == anc_h2.tobytes() and depth_d2.tobytes() == depth_h2.tobytes()
