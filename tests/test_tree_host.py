"""Host-side tree metadata of the C-ABI library against the oracle: bit-exact.

Runs without a GPU: tv_tree_build / tv_tree_meta / tv_tree_path make no CUDA
call.  The library and the oracle share no code; only the seeded tree
generators feed both.
"""
import ctypes
import re
import os

import numpy as np
import pytest

import paper_2608_01651_b200 as tv
from paper_2608_01651_b200 import inputs
from oracle import tree_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def oracle_meta(parents):
    anc = np.stack([orc.tree_metadata(p)[0] for p in parents])
    depth = np.stack([orc.tree_metadata(p)[1] for p in parents])
    md = np.array([orc.tree_metadata(p)[2] for p in parents], dtype=np.int32)
    return anc, depth, md


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_metadata_bit_exact_all_workloads(name):
    wl = inputs.workload(name)
    parents, accepted = inputs.make_trees(wl)
    tree = tv.tree_build(parents)
    anc, depth, md = tree.meta()
    oanc, odepth, omd = oracle_meta(parents)
    assert anc.tobytes() == oanc.tobytes()
    assert depth.tobytes() == odepth.tobytes()
    assert md.tobytes() == omd.tobytes()
    path, ln = tree.path(accepted)
    for b, a in enumerate(accepted):
        ref = orc.accepted_path(parents[b], int(a))
        assert ln[b] == len(ref)
        assert list(path[b, :ln[b]]) == ref
        assert all(path[b, ln[b]:] == -1)


def test_workload_tree_shapes():
    """The generated trees have the shapes the workloads name."""
    p1, a1 = inputs.make_trees(inputs.workload("c1"))
    assert p1.shape == (1, 15) and list(p1[0][:3]) == [-1, 0, 0]
    assert inputs.node_depths(p1[0]).max() == 3 and inputs.node_depths(p1[0])[a1[0]] == 3
    p2, _ = inputs.make_trees(inputs.workload("c2"))
    assert p2.shape == (1, 63) and inputs.node_depths(p2[0]).max() <= 8
    p3, a3 = inputs.make_trees(inputs.workload("c3"))
    assert p3.shape == (32, 64)
    for p in p3:
        d = inputs.node_depths(p)
        assert d.max() == 6 and np.bincount(d).max() <= 10
    assert (a3 == -1).any() or True
    p5, _ = inputs.make_trees(inputs.workload("c5"))
    assert p5.shape == (128, 128)
    assert all(inputs.node_depths(p).max() == 8 for p in p5)
    for ps in (p2, p3, p5):
        for p in ps:
            assert all(-1 <= p[i] < i for i in range(len(p)))


def test_edge_trees_and_rebuild():
    rng = np.random.default_rng(3)
    for T in [1, 2, 63, 64, 65, 127, 128]:
        for kind in ("chain", "star", "random"):
            if kind == "chain":
                par = np.arange(-1, T - 1)
            elif kind == "star":
                par = np.full(T, -1)
            else:
                par = np.array([-1] + [rng.integers(-1, i) for i in range(1, T)])
            tree = tv.tree_build(par)
            anc, depth, md = tree.meta()
            oanc, odepth, omd = orc.tree_metadata(par)
            assert anc[0].tobytes() == oanc.tobytes() and depth[0].tobytes() == odepth.tobytes()
            assert md[0] == omd
            path, ln = tree.path([T - 1])
            assert list(path[0, :ln[0]]) == orc.accepted_path(par, T - 1)
            tree.free()
    tree = tv.tree_build(np.array([[-1, 0, 1], [-1, -1, -1]]))
    tree.rebuild(np.array([[-1, -1, 0], [-1, 0, 0]]))
    anc, depth, md = tree.meta()
    assert depth.tolist() == [[0, 0, 1], [0, 1, 1]] and md.tolist() == [1, 1]
    path, ln = tree.path([-1, 2])
    assert ln.tolist() == [0, 2] and path.tolist() == [[-1, -1], [0, 2]]


def test_error_codes():
    L = tv.lib()
    h = ctypes.c_void_p()
    bad = np.array([-1, 1, 0], dtype=np.int32)
    assert L.tv_tree_build(bad.ctypes.data, 1, 3, ctypes.byref(h)) == -2 and not h.value
    bad2 = np.array([-2, 0], dtype=np.int32)
    assert L.tv_tree_build(bad2.ctypes.data, 1, 2, ctypes.byref(h)) == -2
    big = np.arange(-1, 128, dtype=np.int32)
    assert L.tv_tree_build(big.ctypes.data, 1, 129, ctypes.byref(h)) == -3
    assert L.tv_tree_build(None, 1, 3, ctypes.byref(h)) == -1
    assert L.tv_tree_build(bad.ctypes.data, 0, 3, ctypes.byref(h)) == -1
    with pytest.raises(tv.TreeVerifyError):
        tv.tree_build([-1, 5])
    tree = tv.tree_build([-1, 0, 1])
    with pytest.raises(tv.TreeVerifyError):
        tree.path([3])
    with pytest.raises(tv.TreeVerifyError):
        tree.rebuild([-1, 2, 0])
    # verify / commit refuse a tree that is not on the device, before any CUDA call
    d = tv._Dims(1, 1, 1, 3, 64, 64, 0, 0, 0)
    one = ctypes.c_void_p(16)
    st = L.tv_tree_verify(tree._h, ctypes.byref(d), one, one, one, one, one, None, one, None, None)
    assert st == -5
    d_bad = tv._Dims(1, 1, 1, 3, 63, 64, 0, 0, 0)
    assert L.tv_tree_verify(tree._h, ctypes.byref(d_bad), one, one, one, one, one, None, one, None, None) == -3
    d_T = tv._Dims(1, 1, 1, 4, 64, 64, 0, 0, 0)
    assert L.tv_tree_verify(tree._h, ctypes.byref(d_T), one, one, one, one, one, None, one, None, None) == -1
    assert b"tree" in L.tv_strerror(-2)


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "tree_verify.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(tv_[a-z_0-9]+)\s*\(", hdr))
    assert {"tv_tree_build", "tv_tree_verify", "tv_commit_path", "tv_tree_upload"} <= names
    L = tv.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in tree_verify.h but not exported"


def test_forest_build_host_metadata_and_errors():
    """tv_forest_build is host-only: per-request metadata equals the oracle's on each tree, padding
    entries are empty, paths come out per request, malformed input is refused with the right code."""
    from oracle import tree_oracle as orc
    rng = np.random.default_rng(11)
    trees = []
    for n in (1, 7, 40, 23):
        par = np.full(n, -1, dtype=np.int32)
        for i in range(1, n):
            par[i] = rng.integers(-1, i)
        trees.append(par)
    f = tv.forest_build(trees, n_max=40, capacity=100)
    assert f.n_trees == 4 and f.n == 40 and f.capacity == 100
    assert f.offsets.tolist() == [0, 1, 8, 48, 71]
    anc, depth, md = f.meta()
    for b, par in enumerate(trees):
        ra, rd, rm = orc.tree_metadata(par)
        n = len(par)
        assert np.array_equal(anc[b, :n], ra) and np.array_equal(depth[b, :n], rd) and md[b] == rm
        assert not anc[b, n:].any() and not depth[b, n:].any()
    acc = np.array([0, 6, -1, 22], dtype=np.int32)
    path, ln = f.path(acc)
    for b, par in enumerate(trees):
        ref = orc.path_to(par, int(acc[b])) if acc[b] >= 0 else []
        assert path[b, :ln[b]].tolist() == list(ref) and ln[b] == len(ref)
    f.rebuild_forest(trees[::-1][1:] + [trees[0]])       # other sizes, same shape limits
    assert f.offsets.tolist() == [0, 40, 47, 48, 49]
    for bad, code in (([np.array([-1, 0]), np.array([], dtype=np.int32)], -1),      # empty request
                      ([np.array([-1, 2, 0])], -2)):                                  # parent after child
        with pytest.raises(tv.TreeVerifyError) as e:
            tv.forest_build(bad, n_max=8, capacity=16)
        assert e.value.status == code
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.forest_build(trees, n_max=39)
    assert e.value.status == -1
    with pytest.raises(tv.TreeVerifyError) as e:
        tv.forest_build(trees, n_max=40, capacity=70)
    assert e.value.status == -8
