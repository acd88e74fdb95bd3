#!/usr/bin/env python
"""Benchmark of the tree-verification hot path on B200.

A step is one pass of the whole path over one batch of synthetic trees:
tree_build (host metadata + upload) -> tree_verify for every layer ->
commit_path over all layers, through the C ABI of libtreeverify.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3]
    python bench.py --impl reference ...      # the fp64 CPU oracle, timed

Prints ONE JSON line on rank 0.  ``value`` = verified tree nodes per second
per recurrent layer (B*T*L nodes per step over the step time, all ranks
summed), inputs resident in HBM; ``e2e`` = the same with HOST buffers through
tv_session_round (copies inside the timed region); ``roofline`` = achieved
algorithmic HBM GB/s of the verify kernel against the measured copy peak;
``cpu_baseline`` = the oracle on a bounded sample on the host cores.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_01651_b200 import inputs  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 * 2 ** 20

DESCR = {
    "c1": "c1: B1 H4 T15 dk=dv=64 gated, f32 q/k/v, f32 state",
    "c2": "c2: B1 H16 T63 dk=dv=128 gated, bf16 q/k/v, f32 state",
    "c3": "c3: B32 H32 T64 dk=dv=128 gated, bf16 q/k/v, f32 state, draft-style level trees",
    "c4": "c4: B16 H32 T64 dk=dv=128 gated delta rule, bf16 q/k/v, f32 state",
    "c5": "c5: B128 H32 T128 dk=dv=128 gated, bf16 q/k/v, f32 state, 48 layers",
}


# --------------------------------------------------------------------------
# Algorithmic bytes: what the method must move per launch (state once, q/k/v once, outputs once)
# --------------------------------------------------------------------------
def verify_bytes_per_layer(wl, with_U: bool) -> int:
    eb = 2 if wl.qkv_dtype == inputs.BF16 else 4
    per = 4 * wl.dk * wl.dv + eb * wl.T * (2 * wl.dk + wl.dv) + 4 * wl.T + 4 * wl.T * wl.dv
    if wl.rule == inputs.DELTA:
        per += 4 * wl.T
    if with_U:
        per += 4 * wl.T * wl.dv
    return per * wl.B * wl.H


def commit_bytes_per_layer(wl, acc_len: np.ndarray, with_U: bool) -> int:
    """In-place commit: requests that accept nothing move no bytes."""
    eb = 2 if wl.qkv_dtype == inputs.BF16 else 4
    tot = 0
    for ln in acc_len:
        if ln > 0:
            tot += wl.H * (8 * wl.dk * wl.dv + ln * (eb * wl.dk + (4 if with_U else eb) * wl.dv))
    return tot


def accepted_lengths(parents, accepted):
    out = []
    for b, a in enumerate(accepted):
        d = inputs.node_depths(parents[b if parents.shape[0] > 1 else 0])
        out.append(0 if a < 0 else int(d[a]) + 1)
    return np.array(out)


def ncu_traffic(workload: str):
    """DRAM bytes per verify launch from the committed ncu capture of this workload, if any."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        return json.load(open(p)).get(workload, {}).get("tree_verify")
    except Exception:
        return None


def _jsonable(o):
    return o.item() if hasattr(o, "item") else str(o)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------
# Clock sampling during the timed region
# --------------------------------------------------------------------------
class ClockSampler:
    Q = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(index), "-lms", "10"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def wait_ready(self, timeout: float = 3.0):
        """nvidia-smi takes a few hundred ms to deliver its first sample: wait for it."""
        t0 = time.time()
        while self.p is not None and time.time() - t0 < timeout:
            if os.path.getsize(self.f.name) > 0:
                return
            time.sleep(0.01)

    def _samples(self):
        import datetime
        out = []
        with open(self.f.name) as fh:
            for line in fh.read().splitlines():
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    out.append((ts, float(parts[1]), float(parts[2]), parts[3:7]))
                except ValueError:
                    continue
        return out

    def window(self, w0: float, w1: float) -> dict:
        """Median SM clock and the throttle reasons seen between wall-clock times w0 and w1."""
        time.sleep(0.03)   # let the last sample of the window reach the file
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        sm, mx, reasons = [], [], set()
        for ts, c, m, flags in self._samples():
            if w0 <= ts <= w1:
                sm.append(c); mx.append(m)
                for n, v in zip(names, flags):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}

    def stop(self):
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
        self.f.close()
        os.unlink(self.f.name)


def sample_clocks(sampler, w0: float, w1: float, replay):
    """Clocks during the timed region [w0, w1]; if the region was too short for nvidia-smi to
    sample it, during an untimed replay of the same step loop right after it."""
    if sampler is None or sampler.p is None:
        return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
    c = sampler.window(w0, w1)
    c["sampled"] = "timed region"
    if c["samples"] < 3:
        r0 = time.time()
        while time.time() - r0 < 0.4:
            replay()
        torch.cuda.synchronize()
        c = sampler.window(r0, time.time())
        c["sampled"] = "untimed replay of the step loop (the timed region was too short to sample)"
    sampler.stop()
    return c


# --------------------------------------------------------------------------
# CPU baseline: the oracle, as it stands, on a bounded sample
# --------------------------------------------------------------------------
def oracle_sample(wl, parents, accepted, tens_cpu, budget_s: float, max_items: int):
    """Time the oracle (verify + commit) on (b,h) items until the budget is spent.
    Returns (nodes/s per layer, items, seconds, threads)."""
    from oracle import tree_oracle as orc
    try:
        from threadpoolctl import threadpool_limits
        ctx = threadpool_limits(limits=1)
        threads = 1
    except Exception:
        import contextlib
        ctx = contextlib.nullcontext()
        threads = os.cpu_count() or 1
    f = {k: inputs.to_f64(v) for k, v in tens_cpu.items()}
    done = 0
    t0 = time.perf_counter()
    with ctx:
        for b in range(wl.B):
            for h in range(wl.H):
                orc.verify_batch(f["S_pre"], f["q"], f["k"], f["v"], f["alpha"], f["beta"], parents,
                                 wl.rule_name, memo=True, items=[(b, h)])
                orc.commit_batch(f["S_pre"], f["k"], f["v"], f["alpha"], f["beta"], parents, accepted,
                                 wl.rule_name, items=[(b, h)])
                done += 1
                if time.perf_counter() - t0 > budget_s or done >= max_items:
                    break
            else:
                continue
            break
    dt = time.perf_counter() - t0
    # one "node" of the metric is a tree node through all H heads of a layer
    return done * wl.T / wl.H / dt, done, dt, threads


def slice_request(wl, tens, nb):
    return {k: (None if v is None else v[:nb].contiguous()) for k, v in tens.items()}


def run_reference(args, wl, rank, world):
    """--impl reference: the CPU oracle timed on bounded samples."""
    if rank != 0:
        return
    parents, accepted = inputs.make_trees(wl)
    nb = min(wl.B, 2)
    small = inputs.workload(wl.name, B=nb, L=1)
    tens = inputs.make_tensors(small)
    items_per_step = max(1, min(nb * wl.H, args.ref_items))
    vals = []
    threads = 1
    for s in range(args.warmup + args.steps):
        v, done, dt, threads = oracle_sample(small, parents[:nb] if parents.shape[0] > 1 else parents,
                                             accepted[:nb], tens, 1e9, items_per_step)
        if s >= args.warmup:
            vals.append((v, dt))
    value = float(np.mean([v for v, _ in vals]))
    ms = float(np.mean([dt for _, dt in vals]) * 1e3)
    sample = (f"{items_per_step} (request, head) items of {DESCR[wl.name]} per step: memoised fp64 walk of "
              f"all {wl.T} nodes plus commit")
    line = {
        "impl": "reference", "metric": "verified_tree_nodes_per_s_per_layer", "value": value,
        "unit": "nodes/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": DESCR[wl.name], "sample": sample},
        "cpu_baseline": {"value": value, "unit": "nodes/s", "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "nodes/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line, default=_jsonable), flush=True)


# --------------------------------------------------------------------------
# Multi-GPU bookkeeping (weak scaling, no data-path collective)
# --------------------------------------------------------------------------
def rank_workload(wl, rank: int, layers: int = 0):
    """Every rank verifies its own batch of requests: same shapes, its own seed."""
    import dataclasses
    return dataclasses.replace(wl, seed=wl.seed + 101 * rank, L=layers or wl.L)


def max_over_ranks(values, world: int, device):
    """Element-wise maximum of per-rank timings (the slowest rank sets the job's time)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def job_nodes_per_step(wl, world: int) -> int:
    """Units processed by all ranks in one step (weak scaling: per-rank work is fixed)."""
    return wl.B * wl.T * wl.L * world


# --------------------------------------------------------------------------
# The CUDA path
# --------------------------------------------------------------------------
def stage1_bytes(wl, W: int) -> int:
    """Algorithmic bytes of one tv_tree_conv launch (one layer): x and the context rows in, q/k/v
    out, the filter, and the gate pre-activations in / gates out."""
    es = 2 if wl.qkv_dtype == inputs.BF16 else 4
    C = wl.H * (2 * wl.dk + wl.dv)
    return (wl.B * (2 * wl.T + W - 1) * C * es + C * (W + 1) * 4
            + wl.B * wl.T * wl.H * (2 * es + 2 * 4))


def time_stage1(tv, wl, tree, dev, stream, iters: int, W: int = 4):
    nbytes = stage1_bytes(wl, W)
    n_sets = max(1, min(8, int(np.ceil(4 * L2_BYTES / nbytes))))
    dt = wl.torch_dtype
    calls = []
    for s in range(n_sets):
        ci = inputs.make_conv_inputs(wl, layer=s, device=dev, W=W)
        q = torch.empty(wl.B, wl.H, wl.T, wl.dk, device=dev, dtype=dt)
        k = torch.empty_like(q)
        v = torch.empty(wl.B, wl.H, wl.T, wl.dv, device=dev, dtype=dt)
        al = torch.empty(wl.B, wl.H, wl.T, device=dev, dtype=torch.float32)
        be = torch.empty_like(al)
        calls.append(tv.prepare_tree_conv(tree, ci["x"], ci["ctx"], ci["weight"], ci["bias"], H=wl.H, dk=wl.dk,
                                          dv=wl.dv, gate_a=ci["gate_a"], gate_b=ci["gate_b"], A_log=ci["A_log"],
                                          dt_bias=ci["dt_bias"], normalize_qk=True, q=q, k=k, v=v, alpha=al,
                                          beta=be, stream=stream))
    for i in range(max(3, n_sets)):
        calls[i % n_sets]()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(iters):
        calls[i % n_sets]()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    gbs = nbytes / (ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    return {"kernel": "tree_conv", "taps": W, "normalize_qk": True, "gates": True, "ms_per_layer": ms,
            "nodes_per_s_per_layer": wl.B * wl.T / (ms * 1e-3), "bytes": nbytes, "algorithmic_GBps": gbs,
            "frac_of_measured_copy": gbs / peak, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
            "launches": iters, "l2": f"{n_sets} rotating input set(s)"}


def run_packed(args, wl, local_rank):
    """The same step on a packed forest: every request keeps a random prefix of its tree (between
    a quarter and all of its nodes), the node rows of all requests share flat planes.  One GPU;
    prints a line of its own (not the headline configuration)."""
    import paper_2608_01651_b200 as tv

    tv.lib()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if args.layers:
        wl = dataclasses.replace(wl, L=args.layers)
    parents, _ = inputs.make_trees(wl)
    rng = np.random.Generator(np.random.Philox(key=wl.seed + 77))
    sizes = [wl.T] + [int(rng.integers(max(1, wl.T // 4), wl.T + 1)) for _ in range(wl.B - 1)]
    trees = [np.ascontiguousarray(parents[b if parents.shape[0] > 1 else 0][:n]) for b, n in enumerate(sizes)]
    accepted = np.array([inputs.accepted_walk(t, rng) for t in trees], dtype=np.int32)
    offsets = np.zeros(wl.B + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(sizes)
    total, cap = int(offsets[-1]), wl.B * wl.T
    flat = np.ascontiguousarray(np.concatenate(trees), dtype=np.int32)
    rows = torch.from_numpy(np.concatenate([b * wl.T + np.arange(n) for b, n in enumerate(sizes)])).to(dev)
    delta = wl.rule == inputs.DELTA
    eb = 2 if wl.qkv_dtype == inputs.BF16 else 4

    def pack(t):   # dense [L,B,H,T,...] -> planes [L,H,cap,...] holding the kept rows first
        t = t.transpose(1, 2)
        t = t.reshape(t.shape[0], t.shape[1], wl.B * wl.T, *t.shape[4:])
        out = torch.zeros_like(t)
        out[:, :, :total] = t.index_select(2, rows)
        return out.contiguous()

    set_bytes = wl.L * (wl.B * wl.H * 4 * wl.dk * wl.dv + wl.H * total * (eb * (2 * wl.dk + wl.dv) + 4 * wl.dv))
    n_sets = args.sets or max(2, min(8, int(np.ceil(4 * L2_BYTES / set_bytes))))
    stream = torch.cuda.current_stream()
    forest = tv.forest_build(trees, n_max=wl.T, capacity=cap)
    acc_dev = torch.from_numpy(accepted).to(dev)
    calls = []
    for s in range(n_sets):
        layers = [inputs.make_tensors(wl, layer=s * wl.L + l, device=dev) for l in range(wl.L)]
        st = {k: (None if layers[0][k] is None else torch.stack([x[k] for x in layers])) for k in layers[0]}
        del layers
        P = {k: (None if st[k] is None else pack(st[k].unsqueeze(-1)).squeeze(-1) if k in ("alpha", "beta")
                 else pack(st[k])) for k in ("q", "k", "v", "alpha", "beta")}
        O = torch.empty(wl.L, wl.H, cap, wl.dv, device=dev, dtype=torch.float32)
        U = torch.empty_like(O) if delta else None
        ver = [tv.prepare_tree_verify(forest.upload(), st["S_pre"][l], P["q"][l], P["k"][l], P["v"][l],
                                      P["alpha"][l], None if P["beta"] is None else P["beta"][l], rule=wl.rule,
                                      O=O[l], U=None if U is None else U[l], stream=stream) for l in range(wl.L)]
        com = tv.prepare_commit_path(forest, acc_dev, st["S_pre"], P["k"], P["v"], P["alpha"], P["beta"],
                                     rule=wl.rule, U=U, stream=stream)
        calls.append((ver, com, st, P, O, U))
    refresh = forest.prepare_refresh_forest(flat, offsets, stream)
    probe = max(1, args.probe_every)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    pool = [(ev(), ev(), ev()) for _ in range(args.steps // probe + 1)]
    used = []

    def step(i, record):
        ver, com = calls[i % n_sets][:2]
        refresh()
        if record:
            e0, e1, e2 = pool[len(used)]
            e0.record(stream)
        for c in ver:
            c()
        if record:
            e1.record(stream)
        com()
        if record:
            e2.record(stream)
            used.append((e0, e1, e2))

    for i in range(max(3, args.warmup)):
        step(i, False)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.wait_ready()
    t0, t1 = ev(), ev()
    torch.cuda.synchronize()
    w0 = time.time()
    t0.record(stream)
    for i in range(args.steps):
        step(i, i % probe == 0)
    t1.record(stream)
    torch.cuda.synchronize()
    w1 = time.time()
    clocks = sample_clocks(sampler, w0, w1, lambda: [step(j, False) for j in range(16)])
    ms = t0.elapsed_time(t1) / args.steps
    v_ms = float(np.mean([a.elapsed_time(b) for a, b, _ in used])) / wl.L
    c_ms = float(np.mean([b.elapsed_time(c) for _, b, c in used]))
    # ---- the budget selector that would produce such a forest on the GPU, timed on its own:
    # candidates = the full trees, synthetic draft probabilities, budget = the packed node count
    cand = torch.from_numpy(np.ascontiguousarray(
        np.stack([parents[b if parents.shape[0] > 1 else 0] for b in range(wl.B)]), dtype=np.int32)).to(dev)
    cand[:, 0] = -1
    probs = torch.rand(wl.B, wl.T, device=dev) * 0.9 + 0.1
    sel_forest = tv.forest_build([np.array([-1], dtype=np.int32)] * wl.B, n_max=wl.T, capacity=cap)
    sel = None
    for _ in range(3):
        sel = tv.budget_select(cand, probs, total, stream=stream, out=sel)
        sel_forest.upload_device(sel["parent_packed"], sel["offsets"], max_depth_bound=wl.T - 1, stream=stream)
    torch.cuda.synchronize()
    s0, s1 = ev(), ev()
    n_sel = 50
    s0.record(stream)
    for _ in range(n_sel):
        sel = tv.budget_select(cand, probs, total, stream=stream, out=sel)
        sel_forest.upload_device(sel["parent_packed"], sel["offsets"], max_depth_bound=wl.T - 1, stream=stream)
    s1.record(stream)
    torch.cuda.synchronize()
    sel_ms = s0.elapsed_time(s1) / n_sel

    peak, peak_kind = measured_peak()
    vbytes = (wl.B * wl.H * 4 * wl.dk * wl.dv
              + wl.H * total * (eb * (2 * wl.dk + wl.dv) + 4 + (4 if delta else 0) + 4 * wl.dv * (2 if delta else 1)))
    v_gbs = vbytes / (v_ms * 1e-3) / 1e9
    line = {
        "metric": "verified_tree_nodes_per_s_per_layer", "value": total * wl.L / (ms * 1e-3), "unit": "nodes/s",
        "n_gpus": 1, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": DESCR[wl.name] + f"; PACKED FOREST: {total} nodes in {wl.B} requests of "
                               f"{min(sizes)}..{max(sizes)} nodes, planes of {cap} rows",
                   "layers_per_step": wl.L,
                   "step": "tv_forest_rebuild+upload, tree_verify per layer, commit_path over all layers (in place)",
                   "l2": f"{n_sets} rotating input set(s)"},
        "verify": {"ms_per_layer": v_ms, "nodes_per_s_per_layer": total / (v_ms * 1e-3), "bytes": vbytes,
                   "algorithmic_GBps": v_gbs, "frac_of_measured_copy": v_gbs / peak},
        "commit": {"ms": c_ms},
        "selector": {"ms": sel_ms, "launches": 4, "candidates": wl.B * wl.T, "budget": total,
                     "what": "tv_budget_select (3 kernels) + tv_forest_upload_device (1 kernel), no host sync"},
        "roofline": {"kernel": "tree_verify (packed)", "bound": "hbm", "achieved": v_gbs, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": v_gbs / peak, "traffic": None},
        "cpu_baseline": None, "e2e": None, "gpu_launches": args.steps * (wl.L + 2), "clocks": clocks,
    }
    print(json.dumps(line, default=_jsonable), flush=True)


class StepRig:
    """One workload resident on the device: rotating input sets (so that consecutive steps never
    find their inputs in L2: every set is larger than 4x L2, or there are several), the calls
    marshalled once per set, and the step itself."""

    def __init__(self, tv, wl, dev, stream, impl, n_sets=0):
        self.tv, self.wl, self.stream, self.dev = tv, wl, stream, dev
        self.parents, self.accepted = inputs.make_trees(wl)
        self.acc_len = accepted_lengths(self.parents, self.accepted)
        delta = wl.rule == inputs.DELTA
        eb = 2 if wl.qkv_dtype == inputs.BF16 else 4
        self.set_bytes = wl.L * wl.B * wl.H * (4 * wl.dk * wl.dv + eb * wl.T * (2 * wl.dk + wl.dv)
                                               + 4 * wl.T * wl.dv)
        if not n_sets:
            n_sets = 1 if self.set_bytes > 4 * L2_BYTES else max(2, min(8, int(np.ceil(4 * L2_BYTES / self.set_bytes))))
        self.n_sets = n_sets
        self.sets = []
        for s in range(n_sets):
            layers = [inputs.make_tensors(wl, layer=s * wl.L + l, device=dev) for l in range(wl.L)]
            st = {k: (None if layers[0][k] is None else torch.stack([x[k] for x in layers]))
                  for k in layers[0]}
            del layers
            st["O"] = torch.empty(wl.L, wl.B, wl.H, wl.T, wl.dv, device=dev, dtype=torch.float32)
            st["U"] = torch.empty_like(st["O"]) if delta else None
            self.sets.append(st)
        self.acc_dev = torch.from_numpy(self.accepted).to(dev)
        self.tree = tv.tree_build(self.parents)
        self.calls = []
        for st in self.sets:
            ver = [tv.prepare_tree_verify(self.tree, st["S_pre"][l], st["q"][l], st["k"][l], st["v"][l],
                                          st["alpha"][l], None if st["beta"] is None else st["beta"][l],
                                          rule=wl.rule, O=st["O"][l],
                                          U=None if st["U"] is None else st["U"][l], impl=impl, stream=stream)
                   for l in range(wl.L)]
            com = tv.prepare_commit_path(self.tree, self.acc_dev, st["S_pre"], st["k"], st["v"], st["alpha"],
                                         st["beta"], rule=wl.rule, U=st["U"], stream=stream)
            self.calls.append((ver, com))
        self.refresh = self.tree.prepare_refresh(np.ascontiguousarray(self.parents, dtype=np.int32), stream)
        self.vbytes = verify_bytes_per_layer(wl, with_U=delta)
        self.cbytes = commit_bytes_per_layer(wl, self.acc_len, with_U=delta) * wl.L

    # the whole hot path: tree_build + upload, L verify launches, one commit over all layers
    def step(self, i):
        ver, com = self.calls[i % self.n_sets]
        self.refresh()
        for call in ver:
            call()
        com()

    def step_without_commit(self, i):
        self.refresh()
        for call in self.calls[i % self.n_sets][0]:
            call()

    def verify_only(self, i):          # one launch per call, layers and sets in rotation
        ver = self.calls[i % self.n_sets][0]
        ver[(i // self.n_sets) % len(ver)]()

    def commit_only(self, i):
        self.calls[i % self.n_sets][1]()


def _ev():
    return torch.cuda.Event(enable_timing=True)


def time_loop(stream, n, body, warm=3):
    """Average device time of body(i) over n calls: two events, nothing recorded in between."""
    for i in range(warm):
        body(i)
    torch.cuda.synchronize()
    e0, e1 = _ev(), _ev()
    e0.record(stream)
    for i in range(n):
        body(warm + i)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def copy_yardstick(dev, stream, nbytes, n=48):
    """A plain device copy that moves the same number of bytes as a kernel launch (half read,
    half written), launched back to back over rotating buffers larger than L2: what a launch of
    that SIZE can reach on this GPU, next to the copy peak measured on gigabytes.  torch's
    copy kernel, a yardstick only."""
    half = max(min(int(nbytes), 2**30) // 2 // 16 * 16, 16)   # launches beyond 1 GiB: 1 GiB says it all
    sets = min(max(2, int(4 * 126 * 2**20 // (2 * half)) + 1), 64)
    src = [torch.empty(half, dtype=torch.uint8, device=dev) for _ in range(sets)]
    dst = [torch.empty(half, dtype=torch.uint8, device=dev) for _ in range(sets)]
    for t in src:
        t.zero_()
    ms = time_loop(stream, n, lambda i: dst[i % sets].copy_(src[i % sets]), warm=sets)
    return {"bytes": 2 * half, "ms": ms, "GBps": 2 * half / (ms * 1e-3) / 1e9,
            "what": "torch copy_ of bytes/2, back to back, L2-cold"}


def kernel_split(rig, step_ms, n, peak):
    """Per-kernel times WITHOUT events between launches (an event between two launches costs a
    bubble and undoes the dependent launches): the loop 'metadata + verify' is timed next to the
    full step, the commit's share is the difference, so verify + commit = step by construction.
    The back-to-back loops give each kernel alone (launch gaps included, no dependency on the
    metadata kernel)."""
    wl, stream = rig.wl, rig.stream
    upto_verify = time_loop(stream, n, rig.step_without_commit)
    v_b2b = time_loop(stream, max(n, 16) * min(wl.L, 4), rig.verify_only, warm=max(3, rig.n_sets))
    c_b2b = time_loop(stream, max(n, 16), rig.commit_only, warm=max(3, rig.n_sets))
    v_ms = upto_verify / wl.L
    c_ms = max(step_ms - upto_verify, 0.0)
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
    verify = {"ms_per_layer": v_ms,
              "what": "tree_build + upload + L verify launches, over L; no events between launches",
              "nodes_per_s_per_layer": wl.B * wl.T / (v_ms * 1e-3),
              "bytes_per_layer": rig.vbytes, "algorithmic_GBps": gbs(rig.vbytes, v_ms),
              "frac_of_measured_copy": gbs(rig.vbytes, v_ms) / peak,
              "frac_of_nominal_8TBps": gbs(rig.vbytes, v_ms) / NOMINAL_HBM_GBS,
              "back_to_back_ms": v_b2b,
              "back_to_back_frac_of_measured_copy": gbs(rig.vbytes, v_b2b) / peak,
              "back_to_back_frac_of_nominal_8TBps": gbs(rig.vbytes, v_b2b) / NOMINAL_HBM_GBS}
    commit = {"ms": c_ms, "what": "step minus (tree_build + upload + L verify launches)",
              "bytes": rig.cbytes, "algorithmic_GBps": gbs(rig.cbytes, c_ms),
              "frac_of_measured_copy": gbs(rig.cbytes, c_ms) / peak,
              "frac_of_nominal_8TBps": gbs(rig.cbytes, c_ms) / NOMINAL_HBM_GBS,
              "back_to_back_ms": c_b2b,
              "back_to_back_frac_of_measured_copy": gbs(rig.cbytes, c_b2b) / peak,
              "back_to_back_frac_of_nominal_8TBps": gbs(rig.cbytes, c_b2b) / NOMINAL_HBM_GBS}
    for obj, nbytes in ((verify, rig.vbytes), (commit, rig.cbytes)):
        y = copy_yardstick(rig.dev, stream, nbytes)
        y["frac_of_measured_copy"] = y["GBps"] / peak
        y["kernel_back_to_back_vs_this_copy"] = (nbytes / (obj["back_to_back_ms"] * 1e-3) / 1e9) / y["GBps"]   # rates
        obj["copy_of_same_bytes"] = y
    return verify, commit


def parity_check(rig, layers, n_items, seed=11):
    """One more round of the step exactly as timed (same calls, same launch configuration, commit
    in place), with O, U and S_new of sampled (layer, request, head) items compared with the fp64
    oracle run on the values that sit in device memory.  Outside every timed region."""
    from oracle import tree_oracle as orc
    wl = rig.wl
    st = rig.sets[0]
    rng = np.random.default_rng(seed)
    items = []
    for l in layers:
        picks = {(0, 0), (wl.B - 1, wl.H - 1)}
        while len(picks) < min(n_items, wl.B * wl.H):
            picks.add((int(rng.integers(wl.B)), int(rng.integers(wl.H))))
        items += [(l, b, h) for (b, h) in sorted(picks)]
    S0 = {it: st["S_pre"][it].clone() for it in items}          # the state before this round
    rig.step(0)
    torch.cuda.synchronize()
    rig.tree.device_status()
    f = inputs.to_f64
    eO = eU = eS = 0.0
    for (l, b, h) in items:
        par = rig.parents[b if rig.parents.shape[0] > 1 else 0][None]
        one = lambda t: None if t is None else f(t[l, b, h].cpu())[None, None]
        S_hat, q, k, v, al, be = (f(S0[(l, b, h)].cpu())[None, None], one(st["q"]), one(st["k"]), one(st["v"]),
                                  one(st["alpha"]), one(st["beta"]))
        Or, Ur = orc.verify_batch(S_hat, q, k, v, al, be, par, wl.rule_name)[(0, 0)]
        Sr = orc.commit_batch(S_hat, k, v, al, be, par, [int(rig.accepted[b])], wl.rule_name)[(0, 0)]
        rel = lambda x, r: float((np.linalg.norm(x - r, axis=-1) / np.maximum(np.linalg.norm(r, axis=-1), 1e-300)).max())
        eO = max(eO, rel(f(st["O"][l, b, h].cpu()), Or))
        if st["U"] is not None:
            eU = max(eU, rel(f(st["U"][l, b, h].cpu()), Ur))
        Sn = f(st["S_pre"][l, b, h].cpu())
        eS = max(eS, float(np.linalg.norm(Sn - Sr) / max(np.linalg.norm(Sr), 1e-300)))
    # O and S_new are what the bound is stated on; U is an internal factor whose rows shrink towards
    # zero as the state converges (u = beta (v - S~^T k)), so its relative error is reported only
    return {"max_rel_l2_O": eO, "max_rel_l2_U": eU if st["U"] is not None else None, "max_rel_fro_S": eS,
            "tol": wl.tol, "ok": bool(max(eO, eS) <= wl.tol), "layers": list(layers), "items": len(items),
            "against": "fp64 oracle (per-node path walk) on the device-resident values, after the timed region"}


def throughput_scale(tv, dev, stream, impl, layers, steps, peak, check):
    """The 48-layer workload at a reduced layer count (same kernels, same per-layer work, one input
    set larger than 4x L2): verify and commit against both peaks, driver-visible in the default run."""
    wl = inputs.workload("c5", L=layers)
    rig = StepRig(tv, wl, dev, stream, impl, n_sets=1)
    step_ms = time_loop(stream, steps, rig.step)
    verify, commit = kernel_split(rig, step_ms, steps, peak)
    out = {"workload": DESCR["c5"] + f" -- run with {layers} of its 48 layers "
                       f"({rig.set_bytes / 2**30:.1f} GiB resident, one input set > 4x L2)",
           "steps": steps, "ms_per_step": step_ms, "nodes_per_s_per_layer": wl.B * wl.T * wl.L / (step_ms * 1e-3),
           "verify": verify, "commit": commit}
    if check:
        out["parity"] = parity_check(rig, sorted({0, layers // 2, layers - 1}), 6)
    del rig
    torch.cuda.empty_cache()
    return out


def small_config_latency(tv, dev, stream, impl, name, launches=100):
    """c1 / c2 are launch- and latency-bound (their ideal traffic time is a fraction of a
    microsecond): report them as latency.  Every launch (or whole step) sits between its own pair
    of events; 'warm' = back to back on the same buffers (resident in L2), 'cold' = a buffer
    larger than L2 is overwritten before every launch."""
    wl = inputs.workload(name)
    rig = StepRig(tv, wl, dev, stream, impl, n_sets=1)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)

    def series(body, cold):
        ts = []
        for i in range(launches + 5):
            if cold:
                flush.fill_(i & 0xff)
            e0, e1 = _ev(), _ev()
            e0.record(stream)
            body(i)
            e1.record(stream)
            ts.append((e0, e1))
        torch.cuda.synchronize()
        us = np.array([a.elapsed_time(b) * 1e3 for a, b in ts[5:]])
        return {"median": float(np.median(us)), "min": float(us.min())}

    out = {"workload": DESCR[name], "launches": launches, "unit": "us"}
    rig.step(0)
    torch.cuda.synchronize()
    for key, body in (("verify", rig.verify_only), ("commit", rig.commit_only), ("step", rig.step)):
        out[key] = {"l2_warm": series(body, False), "l2_cold": series(body, True)}
    del rig, flush
    return out


def run_ours(args, wl, rank, world, local_rank):
    import paper_2608_01651_b200 as tv
    import torch.distributed as dist

    tv.lib()  # fail loudly if the library is missing
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    wl = rank_workload(wl, rank, args.layers)
    delta = wl.rule == inputs.DELTA
    impl = {"auto": tv.IMPL_AUTO, "simt": tv.IMPL_SIMT, "tc": tv.IMPL_TC}[args.kernel]
    stream = torch.cuda.current_stream()
    rig = StepRig(tv, wl, dev, stream, impl, n_sets=args.sets)
    parents, accepted, tree, n_sets = rig.parents, rig.accepted, rig.tree, rig.n_sets

    def barrier():
        if world > 1:
            dist.barrier()

    # The clock sampler takes a moment to come up, during which the GPU would sit idle and drop its
    # clocks: start it first, then bring the GPU to its working state with untimed steps (about
    # 30 ms of them, reported as `prewarm_steps`), then the W warm-up steps, then the timed ones.
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.wait_ready()
    barrier()
    prewarm_steps, t_pre = 0, time.time()
    while time.time() - t_pre < 0.03:
        for i in range(8):
            rig.step(i)
        torch.cuda.synchronize()
        prewarm_steps += 8
    for i in range(args.warmup):
        rig.step(i)
    torch.cuda.synchronize()
    barrier()
    t_start, t_end = _ev(), _ev()
    torch.cuda.synchronize()
    w0 = time.time()
    t_start.record(stream)
    for i in range(args.steps):
        rig.step(args.warmup + i)
    t_end.record(stream)
    torch.cuda.synchronize()
    w1 = time.time()
    barrier()
    clocks = sample_clocks(sampler, w0, w1, lambda: [rig.step(j) for j in range(16)]) if sampler else None
    total_ms = t_start.elapsed_time(t_end)
    peak, peak_kind = measured_peak()

    # ---- per-kernel split, event-free loops (their own step counts: short runs stay stable) ----
    n_aux = args.steps if total_ms / args.steps > 1.0 else max(args.steps, 256)
    aux_step_ms = time_loop(stream, n_aux, rig.step) if n_aux != args.steps else total_ms / args.steps
    verify, commit = kernel_split(rig, aux_step_ms, n_aux, peak)
    verify["loops"] = commit["loops"] = n_aux

    # ---- parity of this very configuration against the oracle (outside the timed regions) ------
    parity = None
    if args.check and rank == 0:
        layers = sorted({0, wl.L // 2, wl.L - 1})
        parity = parity_check(rig, layers, args.check_items)

    # ---- Stage 1 (tree convolution + SiLU + normalisation + gates), timed on its own --------
    # Not part of the step above (the metric is defined on verify + commit); one launch per layer
    # would precede each verify launch.  Rotating input sets keep it out of L2 as above.
    stage1 = None
    if world == 1 and not args.no_stage1:
        stage1 = time_stage1(tv, wl, tree, dev, stream, args.stage1_iters)

    # ---- end to end with host buffers through tv_session_round -------------
    e2e = None
    e2e_L = 1 if wl.L > 4 else wl.L
    if not args.no_e2e:
        wl_e = inputs.workload(wl.name, seed=wl.seed, L=e2e_L)
        host = [inputs.make_tensors(wl_e, layer=l) for l in range(e2e_L)]
        hs = {k: (None if host[0][k] is None else torch.stack([x[k] for x in host]).pin_memory())
              for k in host[0]}
        hO = torch.empty(e2e_L, wl.B, wl.H, wl.T, wl.dv, dtype=torch.float32).pin_memory()
        hS = torch.empty_like(hs["S_pre"]).pin_memory()
        sess = tv.Session(e2e_L, wl.B, wl.H, wl.T, wl.dk, wl.dv, rule=wl.rule, qkv_dtype=wl.qkv_dtype,
                          impl=impl)
        n_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            sess.round(parents, accepted, hs["S_pre"], hs["q"], hs["k"], hs["v"], hs["alpha"], hs["beta"],
                       hO, hS, stream)
        torch.cuda.synchronize()
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            sess.round(parents, accepted, hs["S_pre"], hs["q"], hs["k"], hs["v"], hs["alpha"], hs["beta"],
                       hO, hS, stream)
        torch.cuda.synchronize()
        dt_e = (time.perf_counter() - t0) / n_e2e
        h2d = sum(t.numel() * t.element_size() for k, t in hs.items() if t is not None) \
            + parents.size * 24 + accepted.nbytes   # metadata blob: 16 B mask + depth + parent
        d2h = hO.numel() * 4 + hS.numel() * 4
        e2e = [dt_e, h2d, d2h, n_e2e]
        sess.free()
        del hs, hO, hS

    # ---- the throughput-scale workload and the two latency-bound ones, in the default run ------
    scale = small = None
    if world == 1 and wl.name == "c3" and not args.no_extras:
        scale = throughput_scale(tv, dev, stream, impl, args.scale_layers, args.scale_steps, peak, args.check)
        small = {n: small_config_latency(tv, dev, stream, impl, n) for n in ("c1", "c2")}
    if world == 1 and wl.name in ("c1", "c2"):
        small = {wl.name: small_config_latency(tv, dev, stream, impl, wl.name)}

    # ---- max over ranks -----------------------------------------------------
    total_ms, v_ms, c_ms, e2e_dt = max_over_ranks([total_ms, verify["ms_per_layer"], commit["ms"],
                                                   e2e[0] if e2e else 0.0], world, dev)
    if e2e:
        e2e[0] = e2e_dt
    if rank != 0:
        return

    ms_per_step = total_ms / args.steps
    nodes_step = job_nodes_per_step(wl, world)
    value = nodes_step / (ms_per_step * 1e-3)
    v_gbs = rig.vbytes / (v_ms * 1e-3) / 1e9

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        # the oracle on whole requests of this workload, layer after layer, until the budget is spent
        nb = min(wl.B, 32)
        done, dt, threads, layer = 0, 0.0, 1, 0
        while dt < args.cpu_budget and layer < 64:
            small_wl = inputs.workload(wl.name, B=nb, L=1, seed=wl.seed)
            tens = inputs.make_tensors(small_wl, layer=layer)
            _, d1, t1, threads = oracle_sample(small_wl, parents[:nb] if parents.shape[0] > 1 else parents,
                                               accepted[:nb], tens, args.cpu_budget - dt, nb * wl.H)
            done += d1
            dt += t1
            layer += 1
        cpu = {"value": done * wl.T / wl.H / dt, "unit": "nodes/s", "cores": threads, "kind": "oracle",
               "sample": f"{done} (request, head) items of the workload (memoised fp64 walk of all "
                         f"{wl.T} nodes + commit), {dt:.1f} s"}

    tc = wl.qkv_dtype == inputs.BF16 and args.kernel != "simt"
    line = {
        "metric": "verified_tree_nodes_per_s_per_layer",
        "value": value, "unit": "nodes/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "prewarm_steps": prewarm_steps,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": (("bf16 q/k/v, f32 state read by the tensor cores as a bf16 hi+lo pair (16 mantissa bits), "
                   "f32 accumulate, f32 outputs" if wl.rule_name == "gated" else
                   "bf16 q/k/v, f32 state read as tf32 by the tensor cores (mean of the cut compensated), "
                   "f32 accumulate, f32 outputs") if tc
                  else "f32"),
        "data": "synthetic",
        "config": {
            "workload": DESCR[wl.name], "layers_per_step": wl.L, "kernel": args.kernel,
            "step": "tree_build(host)+upload, tree_verify per layer, commit_path over all layers (in place)",
            "l2": f"{n_sets} rotating input set(s) of {rig.set_bytes / 2**20:.0f} MiB each (L2 is 126 MiB)",
            "kernel_split": "event-free loops: 'metadata + verify' timed beside the full step, commit = the difference",
            "trees": inputs.tree_stats(parents, accepted),
        },
        "verify": verify,
        "commit": commit,
        "roofline": {"kernel": "tree_verify", "bound": "hbm", "achieved": v_gbs, "peak": peak,
                     "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": v_gbs / peak,
                     "traffic": args.traffic if args.traffic is not None else ncu_traffic(wl.name),
                     "timing": "in the step (metadata kernel and launch gaps included); "
                               "verify.back_to_back_* is the kernel alone"},
        "parity": parity,
        "throughput_scale": scale,
        "small_configs": small,
        "cpu_baseline": cpu,
        "stage1": stage1,
        "e2e": None if e2e is None else {
            "value": wl.B * wl.T * e2e_L * world / e2e[0], "unit": "nodes/s",
            "h2d_bytes_per_step": int(e2e[1]), "d2h_bytes_per_step": int(e2e[2]),
            "steps": e2e[3], "layers": e2e_L,
            "call": "tv_session_round (pinned host buffers in, O and S_new out)"},
        "gpu_launches": args.steps * (wl.L + 2),   # per step: metadata kernel, L verify, one commit
        "clocks": clocks,
    }
    print(json.dumps(line, default=_jsonable), flush=True)


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` started by hand: run the N replica ranks (one process per GPU,
    the same command line) under torch.distributed.run and hand back its exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default: 5000, or 20 for the 48-layer workload: a few hundred ms, "
                         "long enough for nvidia-smi to sample the clocks inside the timed region)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3", choices=sorted(DESCR))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--layers", type=int, default=0, help="override layers per step")
    ap.add_argument("--sets", type=int, default=0, help="override number of rotating input sets")
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--ref-items", type=int, default=8)
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu dram bytes per verify launch to echo into roofline.traffic")
    ap.add_argument("--probe-every", type=int, default=0,
                    help="(packed-forest line only) record per-kernel CUDA events on every n-th timed step")
    ap.add_argument("--check", action=argparse.BooleanOptionalAction, default=True,
                    help="after the timed region, compare O, U and S_new of sampled (layer, request, head) "
                         "items of this very run with the fp64 oracle and add a 'parity' object "
                         "(on by default, a few seconds outside every timed region; --no-check drops it)")
    ap.add_argument("--check-items", type=int, default=8, help="sampled items per checked layer")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the throughput-scale and small-config objects of the default run")
    ap.add_argument("--scale-layers", type=int, default=6)
    ap.add_argument("--scale-steps", type=int, default=10)
    ap.add_argument("--packed", action="store_true",
                    help="run the step on a packed forest of requests with different node counts (1 GPU)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-stage1", action="store_true")
    ap.add_argument("--no-b2b", action="store_true", help="(kept for old command lines; no effect)")
    ap.add_argument("--stage1-iters", type=int, default=48)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 200 if args.impl == "reference" else (20 if args.workload == "c5" else 5000)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.probe_every <= 0:
        args.probe_every = max(8, args.steps // 64)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not args.packed:
        sys.exit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = inputs.workload(args.workload)

    if args.impl == "reference":
        run_reference(args, wl, rank, world)
        return
    if args.packed:
        if rank == 0:
            run_packed(args, wl, local_rank)
        return
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl")
    try:
        run_ours(args, wl, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
