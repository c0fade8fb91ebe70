#!/usr/bin/env python
"""Benchmark of the VMoBA attention layer hot path on B200.

A step is one pass of the whole layer over one batch of synthetic video-DiT-shaped input:
partition(q, k, v) -> centroids + scores -> global threshold selection -> sparse attention
forward -> inverse partition(o), and for training workloads the backward:
partition(dO) -> sparse attention backward writing dq, dk, dv in raster order (bf16, head_dim 128;
otherwise the backward followed by the inverse partitions of the gradients).  Workloads with
several partitions (c3, c5) run the layer once per partition (1D, 2D, 3D) per step.

    python bench.py --gpus 1 --steps 20 --warmup 3                # default workload: c5
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference                               # the CPU oracle, timed

Prints one JSON line (rank 0).  `value` = selected-pair attention FLOPs of all ranks per second
of whole-step time, inputs resident in HBM.  `e2e` = the same with pinned host inputs copied to
the device and results copied back inside the timed region.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np


def workloads(name):
    """The benchmark configurations: list of (Workload, with_backward) layers run per step."""
    from paper_2506_23858_b200 import inputs as gen
    if name == "c1":
        return [gen.C1], True
    if name == "c2":
        return [gen.C2], False
    if name == "c3":
        return [gen.C2.with_(name="c3_" + k, block=b) for k, b in gen.C3_BLOCKS.items()], False
    if name == "c4":
        return [gen.C4], True
    if name == "c5":
        return [gen.C5.with_(name="c5_" + k, block=b) for k, b in gen.C5_BLOCKS.items()], True
    if name == "t55k":   # the paper's 55K-token fine-tuning grid with its own block counts (Table 4), three layers
        return [gen.T55.with_(name="t55k_" + k, block=b) for k, b in gen.T55_BLOCKS.items()], True
    if name == "t56k":   # the paper's second training grid (Table 4: 141 x 480 x 832 video, latent 36 x 30 x 52)
        return [gen.T56.with_(name="t56k_" + k, block=b) for k, b in gen.T56_BLOCKS.items()], True
    raise SystemExit(f"unknown workload {name}")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], tensor_burst=p["bf16_tflops"], tensor_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.index),
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


_oracle_input_cache = {}


def _oracle_inputs(w, with_bwd):
    """Inputs of (batch 0, head 0) of workload w, generated once (generation is not timed)."""
    from paper_2506_23858_b200 import inputs as gen
    key = (w, with_bwd)
    if key not in _oracle_input_cache:
        _oracle_input_cache[key] = gen.make_inputs(w, with_do=with_bwd, heads=[0])
    return _oracle_input_cache[key]


# ------------------------------------------------------------------------------------------
def oracle_sample(w, with_bwd, n_rows, seed=0):
    """Times the CPU oracle on one (batch, head) unit of workload w: partition, centroids, scores
    and selection in full, attention forward (+ backward) on n_rows sampled query rows.
    Returns (seconds extrapolated to the whole unit, selected-pair flops of the whole unit, detail)."""
    from oracle import vmoba_oracle as orc
    from paper_2506_23858_b200 import inputs as gen
    data = _oracle_inputs(w, with_bwd)
    scale = w.head_dim ** -0.5
    t0 = time.perf_counter()
    perm, inv = orc.partition_perm(w.T, w.H, w.W, *w.block)
    q, k, v = (data[n][0, :, 0][perm] for n in "qkv")
    cent = orc.centroids(k, w.n_blocks)
    sc = orc.block_scores(q, cent)
    mask, k_sel, cutoff = orc.select(sc, w.tau, scale)
    t_front = time.perf_counter() - t0
    rng = np.random.default_rng(seed)
    rows = rng.choice(w.S, size=min(n_rows, w.S), replace=False)
    t0 = time.perf_counter()
    orc.sparse_attn_fwd(q, k, v, mask, scale, rows=rows)
    if with_bwd:
        do = data["do"][0, :, 0][perm]
        orc.sparse_attn_bwd(q, k, v, mask, scale, do, rows=rows)
    t_rows = time.perf_counter() - t0
    pairs_rows = int(mask[rows].sum())
    # attention time scales with the pairs processed
    t_attn = t_rows * (k_sel / max(pairs_rows, 1))
    mult = 14.0 if with_bwd else 4.0
    flops = mult * w.head_dim * w.block_tokens * k_sel
    return t_front + t_attn, flops, dict(front_s=t_front, rows_s=t_rows, rows=int(rows.size), pairs_rows=pairs_rows,
                                         pairs_unit=int(k_sel))


def workload_config(args, layers, with_bwd):
    """The `config` object of the JSON line (both arms print the same one; the product arm adds its L2 note)."""
    w0 = layers[0]
    cfg = {"workload": args.workload, "passes": "fwd+bwd" if with_bwd else "fwd", "B": w0.B, "heads": w0.heads,
           "head_dim": w0.head_dim, "grid": [w0.T, w0.H, w0.W], "blocks": [list(w.block) for w in layers],
           "tau": w0.tau, "rule": args.rule}
    if "topk" in args.rule:
        cfg["topk"] = [int(x) for x in args.topk.split(",")] if args.topk else [2]
    cfg["inputs"] = w0.recipe
    return cfg


def run_reference(args):
    """--impl reference: the oracle as it stands, on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    layers, with_bwd = workloads(args.workload)
    import torch
    cores = torch.get_num_threads()
    times, flops_tot = [], 0.0
    detail = None
    # One untimed step first (also when W = 0): it tells how long a step takes.  If W + K such steps would
    # not end within a few minutes, the later steps take a smaller sample: first fewer query rows for the
    # attention, then fewer of the workload's layers (the value is work / time of whatever was sampled), and
    # only if that is still too slow, fewer steps.
    warmup, steps = 1, args.steps
    n_used = len(layers)
    rows = args.cpu_rows
    it = 0
    while it < warmup + steps:
        wall = time.perf_counter()
        t, f = 0.0, 0.0
        for w in layers[:n_used]:
            tt, ff, detail = oracle_sample(w, with_bwd, rows, seed=it)
            t += tt; f += ff
        wall = time.perf_counter() - wall
        if it >= warmup:
            times.append(t); flops_tot = f
        else:
            budget = 240.0 / (warmup + steps)
            if wall > budget:
                rows = max(32, int(rows * budget / wall) // 32 * 32)
                est = wall * (0.25 + 0.75 * rows / args.cpu_rows)      # part of a step does not depend on the rows
                if est > budget:
                    n_used = max(1, int(len(layers) * budget / est))
                    est = est * n_used / len(layers)
                    if est > 2.0 * budget:
                        steps = max(1, int(240.0 / est) - warmup)
        it += 1
    sec = statistics.mean(times)
    units = layers[0].B * layers[0].heads
    value = flops_tot / sec / 1e12
    sample = (f"1 of {units} (batch, head) units of {n_used} of the {len(layers)} layers; partition, centroids, scores, "
              f"selection in full; attention on {rows} sampled query rows, time scaled to the unit's selected pairs")
    line = {
        "impl": "reference", "metric": "vmoba_layer_selected_pair_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "ms_per_step": sec * 1e3 * units * len(layers) / n_used,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args, layers, with_bwd),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def aggregate_over_ranks(ms_per_step, e2e_ms, flops, device):
    """Whole-job numbers from per-rank ones: times are the MAX over ranks, work is the SUM."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_per_step, e2e_ms, flops], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        tmax = t.clone(); dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        tsum = t.clone(); dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
        return float(tmax[0]), float(tmax[1]), float(tsum[2])
    return float(t[0]), float(t[1]), float(t[2])


def rank_workloads(layers, rank):
    """Weak scaling: every rank runs the full workload shape on its own seeded batch; (batch, head)
    units are independent, so the data path needs no collective."""
    return [w.with_(seed=w.seed + 1000 * rank) for w in layers]


# ------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="vmoba", choices=["vmoba", "reference"])
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5", "t55k", "t56k"])
    ap.add_argument("--inputs", default="", choices=["", "smooth", "white", "sine"],
                    help="override the workload's input recipe; 'white' = no locality component (selection pattern "
                         "essentially random: the worst case for gathered work lists)")
    ap.add_argument("--cpu-rows", type=int, default=256, help="query rows per unit the CPU oracle baseline evaluates")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dense", action="store_true",
                    help="also time the dense vmoba_full_attn path on the same inputs (always done for c5)")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense comparison of c5")
    ap.add_argument("--e2e-steps", type=int, default=0,
                    help="steps of the end-to-end loop (default: as many as --steps); the first step's input copy and the last\n"
                         "step's read-back are not overlapped with anything, so a short loop reads slower than a long one")
    ap.add_argument("--rule", default="threshold_global",
                    choices=["threshold_global", "topk_global", "threshold_local", "topk_local"],
                    help="block-choice rule (Table 3b); the paper's training-free runs use topk_local")
    ap.add_argument("--topk", default="", help="k of the top-k rules: one value, or one per layer (e.g. 2,6,18)")
    ap.add_argument("--no-fold", action="store_true",
                    help="partition dO and inverse-partition dq, dk, dv in passes of their own (instead of the backward reading / writing raster order)")
    ap.add_argument("--fold-do", action="store_true",
                    help="also let the backward read dO in raster order (pays with few heads: c4 yes, c5 no)")
    ap.add_argument("--fold-o", action="store_true",
                    help="let the forward write o in raster order (saves the inverse partition pass of o; measured slower)")
    ap.add_argument("--heads", type=int, default=0, help="override the number of heads (small profiling runs)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2506_23858_b200 import binding as vb
    from paper_2506_23858_b200 import inputs as gen
    from paper_2506_23858_b200.layer import VmobaLayer

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    vb.lib()
    pk = peaks()

    layers, with_bwd = workloads(args.workload)
    if args.heads > 0:
        layers = [w.with_(heads=args.heads) for w in layers]
    if args.inputs:
        layers = [w.with_(recipe=args.inputs) for w in layers]
    layers = rank_workloads(layers, rank)
    w0 = layers[0]
    data = gen.make_inputs(w0, with_do=with_bwd)
    names = ["q", "k", "v"] + (["do"] if with_bwd else [])

    def host_tensor(n):
        if w0.dtype == "bf16":
            return torch.from_numpy(data[n + "_bits"].view(np.int16)).view(torch.bfloat16).pin_memory()
        return torch.from_numpy(data[n]).pin_memory()

    host = {n: host_tensor(n) for n in names}
    dev = {n: host[n].cuda() for n in names}
    outs = {n: torch.empty_like(dev["q"]) for n in (["o"] + (["dq", "dk", "dv"] if with_bwd else []))}
    host_out = {n: torch.empty_like(host["q"]).pin_memory() for n in outs}

    rule = {"threshold_global": vb.SELECT_THRESHOLD_GLOBAL, "topk_global": vb.SELECT_TOPK_GLOBAL,
            "threshold_local": vb.SELECT_THRESHOLD_LOCAL, "topk_local": vb.SELECT_TOPK_LOCAL}[args.rule]
    topks = [int(x) for x in args.topk.split(",")] if args.topk else [2]

    def do_select(layer, w, i):
        if rule == vb.SELECT_THRESHOLD_GLOBAL:
            layer.select(w.tau)
        else:
            layer.select_rule(rule, tau=w.tau, topk=topks[min(i, len(topks) - 1)])

    # capacity of the work lists: measured selection size of this workload plus headroom
    L = []
    for w in layers:
        shape = vb.shape_of(w)
        probe = VmobaLayer(shape, capacity=1)          # scores + selection only, to size the lists
        probe.partition(dev["q"], probe.q_bm); probe.partition(dev["k"], probe.k_bm)
        probe.block_scores(); do_select(probe, w, len(L))
        torch.cuda.synchronize()
        n_sel = probe.n_selected()
        del probe
        torch.cuda.empty_cache()
        L.append(VmobaLayer(shape, capacity=int(n_sel * 1.05) + 4096, with_backward=with_bwd))

    stage_names = ["partition", "scores", "select", "attn_fwd"] + (["attn_bwd"] if with_bwd else [])
    stage_ms = {s: 0.0 for s in stage_names}

    fold = with_bwd and not args.no_fold and L[0].can_fold_inverse(outs["dq"], outs["dk"], outs["dv"])
    fold_o = args.fold_o and L[0].can_fold_o()            # the forward writes o in raster order itself

    def step(record, dev=dev, outs=outs):
        evs = []

        def mark(tag):
            if record:
                e = torch.cuda.Event(enable_timing=True); e.record(); evs.append((tag, e))

        for layer in L:
            mark("start")
            layer.partition(dev["q"], layer.q_bm, perm=layer.perm); layer.partition(dev["k"], layer.k_bm)
            layer.partition(dev["v"], layer.v_bm)
            mark("partition")
            layer.block_scores(); mark("scores")
            do_select(layer, layer_w[id(layer)], layer_pos[id(layer)]); mark("select")
            if fold_o:
                layer.attn_fwd_raster(outs["o"]); mark("attn_fwd")
            else:
                layer.attn_fwd(); mark("attn_fwd")
                layer.partition(outs["o"], layer.o_bm, inverse=True); mark("partition")
            if with_bwd:
                if fold and args.fold_do:
                    # the backward kernels read dO and write dq, dk, dv in raster order themselves (Eq. 1 folded in)
                    layer.attn_bwd_raster(dev["do"], outs["dq"], outs["dk"], outs["dv"]); mark("attn_bwd")
                elif fold:
                    layer.partition(dev["do"], layer.do_bm); mark("partition")
                    layer.attn_bwd_raster(None, outs["dq"], outs["dk"], outs["dv"]); mark("attn_bwd")
                else:
                    layer.partition(dev["do"], layer.do_bm); mark("partition")
                    if layer.o_raster is not None:
                        layer.partition(layer.o_raster, layer.o_bm)
                    layer.attn_bwd(); mark("attn_bwd")
                    layer.partition(outs["dq"], layer.dq_bm, inverse=True)
                    layer.partition(outs["dk"], layer.dk_bm, inverse=True)
                    layer.partition(outs["dv"], layer.dv_bm, inverse=True)
                    mark("partition")
        return evs

    layer_tau = {id(layer): w.tau for layer, w in zip(L, layers)}
    layer_w = {id(layer): w for layer, w in zip(L, layers)}
    layer_pos = {id(layer): i for i, layer in enumerate(L)}

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    barrier()
    for layer in L:
        layer.check_status()
    n_sel = [layer.n_selected() for layer in L]

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = vb.kernel_launches()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    all_evs = [step(True) for _ in range(args.steps)]
    t_end.record()
    barrier()
    launches = vb.kernel_launches() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t_start.elapsed_time(t_end)
    for evs in all_evs:
        for (tag0, e0), (tag1, e1) in zip(evs[:-1], evs[1:]):
            if tag1 != "start":
                stage_ms[tag1] += e0.elapsed_time(e1)
    stage_ms = {k: v / args.steps for k, v in stage_ms.items()}
    ms_per_step = total_ms / args.steps
    for layer in L:
        layer.check_status()

    # ---- end to end: pinned host -> device, layer, device -> host, every step.  The entry points are
    # asynchronous on the caller's stream, so a caller overlaps the copies with the layer: inputs of step
    # i + 1 travel on a second stream while step i computes, results of step i on a third while step
    # i + 1 computes (two sets of device buffers).  Every step's copies are inside the timed region.
    dev_b = {n: torch.empty_like(dev[n]) for n in names}
    outs_b = {n: torch.empty_like(outs[n]) for n in outs}
    sets = [(dev, outs), (dev_b, outs_b)]
    main_s = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_run(n_steps):
        ev_in = [torch.cuda.Event(), torch.cuda.Event()]
        ev_done = [torch.cuda.Event(), torch.cuda.Event()]
        ev_out = [torch.cuda.Event(), torch.cuda.Event()]
        s_in.wait_stream(main_s); s_out.wait_stream(main_s)
        with torch.cuda.stream(s_in):
            for n in names:
                sets[0][0][n].copy_(host[n], non_blocking=True)
            ev_in[0].record(s_in)
        for i in range(n_steps):
            d, o = sets[i % 2]
            main_s.wait_event(ev_in[i % 2])            # this step's inputs have arrived
            if i >= 2:
                main_s.wait_event(ev_out[i % 2])       # this output set has been read back (step i - 2)
            step(False, d, o)
            ev_done[i % 2].record(main_s)
            if i + 1 < n_steps:
                with torch.cuda.stream(s_in):
                    if i >= 1:
                        s_in.wait_event(ev_done[(i + 1) % 2])   # step i - 1 no longer reads that input set
                    for n in names:
                        sets[(i + 1) % 2][0][n].copy_(host[n], non_blocking=True)
                    ev_in[(i + 1) % 2].record(s_in)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i % 2])
                for n in o:
                    host_out[n].copy_(o[n], non_blocking=True)
                ev_out[i % 2].record(s_out)
        main_s.wait_stream(s_out); main_s.wait_stream(s_in)

    if args.e2e_steps <= 0:
        args.e2e_steps = args.steps
    e2e_run(2); barrier()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    e2e_run(args.e2e_steps)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.e2e_steps

    # ---- the dense path on the same inputs (config 5's speed-up denominator; Section 4.1's "Full Attention"):
    # one dense layer, forward (+ backward), one warm-up call and two timed ones
    dense_ms = None
    if (args.dense or args.workload == "c5") and not args.no_dense:
        del dev_b, outs_b, sets
        torch.cuda.empty_cache()
        shape = vb.shape_of(w0)
        qd, kd, vd = (dev[n].permute(0, 2, 1, 3).contiguous() for n in "qkv")
        od = torch.empty_like(qd)
        lse = torch.empty(w0.B * w0.heads * w0.S, dtype=torch.float32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        extra = {}
        if with_bwd:
            extra = dict(do=dev["do"].permute(0, 2, 1, 3).contiguous(), dq=torch.empty_like(qd),
                         dk=torch.empty_like(qd), dv=torch.empty_like(qd),
                         ws=torch.empty(vb.workspace_bytes(shape, vb.STAGE_FULL_BWD), dtype=torch.uint8, device="cuda"))
        vb.vmoba_full_attn(shape, qd, kd, vd, od, lse, dev_status=st, **extra)
        torch.cuda.synchronize()
        d0 = torch.cuda.Event(enable_timing=True); d1 = torch.cuda.Event(enable_timing=True)
        d0.record()
        for _ in range(2):
            vb.vmoba_full_attn(shape, qd, kd, vd, od, lse, dev_status=st, **extra)
        d1.record(); torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / 2
        if int(st.item()) != 0:
            raise vb.VmobaError(int(st.item()), "dense path")
        del qd, kd, vd, od, extra

    # ---- aggregate over ranks (max time, summed work)
    mult = 14.0 if with_bwd else 4.0
    flops = sum(mult * w.head_dim * w.block_tokens * n for w, n in zip(layers, n_sel))
    ms_per_step, e2e_ms, flops_all = aggregate_over_ranks(ms_per_step, e2e_ms, flops, "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    es = 2 if w0.dtype == "bf16" else 4
    tensor_bytes = w0.B * w0.S * w0.heads * w0.head_dim * es
    # partition passes of a step: q, k, v in; o out unless the forward writes raster order; dO in unless the backward
    # reads raster order; dq, dk, dv out unless the backward writes raster order
    n_part = len(layers) * (3 + (0 if fold_o else 1)
                            + ((0 if (fold and args.fold_do) else 1) + (0 if fold else 3) if with_bwd else 0))
    alg = {
        "partition": ("hbm", 2.0 * tensor_bytes * n_part),
        "scores": ("hbm", sum(2.0 * tensor_bytes + 4.0 * w.B * w.heads * (w.S * w.n_blocks + w.n_blocks * w.head_dim)
                              for w in layers)),
        "select": ("hbm", sum(2.0 * 4.0 * w.B * w.heads * w.S * w.n_blocks
                              + 4.0 * w.B * w.heads * w.S * ((w.n_blocks + 31) // 32) + 8.0 * n
                              for w, n in zip(layers, n_sel))),
        "attn_fwd": ("tensor", sum(4.0 * w.head_dim * w.block_tokens * n for w, n in zip(layers, n_sel))),
        "attn_bwd": ("tensor", sum(10.0 * w.head_dim * w.block_tokens * n for w, n in zip(layers, n_sel))),
    }
    stages = {}
    for s in stage_names:
        bound, work = alg[s]
        ms = stage_ms[s]
        if bound == "hbm":
            ach = work / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
            stages[s] = {"ms": ms, "bound": "hbm", "achieved": ach, "unit": "GB/s", "frac": ach / pk["hbm"]}
        else:
            ach = work / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
            stages[s] = {"ms": ms, "bound": "tensor", "achieved": ach, "unit": "TFLOP/s",
                         "frac": ach / pk["tensor_sustained"]}
    dom = max(stage_names, key=lambda s: stage_ms[s])
    # DRAM bytes per launch of the stage's main kernel, from the committed ncu capture of this workload
    traffic = None
    tpath = os.path.join(ROOT, "profiles", f"traffic_bench_{args.workload}.txt")
    if os.path.exists(tpath) and args.heads <= 0:
        for line in open(tpath):
            f = line.split()
            if len(f) == 2 and f[0] == dom:
                traffic = int(f[1])
    roofline = {"kernel": dom, "bound": stages[dom]["bound"], "achieved": stages[dom]["achieved"],
                "peak": pk["hbm"] if stages[dom]["bound"] == "hbm" else pk["tensor_sustained"],
                "unit": stages[dom]["unit"], "frac": stages[dom]["frac"], "traffic": traffic,
                "peak_source": pk["source"] + (" sustained bf16" if stages[dom]["bound"] == "tensor" else " copy"),
                "note": "duration is the stage's entry-point call (its main kernel plus small helper kernels), "
                        "CUDA events on the launching stream, averaged over the timed steps"}

    cpu = None
    if not args.no_cpu_baseline:
        t_cpu, f_cpu = 0.0, 0.0
        for w in layers:
            tt, ff, _ = oracle_sample(w, with_bwd, args.cpu_rows)
            t_cpu += tt; f_cpu += ff
        cpu = {"value": f_cpu / t_cpu / 1e12, "unit": "TFLOP/s", "cores": torch.get_num_threads(), "kind": "oracle",
               "sample": f"1 of {w0.B * w0.heads} (batch, head) units per layer: partition, centroids, scores, selection "
                         f"in full; attention on {args.cpu_rows} sampled query rows scaled to the unit's selected pairs"}

    P_tot = sum(w.B * w.heads * w.S * w.n_blocks for w in layers)
    # every timed step streams its inputs, block-major copies, scores and outputs: no buffer is flushed
    # between steps, the working set itself is what evicts the L2 (126 MB)
    touched = (len(names) + len(outs)) * 2 * tensor_bytes
    if tensor_bytes > 126e6:
        l2_note = "no flush: each input tensor (%.0f MB) exceeds L2" % (tensor_bytes / 1e6)
    elif touched > 126e6:
        l2_note = "no flush: tensors of %.0f MB each, %.0f MB streamed per step exceed L2" % (tensor_bytes / 1e6, touched / 1e6)
    else:
        l2_note = "no flush: working set (%.1f MB) fits L2, numbers are L2-warm (parity-size workload)" % (touched / 1e6)
    line = {
        "metric": "vmoba_layer_selected_pair_tflops", "value": flops_all / (ms_per_step * 1e-3) / 1e12,
        "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w0.dtype, "data": "synthetic",
        "config": {**workload_config(args, layers, with_bwd), "l2": l2_note},
        "clocks": clocks,
        "e2e": {"value": flops_all / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": len(names) * tensor_bytes, "d2h_bytes_per_step": len(outs) * tensor_bytes},
        "gpu_launches": launches,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "stages": stages,
        "density": sum(n_sel) / P_tot,
        "selected_pairs": n_sel,
        "attn_tflops": (alg["attn_fwd"][1] + (alg["attn_bwd"][1] if with_bwd else 0.0))
                       / ((stage_ms["attn_fwd"] + stage_ms.get("attn_bwd", 0.0)) * 1e-3) / 1e12,
        "dense_ms": dense_ms,
        # which build of the library was timed (binding.lib() rebuilds it when a source is newer)
        "library": {"path": os.path.relpath(vb.lib_path(), ROOT), "mtime": int(os.path.getmtime(vb.lib_path())),
                    "bytes": os.path.getsize(vb.lib_path())},
    }
    if dense_ms is not None:
        # one dense layer against one sparse layer (the step's time over its layers, every stage included)
        dense_flops = (14.0 if with_bwd else 4.0) * w0.B * w0.heads * float(w0.S) ** 2 * w0.head_dim
        line["dense"] = {"ms_per_layer": dense_ms, "tflops": dense_flops / (dense_ms * 1e-3) / 1e12,
                         "frac": dense_flops / (dense_ms * 1e-3) / 1e12 / pk["tensor_sustained"],
                         "sparse_ms_per_layer": ms_per_step / len(layers),
                         "speedup_sparse_vs_dense": dense_ms / (ms_per_step / len(layers))}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
