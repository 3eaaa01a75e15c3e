#!/usr/bin/env python
"""Benchmark of the GDN tree verify + commit hot path.

One *step* = one decode iteration of the path: the commit of the previous step's accepted paths and the verification
of the tree (all nodes of all trees, all heads, all layer slots), through the C ABI.  The default workload is the stack
configuration the headline target is quoted on: all GDN heads of a 48-layer stack (48 layer slots x 32 value heads,
d_k = d_v = 128), one 64-node draft tree, batch 1, bf16 inputs, fp32 state, one call per step.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference|recurrent] [--workload NAME] [--mode M]

The K-step timed region (barrier + synchronize on both sides, CUDA events on the launching stream) is repeated until
at least --min-time seconds of device time have been measured; the line reports the median region (and the fastest),
and the clock samples cover the whole repeated span.  With N > 1 (under torchrun) every rank runs its own replica of
the workload (the path has no exchange step: each (sequence, layer, head) is independent), timing is the max over
ranks and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_06763_b200 import synth  # noqa: E402

METRIC = "verified tree-nodes/sec per GDN layer"
UNIT = "nodes/s"
CONFIG_WORKLOADS = {"stack48_T64": 5, "layer_T64": 1, "stack48_T256": 2, "ragged32": 3, "chains64x16": 4}
SWEEP_T = (32, 64, 128, 256, 512)
WORKLOADS = sorted(CONFIG_WORKLOADS) + [f"sweep_T{t}" for t in SWEEP_T] + ["stack48_T64_deep", "stack48_T64_bestfirst"]
DTYPE = "bf16 inputs/outputs, fp32 state; contractions as bf16 hi+lo splits on tcgen05 with fp32 accumulation"


def make_workload(args) -> synth.Workload:
    if args.workload in CONFIG_WORKLOADS:
        return synth.config(CONFIG_WORKLOADS[args.workload], 0, n_layers=args.layers)
    if args.workload == "stack48_T64_deep":
        return synth.deep_stack(args.path_len, n_layers=args.layers)
    if args.workload == "stack48_T64_bestfirst":
        return synth.bestfirst_stack(n_layers=args.layers)
    return synth.layer_sweep(int(args.workload.split("_T")[1]))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def captured_traffic(workload: str, mode: str, n_slots: int):
    """DRAM bytes per launch of the dominant kernel, from the ncu captures summarised in profiles/traffic.json
    (a capture of a slice of the workload, scaled by layer slots); None if no capture covers this run."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    for e in json.load(open(path)).get("captures", []):
        if e.get("workload") == workload and e.get("mode") == mode:
            per_slot = (e["dram_bytes_read"] + e["dram_bytes_write"]) / e["slots"]
            return {"bytes_per_launch": per_slot * n_slots, "source": "profiles/traffic.json: " + e.get("file", ""),
                    "captured_slots": e["slots"], "dram_bytes_read": e["dram_bytes_read"],
                    "dram_bytes_write": e["dram_bytes_write"]}
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.file = index, None, None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.file,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t0=None, t1=None):
        """Median SM clock over the samples taken inside the wall-clock window [t0, t1] (the timed span); all
        samples if none fell inside."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()   # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, power, reasons, inside = [], [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                stamp = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            under_load = t0 is not None and t1 is not None and t0 <= stamp <= t1
            inside.append(under_load)
            if under_load or t0 is None:
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if any(inside):
            sm = [v for v, keep in zip(sm, inside) if keep]
            power = [v for v, keep in zip(power, inside) if keep]
            out["window"] = "timed span"
        elif sm:
            out["window"] = "whole run (no sample fell inside the timed span)"
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w_median=statistics.median(power))
        return out


def algorithmic_bytes(w: synth.Workload):
    """(verify bytes, commit bytes, step bytes).  Step bytes follow the headline definition: S0 read once + S_new
    written once + q,k,v,g,beta read + o written.  Per launch: verify reads S0 and the node tensors and writes o;
    commit reads and writes the state (its re-read of the accepted nodes' rows is not counted)."""
    isz = 4 if w.in_dtype == synth.F32 else 2
    osz = 4 if w.out_dtype == synth.F32 else 2
    N = w.total_nodes
    state = w.n_seq * w.h_v * w.d_v * w.d_k * 4
    nodes_in = 2 * N * w.h_qk * w.d_k * isz + N * w.h_v * w.d_v * isz + 2 * N * w.h_v * isz
    o = N * w.h_v * w.d_v * osz
    return state + nodes_in + o, 2 * state, 2 * state + nodes_in + o


def oracle_sample(w: synth.Workload, target_slots: int):
    """Time the fp64 oracle on the first `target_slots` sequences (verify + commit)."""
    from oracle import gdn_oracle as orc
    n = max(1, min(target_slots, w.n_seq))
    lo, hi = 0, int(w.node_offsets[n])
    args = dict(S0=w.S0[:n].astype(np.float64), q=synth.widen(w.q[lo:hi], w.in_dtype),
                k=synth.widen(w.k[lo:hi], w.in_dtype), v=synth.widen(w.v[lo:hi], w.in_dtype),
                g=synth.widen(w.g[lo:hi], w.in_dtype), beta=synth.widen(w.beta[lo:hi], w.in_dtype))
    parent, offs = w.parent[lo:hi], w.node_offsets[: n + 1]
    poffs = w.path_offsets[: n + 1]
    path = w.path[: int(poffs[-1])]

    def run():
        t0 = time.perf_counter()
        orc.verify(args["S0"], args["q"], args["k"], args["v"], args["g"], args["beta"], parent, offs, w.scale)
        orc.commit(args["S0"], args["k"], args["v"], args["g"], args["beta"], parent, offs, path, poffs)
        return time.perf_counter() - t0

    return run, hi - lo, n, orc.threads()


def run_reference(args, w: synth.Workload):
    """--impl reference: the oracle as it stands, timed on the host cores on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # A step is a bounded sample of the workload: as many layer slots / sequences as keep the whole
    # --steps/--warmup run near two minutes of host time (at least one), found from one probe slot.
    probe, _, _, _ = oracle_sample(w, 1)
    probe()
    t_slot = min(probe(), probe())
    budget_s = 120.0
    fit = int(budget_s / max((args.steps + args.warmup) * t_slot, 1e-9))
    run, nodes, n_slots, cores = oracle_sample(w, max(1, min(fit, args.oracle_slots)))
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = (time.perf_counter() - t0) / args.steps
    value = nodes / dt
    sample = (f"first {n_slots} of {w.n_seq} layer slots/sequences ({nodes} nodes) per step, verify + commit; "
              f"sample sized for about {budget_s:.0f} s over {args.steps}+{args.warmup} steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(w: synth.Workload, args):
    sizes = np.diff(w.node_offsets)
    return {"workload": args.workload, "mode": getattr(args, "mode", "fused"), "layout": getattr(args, "layout", "ragged"),
            "launch": "cuda graph replay" if getattr(args, "graph", False) else "api call per step", "name": w.name,
            "n_seq_or_layer_slots": w.n_seq, "h_qk": w.h_qk, "h_v": w.h_v,
            "d_k": w.d_k, "d_v": w.d_v, "tree_nodes": int(sizes.max()), "total_nodes": w.total_nodes,
            "in_dtype": w.in_dtype, "state_dtype": "f32", "out_dtype": w.out_dtype,
            "accepted_path_len_mean": float(np.diff(w.path_offsets).mean()),
            "tree_plan": "built once in front of the timed region" if getattr(args, "plan_once", False) else "per step",
            "l2_policy": "inputs rotate over buffer sets larger than L2 in total"}


def report(args):
    """--report: every workload once (this program as a child process per line), one markdown table on stdout."""
    peak, src = measured_peaks()
    rows = []
    runs = [(wl, "fused", "ours") for wl in WORKLOADS] + [(wl, "verify", "ours") for wl in WORKLOADS
                                                          if wl.startswith("sweep_")]
    runs += [(wl, "verify", "recurrent") for wl in WORKLOADS if wl.startswith("sweep_")]
    runs += [("stack48_T64", "separate", "ours")]
    runs = [r + ("ragged",) for r in runs]
    # the shape-static entry points on the padded layout (slots sharing one full-size tree)
    runs += [(wl, "fused", "ours", "padded") for wl in ("stack48_T64", "stack48_T256", "layer_T64")]
    runs += [(wl, "verify", "ours", "padded") for wl in WORKLOADS if wl.startswith("sweep_")]
    # ... with the plan of the shared tree built once for all layers (a layer's call is then the verify kernel alone)
    runs += [(wl, "verify", "ours", "padded, plan once") for wl in ("sweep_T128", "sweep_T256", "sweep_T512")]
    for wl, mode, impl, layout in runs:
        cmd = [sys.executable, os.path.abspath(__file__), "--workload", wl, "--mode", mode, "--impl", impl, "--steps",
               str(args.steps), "--warmup", str(args.warmup), "--min-time", str(args.min_time), "--no-e2e"]
        if layout != "ragged":
            cmd += ["--layout", "padded"] + (["--plan-once"] if "plan once" in layout else [])
        if wl != "stack48_T64" or mode != "fused":
            cmd += ["--oracle-slots", "4"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        line = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
        if res.returncode != 0 or not line:
            rows.append(f"| {wl} | {mode} | {impl}{'' if layout == 'ragged' else ', ' + layout} | failed (rc {res.returncode}) | | | | | |")
            continue
        d = json.loads(line[-1])
        cpu = d.get("cpu_baseline", {})
        rows.append("| {} | {} | {} | {:.1f} | {:.1f} | {:.0f} | {:.3f} | {:.3g} | {} |".format(
            wl, mode, impl if layout == "ragged" else impl + ", " + layout, d["ms_per_step"] * 1e3, d["timing"]["ms_per_step_fastest_region"] * 1e3,
            d["step_roofline"]["achieved_gbs"], d["step_roofline"]["frac_of_" + src], d["value"],
            "{:.3g} ({} cores)".format(cpu["value"], cpu["cores"]) if cpu else ""))
    print(f"| workload | mode | impl | us/step (median region) | us/step (fastest) | GB/s | fraction of {src} "
          f"{peak:.0f} GB/s | nodes/s | oracle nodes/s |")
    print("|---|---|---|---|---|---|---|---|---|")
    print("\n".join(rows))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "recurrent"],
                    help="ours: the library's kernels; reference: the fp64 oracle on the host cores; recurrent: the "
                         "per-branch recurrent GPU baseline (verify only)")
    ap.add_argument("--workload", default="stack48_T64", choices=WORKLOADS)
    ap.add_argument("--sets", type=int, default=0, help="buffer sets to rotate over (0 = enough to exceed 2x L2)")
    ap.add_argument("--min-time", type=float, default=0.5,
                    help="repeat the K-step timed region until this many seconds of device time are measured")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--oracle-slots", type=int, default=48, help="layer slots / sequences in the oracle's sample")
    ap.add_argument("--mode", default="fused", choices=["fused", "separate", "verify"],
                    help="fused: one gdn_tree_commit_verify call per step; separate: gdn_tree_verify + gdn_tree_commit; "
                         "verify: gdn_tree_verify alone (no commit; for kernel comparisons)")
    ap.add_argument("--layout", default="ragged", choices=["ragged", "padded"],
                    help="padded: the shape-static entry points on the dense [slots, T, heads, d] layout with the tree given "
                         "once for all layer slots (workloads whose slots share one full-size tree); trees of more than 64 "
                         "nodes then run as gdn_tree_plan once per step + gdn_tree_commit_padded + gdn_tree_verify_planned")
    ap.add_argument("--plan-once", action="store_true",
                    help="--layout padded, trees of more than 64 nodes: build the tree plan once in front of the timed "
                         "region instead of in every step (a stack of layers calling one after the other shares it)")
    ap.add_argument("--path-len", type=int, default=16,
                    help="workload stack48_T64_deep: nodes on the accepted path (0..16)")
    ap.add_argument("--graph", action="store_true",
                    help="fused mode: capture one step per buffer set in a CUDA graph and time replays")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--layers", type=int, default=48, help="layer slots of the stack workloads (profiling: fewer)")
    ap.add_argument("--report", action="store_true",
                    help="run every workload once (fused; the tree-size sweep also verify-only and with the recurrent "
                         "baseline) and print one markdown table")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.report:
        report(args)
        return
    if args.impl == "recurrent":
        args.mode = "verify"

    w = make_workload(args)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    import paper_2607_06763_b200 as gdn
    from paper_2607_06763_b200 import multi
    from paper_2607_06763_b200.binding import to_device as to_dev

    gdn.load_library()   # raises if the CUDA library is missing: there is no fallback
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    shape = gdn.GdnShape.from_workload(w)
    vbytes, cbytes, sbytes = algorithmic_bytes(w)
    n_sets = args.sets or max(2, int(np.ceil(2 * 126e6 / sbytes)) + 1)
    n_sets = min(n_sets, 64)
    sets = []
    ws_bytes = gdn.gdn_tree_workspace_bytes(shape)
    for _ in range(n_sets):   # same bytes in every set, distinct device buffers
        d = {n: to_dev(getattr(w, n)) for n in ("S0", "q", "k", "v", "g", "beta", "parent", "node_offsets",
                                                   "path_offsets")}
        d["path"] = to_dev(w.path if w.path.size else np.zeros(1, np.int32))
        odt = torch.float32 if w.out_dtype == synth.F32 else torch.bfloat16
        d["o"] = torch.empty((w.total_nodes, w.h_v, w.d_v), dtype=odt, device="cuda")
        d["ws"] = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        sets.append(d)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    padded = args.layout == "padded"
    if padded:
        # every slot carries the same full-size tree, so the ragged packing of the workload already is the padded
        # layout [slots, T, heads, d]; the tree, its node count and its accepted path are given once
        T = int(w.node_offsets[1])
        same = all(np.array_equal(w.parent[b * T:(b + 1) * T], w.parent[:T]) for b in range(w.n_seq))
        assert same and w.total_nodes == w.n_seq * T and args.impl == "ours", "--layout padded: one shared full-size tree"
        plen = int(w.path_offsets[1])
        path1 = np.zeros((1, shape.max_depth), np.int32)
        path1[0, :plen] = w.path[:plen]
        p_parent, p_nodes = to_dev(w.parent[:T].reshape(1, T).copy()), to_dev(np.array([T], np.int32))
        p_path, p_len = to_dev(path1), to_dev(np.array([plen], np.int32))
        plan_bytes = gdn.gdn_tree_plan_bytes(shape, 1)
        plan = torch.empty(max(plan_bytes, 256), dtype=torch.uint8, device="cuda")
        small = T <= 64
        if args.plan_once and not small:
            assert gdn.gdn_tree_plan(shape, 1, p_parent, p_nodes, plan, status, stream) == 0

    def step_verify_padded(d, stream=stream):
        if small:
            rc = gdn.gdn_tree_verify_padded(shape, 1, False, d["S0"], d["q"], d["k"], d["v"], d["g"], d["beta"], p_parent,
                                            p_nodes, d["o"], status, stream)
        else:
            if not args.plan_once:
                rc = gdn.gdn_tree_plan(shape, 1, p_parent, p_nodes, plan, status, stream)
                assert rc == 0, gdn.gdn_status_string(rc)
            rc = gdn.gdn_tree_verify_planned(shape, 1, False, d["S0"], d["q"], d["k"], d["v"], d["g"], d["beta"], plan,
                                             d["o"], status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)

    def step_fused_padded(d, stream=stream):
        if small:
            rc = gdn.gdn_tree_commit_verify_padded(shape, 1, False, d["S0"], T, d["k"], d["v"], d["g"], d["beta"],
                                                   p_parent, p_nodes, p_path, p_len, d["q"], d["k"], d["v"], d["g"],
                                                   d["beta"], p_parent, p_nodes, d["o"], status, stream)
            assert rc == 0, gdn.gdn_status_string(rc)
            return
        # the decode step of a larger tree: metadata once, commit of the previous path, verification
        if not args.plan_once:
            rc = gdn.gdn_tree_plan(shape, 1, p_parent, p_nodes, plan, status, stream)
            assert rc == 0, gdn.gdn_status_string(rc)
        rc = gdn.gdn_tree_commit_padded(shape, 1, False, d["S0"], d["k"], d["v"], d["g"], d["beta"], p_parent, p_nodes,
                                        p_path, p_len, status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)
        rc = gdn.gdn_tree_verify_planned(shape, 1, False, d["S0"], d["q"], d["k"], d["v"], d["g"], d["beta"], plan,
                                         d["o"], status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)

    def step_verify(d, stream=stream):
        if args.impl == "recurrent":
            rc = gdn.gdn_tree_verify_recurrent(shape, d["S0"], d["q"], d["k"], d["v"], d["g"], d["beta"], d["parent"],
                                               d["node_offsets"], d["o"], status, stream)
        else:
            rc = gdn.gdn_tree_verify(shape, d["S0"], d["q"], d["k"], d["v"], d["g"], d["beta"], d["parent"],
                                     d["node_offsets"], d["o"], d["ws"], ws_bytes, status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)

    def step_separate(d, stream=stream):
        step_verify(d, stream)
        rc = gdn.gdn_tree_commit(shape, d["S0"], d["k"], d["v"], d["g"], d["beta"], d["parent"], d["node_offsets"],
                                 d["path"], d["path_offsets"], status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)

    def step_fused(d, stream=stream):
        # one decode iteration as the paper schedules it: commit the previous step's accepted path, then verify
        # the new tree against the advanced state (here the previous and the new tree carry the same tensors)
        rc = gdn.gdn_tree_commit_verify(shape, d["S0"], d["k"], d["v"], d["g"], d["beta"], d["parent"],
                                        d["node_offsets"], d["path"], d["path_offsets"], d["q"], d["k"], d["v"],
                                        d["g"], d["beta"], d["parent"], d["node_offsets"], d["o"], d["ws"], ws_bytes,
                                        status, stream)
        assert rc == 0, gdn.gdn_status_string(rc)

    step = {"fused": step_fused, "separate": step_separate, "verify": step_verify}[args.mode]
    if padded:
        assert args.mode in ("fused", "verify"), "--layout padded: modes fused and verify"
        step = step_fused_padded if args.mode == "fused" else step_verify_padded

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(sets[i % n_sets])
    barrier()
    graphs = None
    if args.graph and args.mode == "fused" and padded:
        graphs, side = [], torch.cuda.Stream()
        for d in sets:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                step_fused_padded(d, torch.cuda.current_stream())
            graphs.append(g)
        for i in range(args.warmup):
            graphs[i % n_sets].replay()
        barrier()
    elif args.graph and args.mode == "fused":
        # one captured step per buffer set (the launches of a call, dependent-launch edge included)
        graphs, side = [], torch.cuda.Stream()
        for d in sets:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                step_fused(d, torch.cuda.current_stream())
            graphs.append(g)
        for i in range(args.warmup):
            graphs[i % n_sets].replay()
        barrier()
    assert int(status.item()) == 0, gdn.gdn_status_string(int(status.item()))

    # ---- timed span: the K-step region, repeated.  Nothing but the calls themselves sits inside a region (an event
    # between two steps would keep the next call's kernel from being launched under the tail of this one).
    counter = [args.warmup]

    def region():
        t_start = torch.cuda.Event(enable_timing=True)
        t_end = torch.cuda.Event(enable_timing=True)
        barrier()
        t_start.record()
        for _ in range(args.steps):
            i = counter[0] % n_sets
            counter[0] += 1
            if graphs is not None:
                graphs[i].replay()
            else:
                step(sets[i])
        t_end.record()
        barrier()
        return t_start.elapsed_time(t_end)

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    wall0 = time.time()
    region_ms = [region()]
    # every rank runs the same number of regions: enough for --min-time at the slowest rank's first region
    first = multi.reduce_max(region_ms[0], "cuda")
    n_regions = max(1, min(5000, int(np.ceil(args.min_time * 1e3 / max(first, 1e-3)))))
    for _ in range(n_regions - 1):
        region_ms.append(region())
    wall1 = time.time()
    time.sleep(0.15)
    clocks = sampler.stop(wall0, wall1)
    assert int(status.item()) == 0, gdn.gdn_status_string(int(status.item()))
    med_region, min_region = statistics.median(region_ms), min(region_ms)
    value, ms_per_step = multi.aggregate_throughput(w.total_nodes, med_region / args.steps, "cuda")
    nodes_per_step = w.total_nodes * world

    # separate mode: how the step splits between the two kernels (events between the calls; not the headline timing)
    split = None
    if args.mode == "separate":
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(50)]
        for e in ev:
            d = sets[counter[0] % n_sets]
            counter[0] += 1
            e[0].record()
            step_verify(d)
            e[1].record()
            rc = gdn.gdn_tree_commit(shape, d["S0"], d["k"], d["v"], d["g"], d["beta"], d["parent"], d["node_offsets"],
                                     d["path"], d["path_offsets"], status, stream)
            assert rc == 0
            e[2].record()
        barrier()
        split = (statistics.median(e[0].elapsed_time(e[1]) for e in ev),
                 statistics.median(e[1].elapsed_time(e[2]) for e in ev))

    # ---- end-to-end: host buffers through the *_host entry points (copies inside the timed region)
    L = int(w.path_offsets[-1])
    fused_e2e = args.mode == "fused"
    isz = 4 if w.in_dtype == synth.F32 else 2
    osz = 4 if w.out_dtype == synth.F32 else 2
    state_b = w.n_seq * w.h_v * w.d_v * w.d_k * 4
    qk_b, v_b, gb_b = w.total_nodes * w.h_qk * w.d_k * isz, w.total_nodes * w.h_v * w.d_v * isz, w.total_nodes * w.h_v * isz
    idx_b = 4 * (w.total_nodes + 2 * (w.n_seq + 1) + (w.n_seq + 1) + L)
    if fused_e2e:   # state up once; the previous step's k, v, g, beta and the new tree's q, k, v, g, beta
        h2d = state_b + (qk_b + v_b + 2 * gb_b) + (2 * qk_b + v_b + 2 * gb_b) + idx_b + 4 * (w.total_nodes + w.n_seq + 1)
        d2h = w.total_nodes * w.h_v * w.d_v * osz + state_b + 4
    else:
        h2d = (state_b + 2 * qk_b + v_b + 2 * gb_b) + (state_b + qk_b + v_b + 2 * gb_b) + idx_b
        d2h = w.total_nodes * w.h_v * w.d_v * osz + state_b + 8
    e2e = None
    if not args.no_e2e and args.impl == "ours" and args.mode != "verify":
        arena_bytes = (gdn.gdn_tree_commit_verify_host_arena_bytes(shape, w.total_nodes, L) if fused_e2e
                       else gdn.gdn_tree_host_arena_bytes(shape, L))
        arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
        pin = {n: torch.from_numpy(np.ascontiguousarray(getattr(w, n)).view(np.int16) if getattr(w, n).dtype == np.uint16
                                   else np.ascontiguousarray(getattr(w, n))).pin_memory()
               for n in ("S0", "q", "k", "v", "g", "beta", "parent", "node_offsets", "path_offsets")}
        pin["path"] = torch.from_numpy(w.path if w.path.size else np.zeros(1, np.int32)).pin_memory()
        o_pin = torch.empty(w.total_nodes * w.h_v * w.d_v * osz, dtype=torch.uint8).pin_memory()

        def e2e_step():
            if fused_e2e:
                # the user's call for one decode iteration: commit of the previous step's paths + verify of the tree,
                # every tensor in pinned host memory (here the previous and the new tree carry the same tensors)
                rc = gdn.gdn_tree_commit_verify_host(shape, pin["S0"], w.total_nodes, pin["k"], pin["v"], pin["g"],
                                                     pin["beta"], pin["parent"], pin["node_offsets"], pin["path"],
                                                     pin["path_offsets"], L, pin["q"], pin["k"], pin["v"], pin["g"],
                                                     pin["beta"], pin["parent"], pin["node_offsets"], o_pin, arena,
                                                     arena_bytes, stream)
                assert rc == 0, gdn.gdn_status_string(rc)
                return
            rc = gdn.gdn_tree_verify_host(shape, pin["S0"], pin["q"], pin["k"], pin["v"], pin["g"], pin["beta"],
                                          pin["parent"], pin["node_offsets"], o_pin, arena, arena_bytes, stream)
            assert rc == 0, gdn.gdn_status_string(rc)
            rc = gdn.gdn_tree_commit_host(shape, pin["S0"], pin["k"], pin["v"], pin["g"], pin["beta"], pin["parent"],
                                          pin["node_offsets"], pin["path"], pin["path_offsets"], L, arena, arena_bytes,
                                          stream)
            assert rc == 0, gdn.gdn_status_string(rc)

        for _ in range(2):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        barrier()
        e2e_s = multi.reduce_max((time.perf_counter() - t0) / args.e2e_steps, "cuda")
        e2e = {"value": nodes_per_step / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": e2e_s * 1e3}

    if rank == 0:
        peak, peak_src = measured_peaks()
        fused = args.mode == "fused"
        single_cta_trees = int(np.diff(w.node_offsets).max()) <= 64
        # dominant kernel and what one launch of it moves: fused mode -- the commit+verify kernel moves the whole
        # step's bytes; otherwise the verify kernel moves S0 + node tensors + o
        if args.impl == "recurrent":
            kernel_name, launches_per_step, dom_bytes, dom_ms = "verify_recurrent_kernel", 1, vbytes, ms_per_step
        elif single_cta_trees:
            kernel_name = "verify_sm100_persistent_kernel<fused commit>" if fused else "verify_sm100_persistent_kernel"
            launches_per_step = {"fused": 1, "separate": 2, "verify": 1}[args.mode]
            dom_bytes = sbytes if fused else vbytes
            dom_ms = ms_per_step if args.mode != "separate" else split[0]
        else:   # larger trees: tree plan + the verify kernel in its grouped mode; the fused call builds the plan in
                # extra CTAs of the commit kernel's grid (two launches), the padded layout plans in a call of its own
            kernel_name = "verify_sm100_persistent_kernel<grouped>"
            launches_per_step = {"fused": 3 if args.layout == "padded" else 2, "separate": 3, "verify": 2}[args.mode]
            dom_bytes = vbytes
            dom_ms = None if args.mode == "fused" else (ms_per_step if args.mode == "verify" else split[0])
        step_bytes = sbytes if args.mode != "verify" else vbytes
        achieved = dom_bytes / (dom_ms * 1e-3) / 1e9 if dom_ms else step_bytes / (ms_per_step * 1e-3) / 1e9
        traffic = captured_traffic(args.workload, args.mode, w.n_seq) if args.impl == "ours" else None
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": DTYPE if w.in_dtype == synth.BF16 else "f32", "data": "synthetic",
            "config": workload_config(w, args), "mode": args.mode, "impl": args.impl,
            "timing": {"regions": len(region_ms), "steps_per_region": args.steps,
                       "ms_per_step_median_region": med_region / args.steps,
                       "ms_per_step_fastest_region": min_region / args.steps,
                       "device_time_s": sum(region_ms) * 1e-3},
            "verify_commit_us": ms_per_step * 1e3,
            "step_bytes": step_bytes,
            "step_roofline": {"achieved_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9, "peak_gbs": peak,
                              "frac_of_" + peak_src: step_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
                              "frac_of_nominal_8000": step_bytes / (ms_per_step * 1e-3) / 1e9 / 8000.0},
            "roofline": {"kernel": kernel_name, "bound": "hbm", "achieved": achieved, "peak": peak,
                         "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic["bytes_per_launch"] if traffic else None,
                         "traffic_detail": traffic,
                         "bytes_per_launch": dom_bytes if dom_ms else step_bytes,
                         "avg_launch_us": (dom_ms if dom_ms else ms_per_step) * 1e3,
                         "note": ("launch time = timed region / steps (one kernel per call)" if dom_ms == ms_per_step
                                  else "launch time from events around the verify call" if dom_ms
                                  else "whole step (commit + plan kernel, grouped verify kernel) over the step's bytes")},
            "gpu_launches": launches_per_step * args.steps * len(region_ms),
            "gpu_launches_per_step": launches_per_step,
            "clocks": clocks, "buffer_sets": n_sets,
            "paper_context": {"fused_verify_us_one_layer_B200": {"T64": 27.8, "T128": 44.7},
                              "recurrent_over_fused_at_T128": 7.1,
                              "note": "Table 1 / Section 5.2, the paper's own build; context only"},
        }
        if e2e:
            out["e2e"] = e2e
        else:
            out["e2e"] = {"value": None, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                          "note": "skipped (--no-e2e, --mode verify or --impl recurrent)"}
        if split:
            out["verify_us"], out["commit_us"] = split[0] * 1e3, split[1] * 1e3
            out["commit_roofline"] = {"bound": "hbm", "achieved": cbytes / (split[1] * 1e-3) / 1e9, "peak": peak,
                                      "unit": "GB/s", "frac": cbytes / (split[1] * 1e-3) / 1e9 / peak,
                                      "bytes_per_launch": cbytes}
        if world == 1 and not args.no_cpu_baseline:
            run, nodes, n_slots, cores = oracle_sample(w, args.oracle_slots)
            dt = run()
            out["cpu_baseline"] = {"value": nodes / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": f"first {n_slots} of {w.n_seq} layer slots/sequences ({nodes} nodes), "
                                             f"verify + commit, one pass, {dt:.2f} s"}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
