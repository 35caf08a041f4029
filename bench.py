#!/usr/bin/env python
"""Benchmark of the sampling-verification hot path (SpecHub + RRS + RRSw).

One step = the whole hot path over one synthetic batch: for each of the three
methods, the draft step, the verification of every tree node and the tree walk,
all on one stream.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl reference]
  python bench.py --workload all      # every configuration and both layouts, one JSON line with a table

Timing: CUDA events on the launching stream, barrier + synchronize on both
sides, max over ranks.  The headline workloads' inputs (several GB) are far
larger than L2, so no flush is needed between steps; the small workloads rotate
over enough distinct input copies to exceed L2.  Multi-GPU: every rank runs its own batch of the same
shape (no collective on the data path), so scaling is weak.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "tree-nodes verified/sec"
UNIT = "nodes/s"
METHODS = ("spechub", "rrs", "rrsw")

# dram__bytes_read.sum + dram__bytes_write.sum of one launch over 992 (sequence, node) rows of the
# headline shape, from an ncu capture of the kernels as they stand (the test suite checks these numbers
# against the committed capture summary); a launch's traffic is this per row times its row count
# (traffic grows in proportion to the rows).  Keyed by (API call, workload); absent = not captured.  The capture
# is of the default step (--draft-stats on, --verify-path default); any other path reports no traffic.
TRAFFIC_PER_ROW = {
    ("spechub_draft_sample", "c4"): 275593472.0 / 992,
    ("spechub_verify_tree", "c4"): 624340992.0 / 992,
    ("rrs_draft_sample[rrs]", "c4"): 281195008.0 / 992,
    ("rrs_verify_tree[rrs]", "c4"): 977194496.0 / 992,
    ("rrs_draft_sample[rrsw]", "c4"): 279507712.0 / 992,
    ("rrs_verify_tree[rrsw]", "c4"): 1008760320.0 / 992,
}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(workloads.all_configs()) + ["all"])
    ap.add_argument("--layout", default="dense", choices=["dense", "paper"],
                    help="dense: every node verifies; paper: last-level nodes only draw the bonus token")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch (profiling on a small case; not a bench value)")
    ap.add_argument("--verify-path", default="default", choices=["default", "streaming", "split2", "split4", "resident"],
                    help="large-vocabulary verification kernels: the library's choice, the two-pass streaming "
                         "kernels (one CTA per row, or a row split over 2 / 4 CTAs), or the kernels that keep the "
                         "exponentials on chip")
    ap.add_argument("--draft-stats", default="on", choices=["on", "off"],
                    help="on: the step goes through the *_stats entry points (the draft call hands its per-row "
                         "statistics of the draft logits to the verification call); off: the plain entry points")
    ap.add_argument("--kary-leg", action="store_true",
                    help="also time RRS / RRSw with three drafts per node on a ternary 40-node tree of the "
                         "workload's vocabulary (reported in breakdown, not part of `value`)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the oracle timing leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def config_dict(cfg, layout, n_gpus):
    return {
        "workload": "%s: batch %d x %d-node binary tree, V=%d, %s logits, T=%g, layout=%s" % (
            cfg.name, cfg.batch, cfg.nodes, cfg.vocab, cfg.dtype, cfg.temperature, layout),
        "methods": list(METHODS),
        "global_batch": cfg.batch * n_gpus,
        "nodes": cfg.nodes,
        "vocab": cfg.vocab,
        "parallelism": "batch-sharded x%d, no collective" % n_gpus,
        "l2": l2_note(cfg),
    }


L2_BYTES = 126e6


def esz0(cfg):
    return 2 if cfg.dtype == "bf16" else 4


def input_bytes(cfg):
    return 2 * cfg.rows * cfg.vocab * (2 if cfg.dtype == "bf16" else 4)


def input_copies(cfg):
    """Distinct copies of the inputs the timed steps rotate over, so that no step finds its rows
    in L2: one when a single copy is already larger than twice the L2, else enough to exceed it."""
    b = input_bytes(cfg)
    return 1 if b >= 2 * L2_BYTES else int(-(-3 * L2_BYTES // b))


def l2_note(cfg):
    n = input_copies(cfg)
    if n == 1:
        return "inputs larger than L2 (%.2f GB per rank)" % (input_bytes(cfg) / 1e9)
    return "steps rotate over %d distinct input copies (%.2f GB in all per rank), more than L2" % (
        n, n * input_bytes(cfg) / 1e9)


# ---- the oracle leg (CPU baseline, and --impl reference) -----------------------------------------

def oracle_sample(cfg, layout, seconds):
    """Time the CPU oracle, as it stands, on whole sequences of the workload until about
    `seconds` of work is done.  Returns (node verifications per second, description)."""
    import oracle

    oracle.build()
    kind = workloads.paper_node_kind(cfg.nodes) if layout == "paper" else None
    prior = workloads._prior(cfg)
    done_nodes, spent, b = 0, 0.0, 0
    while True:
        lp, lq = workloads.host_sequence(cfg, b % cfg.batch, prior)
        un = workloads.host_uniforms(cfg, [b % cfg.batch])
        lp, lq = lp[None], lq[None]
        t0 = time.perf_counter()
        for m in METHODS:
            d = oracle.draft_batch(m, lq, cfg.temperature, un)
            out = oracle.verify_batch(m, lp, lq, cfg.temperature, d["tokens"], un, kind)
            oracle.walk(out["accept_idx"], out["token"], cfg.levels, node_kind=kind)
        spent += time.perf_counter() - t0
        done_nodes += len(METHODS) * cfg.nodes
        b += 1
        if spent >= seconds or b >= cfg.batch:
            break
    return done_nodes / spent, "%d whole sequences (%d nodes each) x %d methods, %.1f s" % (
        b, cfg.nodes, len(METHODS), spent), spent


def oracle_all_cores(cfg, layout, one_core_rate, seconds):
    """The same oracle fanned out over the host's cores by ranges of sequences (processes; the oracle
    itself stays single-threaded).  `one_core_rate` sizes the sample to about `seconds` of wall time."""
    from oracle import fanout

    n = fanout.cores()
    per_seq = len(METHODS) * cfg.nodes / max(one_core_rate, 1e-9)          # seconds of one core per sequence
    S = int(max(n, min(cfg.batch, 4 * n, seconds * n / max(per_seq, 1e-9))))
    S = min(S, cfg.batch)
    kind = workloads.paper_node_kind(cfg.nodes) if layout == "paper" else None
    prior = workloads._prior(cfg)
    seqs = [workloads.host_sequence(cfg, b, prior) for b in range(S)]
    lp = np.stack([s[0] for s in seqs]); lq = np.stack([s[1] for s in seqs])
    un = workloads.host_uniforms(cfg, list(range(S)))
    del seqs
    with fanout.Pool(n) as pool:
        pool.draft_batch("rrs", lq[:n], cfg.temperature, un[:n])             # workers started and warm
        t0 = time.perf_counter()
        for m in METHODS:
            d = pool.draft_batch(m, lq, cfg.temperature, un)
            pool.verify_batch(m, lp, lq, cfg.temperature, d["tokens"], un, kind)
        spent = time.perf_counter() - t0
    return {"value": len(METHODS) * S * cfg.nodes / spent, "unit": UNIT, "cores": n, "kind": "oracle",
            "sample": "%d whole sequences (%d nodes each) x %d methods over %d worker processes, %.1f s "
                      "(logits handed over in shared memory, inside the timed region)" % (
                          S, cfg.nodes, len(METHODS), n, spent)}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = max(0.5, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(cfg, args.layout, per_step / 4)
    vals, times = [], []
    for _ in range(args.steps):
        v, desc, spent = oracle_sample(cfg, args.layout, per_step)
        vals.append(v); times.append(spent)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(cfg, args.layout, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": "each step: " + desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---- clocks ------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.rows = []
        self.proc = None

    def start(self):
        try:
            cmd = ["nvidia-smi", "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "100"]
            if self.uuid:
                cmd += ["-i", self.uuid]
            self.proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(np.max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---- the GPU arm -------------------------------------------------------------------------------------

def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s)"


def run_table(args):
    """Every configuration (config 3 as its four variants) in both layouts: one bench run each, in a
    process of its own, gathered into one JSON line.  The headline `value` stays config 4's."""
    names = ["c1", "c2"] + [v.name for v in workloads.variants("c3")] + ["c4", "c5"]
    peak, peak_src = measured_peak()
    table = []
    for name in names:
        for layout in ("dense", "paper"):
            cmd = [sys.executable, os.path.abspath(__file__), "--workload", name, "--layout", layout,
                   "--steps", str(args.steps), "--warmup", str(args.warmup), "--e2e-steps", "1",
                   "--no-cpu-baseline", "--verify-path", args.verify_path, "--draft-stats", args.draft_stats]
            out = subprocess.run(cmd, capture_output=True, text=True)
            lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
            if out.returncode != 0 or not lines:
                table.append({"workload": name, "layout": layout, "error": (out.stderr or "no output")[-300:]})
                continue
            d = json.loads(lines[-1])
            k = d["kernels"]
            table.append({
                "workload": name, "layout": layout,
                "nodes_per_s_three_methods": d["value"], "ms_per_step": d["ms_per_step"],
                "spechub_nodes_per_s": d["breakdown"]["spechub_only_step"]["nodes_per_s"],
                "spechub_verify_vocab_elements_per_s": d["breakdown"]["spechub_verify_vocab_elements_per_s"],
                "ms_per_call": {c: k[c]["ms_per_launch"] for c in k},
                "frac_of_measured_peak": {c: k[c]["frac"] for c in k},
                "frac_of_8TBs": {c: k[c]["frac_of_nominal_8TBs"] for c in k},
                "clocks": d.get("clocks"),
            })
    print(json.dumps({"metric": METRIC, "unit": UNIT, "table": table, "peak_GBs": peak, "peak_source": peak_src,
                      "steps": args.steps, "note": "one process per row of the table; fractions are algorithmic "
                      "bytes / CUDA-event time over the HBM peak"}), flush=True)


def main():
    args = parse()
    if args.workload == "all":
        if int(os.environ.get("RANK", "0")) == 0:
            run_table(args)
        return
    cfg = workloads.lookup(args.workload)
    if args.batch:
        from dataclasses import replace as _replace

        cfg = _replace(cfg, name=cfg.name + "-batch%d" % args.batch, batch=args.batch)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist

    import paper_2411_05289_b200 as sh

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sh.load_library()
    sh.set_row_split({"default": 0, "streaming": 1, "split2": 2, "split4": 4, "resident": 8}[args.verify_path])

    # this rank's batch (same shape on every rank, its own seed)
    from dataclasses import replace

    rcfg = replace(cfg, seed=cfg.seed + 17 * rank)
    tp, tq = workloads.device_logits(rcfg, device=dev)
    un = workloads.device_uniforms(rcfg, device=dev)
    B, N, V = tp.shape
    # small workloads: the timed steps rotate over distinct copies so that none runs out of L2
    copies = [(tp, tq, un)]
    for i in range(1, input_copies(cfg)):
        ccfg = replace(rcfg, seed=rcfg.seed + 1009 * i)
        copies.append(workloads.device_logits(ccfg, device=dev) + (workloads.device_uniforms(ccfg, device=dev),))
    turn = [0]
    tree = sh.Tree.heap(N, leaves_sample=(args.layout == "paper"), device=dev)
    from paper_2411_05289_b200.binding import alloc_verify_outputs

    outs = {m: alloc_verify_outputs(B, N, tree.levels, dev) for m in METHODS}
    stream = torch.cuda.current_stream()
    ev_pairs = {}  # API call -> list of (start, stop) events recorded inside the timed steps

    def timed(name, record, fn):
        if not record:
            return fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        r = fn()
        e1.record(stream)
        ev_pairs.setdefault(name, []).append((e0, e1))
        return r

    # The two calls of a method: with --draft-stats on (default) the draft call leaves its per-row statistics
    # of the draft logits (16 bytes a row) for the verification call, which then reads the draft rows once
    # instead of twice; off = the plain entry points.
    hand_over = args.draft_stats == "on"

    def do_draft(m, tq, un, ho=None):
        ho = hand_over if ho is None else ho
        if m == "spechub":
            return (sh.spechub_draft_sample_stats if ho else sh.spechub_draft_sample)(tq, un, tree, cfg.temperature)
        return (sh.rrs_draft_sample_stats if ho else sh.rrs_draft_sample)(tq, un, tree, m == "rrsw", cfg.temperature)

    def do_verify(m, tp, tq, d, un, out, ho=None):
        ho = hand_over if ho is None else ho
        if m == "spechub":
            if ho:
                return sh.spechub_verify_tree_stats(tp, tq, d["stats"], d["tokens"], un, tree, cfg.temperature, out=out)
            return sh.spechub_verify_tree(tp, tq, d["tokens"], un, tree, cfg.temperature, out=out)
        if ho:
            return sh.rrs_verify_tree_stats(tp, tq, d["stats"], d["tokens"], un, tree, m == "rrsw", cfg.temperature, out=out)
        return sh.rrs_verify_tree(tp, tq, d["tokens"], un, tree, m == "rrsw", cfg.temperature, out=out)

    def call_name(kind, m):
        return "spechub_%s" % kind if m == "spechub" else "rrs_%s[%s]" % (kind, m)

    def step(record=False):
        tp, tq, un = copies[turn[0] % len(copies)]
        turn[0] += 1
        for m in METHODS:
            d = timed(call_name("draft_sample", m), record, lambda: do_draft(m, tq, un))
            timed(call_name("verify_tree", m), record, lambda: do_verify(m, tp, tq, d, un, outs[m]))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        pass
    clk = ClockSampler(uuid)
    if rank == 0:
        clk.start()
        time.sleep(0.3)
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(args.steps):
        step(record=True)
    t1.record(stream)
    barrier()
    ms = t0.elapsed_time(t1)
    clocks = clk.stop() if rank == 0 else None
    # per API call: mean device time of its kernels (a verify call = verification kernel + walk kernel)
    call_ms = {k: float(np.mean([a.elapsed_time(b) for a, b in v])) for k, v in ev_pairs.items()}
    verify_ms = call_ms["spechub_verify_tree"]

    # ---- extra: the same step through the other set of entry points (plain if the timed step hands the draft
    # statistics over, and the other way round) ----
    def other_step():
        tp_, tq_, un_ = copies[turn[0] % len(copies)]
        turn[0] += 1
        for m in METHODS:
            d = do_draft(m, tq_, un_, not hand_over)
            do_verify(m, tp_, tq_, d, un_, outs[m], not hand_over)

    for _ in range(3):
        other_step()
    barrier()
    o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    o0.record(stream)
    for _ in range(args.steps):
        other_step()
    o1.record(stream)
    barrier()
    other_ms = o0.elapsed_time(o1) / args.steps

    # ---- extra: SpecHub verification when the caller asks for decisions and tokens only ----
    d0 = sh.spechub_draft_sample(tq, un, tree, cfg.temperature)
    for _ in range(2):
        sh.spechub_verify_tree(tp, tq, d0["tokens"], un, tree, cfg.temperature, out=outs["spechub"], probabilities=False)
    barrier()
    q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    q0.record(stream)
    for _ in range(args.steps):
        sh.spechub_verify_tree(tp, tq, d0["tokens"], un, tree, cfg.temperature, out=outs["spechub"], probabilities=False)
    q1.record(stream)
    barrier()
    lite_ms = q0.elapsed_time(q1) / args.steps

    # ---- extra: the same step through the three-method calls (shared reads of p and q) ----
    def fused_step():
        if hand_over:
            d = sh.mdsd_compare_draft_sample_stats(tq, un, tree, cfg.temperature)
            sh.mdsd_compare_verify_tree_stats(tp, tq, d["stats"], {m: d[m]["tokens"] for m in METHODS}, un, tree,
                                              cfg.temperature, out=outs)
            return
        d = sh.mdsd_compare_draft_sample(tq, un, tree, cfg.temperature)
        sh.mdsd_compare_verify_tree(tp, tq, {m: d[m]["tokens"] for m in METHODS}, un, tree, cfg.temperature,
                                    out=outs)

    for _ in range(3):
        fused_step()
    barrier()
    q0.record(stream)
    for _ in range(args.steps):
        fused_step()
    q1.record(stream)
    barrier()
    fused_ms = q0.elapsed_time(q1) / args.steps

    # ---- extra: the timed step replayed as CUDA graphs (one per input copy): what is left when the
    # host cost of nine Python calls per step is taken away; matters for the small workloads ----
    graph_ms = None
    try:
        graphs = []
        for i in range(len(copies)):
            turn[0] = i
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph):
                step()
            graphs.append(gph)
        for gph in graphs:
            gph.replay()
        barrier()
        q0.record(stream)
        for i in range(args.steps):
            graphs[i % len(graphs)].replay()
        q1.record(stream)
        barrier()
        graph_ms = q0.elapsed_time(q1) / args.steps
    except Exception as exc:  # reported, never fatal: the timed region above does not depend on it
        graph_ms = None
        graph_note = "capture failed: %s" % (str(exc).splitlines()[0][:120])
    else:
        graph_note = "same nine launches per step, replayed from %d captured graph(s); not part of `value`" % len(copies)

    # ---- extra: Algorithm 1 with three drafts per node (the paper's ternary trees) ----
    kary = None
    if args.kary_leg:
        t3 = sh.Tree.kary(3, 4, device=dev)
        N3 = t3.nodes_of_complete_tree()
        gen = torch.Generator(device=dev); gen.manual_seed(cfg.seed + 3)
        dt = tp.dtype
        kp = (torch.randn((B, N3, V), device=dev, generator=gen) * 2.0).to(dt)
        kq = (kp.float() + torch.randn((B, N3, V), device=dev, generator=gen)).to(dt)
        ku = (torch.randint(0, 1 << 24, (B, N3, 7), device=dev, generator=gen).float() * 2.0 ** -24)
        kary = {"tree": "ternary, 4 levels, %d nodes" % N3, "batch": B, "vocab": V,
                "alg_bytes_per_verify": B * N3 * (2 * V * esz0(cfg) + 12 + 28 + 44)}
        for wo in (False, True):
            kd = sh.rrs_draft_sample(kq, ku, t3, wo, cfg.temperature)
            ko = alloc_verify_outputs(B, N3, t3.levels, dev, 3)
            for _ in range(3):
                sh.rrs_verify_tree(kp, kq, kd["tokens"], ku, t3, wo, cfg.temperature, out=ko)
            barrier()
            q0.record(stream)
            for _ in range(args.steps):
                sh.rrs_verify_tree(kp, kq, kd["tokens"], ku, t3, wo, cfg.temperature, out=ko)
            q1.record(stream)
            barrier()
            t_ms = q0.elapsed_time(q1) / args.steps
            kary["rrsw" if wo else "rrs"] = {"verify_ms": t_ms, "nodes_per_s": B * N3 / (t_ms * 1e-3),
                                             "algorithmic_GBs": kary["alg_bytes_per_verify"] / (t_ms * 1e-3) / 1e9}
        del kp, kq, ku

    # ---- end to end: host buffers in, host results out, through the public API ----
    esz = 2 if cfg.dtype == "bf16" else 4
    h_tp = torch.empty(tp.shape, dtype=tp.dtype, pin_memory=True); h_tp.copy_(tp)
    h_tq = torch.empty(tq.shape, dtype=tq.dtype, pin_memory=True); h_tq.copy_(tq)
    h_un = torch.empty(un.shape, dtype=un.dtype, pin_memory=True); h_un.copy_(un)
    res_keys = ("n_accepted", "n_emitted", "path_tokens", "accept_idx", "token")
    h_res = {m: {k: torch.empty(outs[m][k].shape, dtype=outs[m][k].dtype, pin_memory=True) for k in res_keys}
             for m in METHODS}
    h2d = (h_tp.numel() + h_tq.numel()) * esz + h_un.numel() * 4
    d2h = sum(v.numel() * v.element_size() for m in METHODS for v in h_res[m].values())

    # The batch goes through in chunks of whole sequences on two streams, so that the copy of one
    # chunk overlaps the kernels of the one before; the library only enqueues on the given stream.
    n_chunks = max(1, min(8, B, int(input_bytes(cfg) // 400e6)))  # chunks of >= 0.4 GB: launches stay rare
    bounds = [(B * i // n_chunks, B * (i + 1) // n_chunks) for i in range(n_chunks)]
    side = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]
    chunk_outs = [{m: {k: v[b0:b1] for k, v in outs[m].items()} for m in METHODS} for b0, b1 in bounds]

    def e2e_step():
        fork = torch.cuda.Event()
        fork.record(stream)
        for ci, (b0, b1) in enumerate(bounds):
            st = side[ci % 2]
            if ci < 2:
                st.wait_event(fork)
            with torch.cuda.stream(st):
                ctp, ctq, cun = tp[b0:b1], tq[b0:b1], un[b0:b1]
                ctp.copy_(h_tp[b0:b1], non_blocking=True)
                ctq.copy_(h_tq[b0:b1], non_blocking=True)
                cun.copy_(h_un[b0:b1], non_blocking=True)
                co = chunk_outs[ci]
                d = do_draft("spechub", ctq, cun)
                do_verify("spechub", ctp, ctq, d, cun, co["spechub"])
                for m, wo in (("rrs", False), ("rrsw", True)):
                    d = do_draft(m, ctq, cun)
                    do_verify(m, ctp, ctq, d, cun, co[m])
                for m in METHODS:
                    for k in res_keys:
                        h_res[m][k][b0:b1].copy_(co[m][k], non_blocking=True)
        for st in side:
            join = torch.cuda.Event()
            join.record(st)
            stream.wait_event(join)

    e2e_step()
    barrier()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record(stream)
    for _ in range(args.e2e_steps):
        e2e_step()
    g1.record(stream)
    barrier()
    e2e_s = g0.elapsed_time(g1) * 1e-3

    # ---- several GPUs only: the same SpecHub step with the VOCABULARY sharded over the ranks (a tensor-
    # parallel LM head): every rank holds an id range of the same rows, runs the phase kernels on its own
    # slice and exchanges 32 bytes per row between them (two all-gathers and one maximum per call over
    # NCCL; no kernel is given a peer's memory).  Reported beside the batch-sharded headline.
    vs_ms, vs_err = None, None
    if world > 1:
        try:
            from paper_2411_05289_b200 import vocab_sharded as vsh

            ctp, ctq = workloads.device_logits(cfg, device=dev)      # the common rows: same seed on every rank
            cun = workloads.device_uniforms(cfg, device=dev)
            shard, sp = vsh.slice_of_rank(ctp, rank, world)
            _, sq = vsh.slice_of_rank(ctq, rank, world)
            del ctp, ctq

            def vs_step():
                d = vsh.spechub_draft_sample_sharded(sq, cun, tree, shard, cfg.temperature)
                return vsh.spechub_verify_tree_sharded(sp, sq, d["tokens"], cun, tree, shard, cfg.temperature)

            for _ in range(3):
                vs_step()
            barrier()
            q0.record(stream)
            for _ in range(args.steps):
                vs_step()
            q1.record(stream)
            barrier()
            vs_ms = q0.elapsed_time(q1) / args.steps
            del sp, sq
        except Exception as exc:   # every rank runs the same code on the same shapes: a failure is common to all
            vs_err = str(exc).splitlines()[0][:160] if str(exc) else repr(exc)

    tms = torch.tensor([ms, e2e_s * 1e3, verify_ms, vs_ms or 0.0], device=dev, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(tms, op=dist.ReduceOp.MAX)
    ms, e2e_ms, verify_ms, vs_ms = [float(x) for x in tms.tolist()]

    if rank == 0:
        nodes_per_step = len(METHODS) * B * N * world
        value = nodes_per_step * args.steps / (ms * 1e-3)
        e2e_value = nodes_per_step * args.e2e_steps / (e2e_ms * 1e-3)
        kind = workloads.paper_node_kind(N) if args.layout == "paper" else np.zeros(N, np.uint8)
        n_leaf = int(kind.sum())
        rec = 16 if hand_over else 0   # the per-row record of draft statistics: written by the draft call, read by verification
        alg_bytes = B * ((N - n_leaf) * (2 * V * esz + 8 + 20 + 44 + rec) + n_leaf * (V * esz + 20 + 44))
        draft_bytes = B * N * (V * esz + 8 + 8 + 16 + rec)
        peak, peak_src = measured_peak()
        total_call_ms = sum(call_ms.values())
        roof = {}
        for name, t_ms in call_ms.items():
            nbytes = draft_bytes if "draft" in name else alg_bytes
            ach = nbytes / (t_ms * 1e-3) / 1e9
            roof[name] = {"bound": "hbm", "kernel": name, "achieved": ach, "peak": peak, "unit": "GB/s",
                          "frac": ach / peak, "peak_source": peak_src, "frac_of_nominal_8TBs": ach / 8000.0,
                          "traffic": (TRAFFIC_PER_ROW[(name, args.workload)] * B * N
                                      if (name, args.workload) in TRAFFIC_PER_ROW and args.layout == "dense"
                                      and args.verify_path == "default" and hand_over else None),
                          "alg_bytes_per_launch": nbytes,
                          "ms_per_launch": t_ms, "share_of_step": t_ms / total_call_ms}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(config_dict(cfg, args.layout, world),
                           draft_stats=("the draft call hands max / argmax / sum of each draft row to the verification "
                                        "call (*_stats entry points), written and read inside every timed step: verification's first pass "
                                        "reads the target row only"
                                        if hand_over else "off: plain entry points")),
            "value_note": "each node is counted once per method (SpecHub, RRS, RRSw run one after another on the "
                          "same inputs): node-method verifications; SpecHub alone is breakdown.spechub_only_step",
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": args.e2e_steps, "chunks": n_chunks,
                    "note": "pinned host buffers -> device -> public API -> pinned host results; "
                            "chunks of whole sequences on two streams (copies overlap kernels).  Bound by the "
                            "host link: the logits (h2d_bytes_per_step) cross it every step, so this is not a "
                            "kernel number"},
            # per step and method: draft kernel, verification kernel, walk kernel; in paper layout the
            # large-vocabulary bf16 path adds a kernel for the leaf rows
            "gpu_launches": (9 + (3 if args.layout == "paper" and cfg.dtype == "bf16" and cfg.vocab >= 8192
                                  and cfg.vocab % 8 == 0 else 0)) * args.steps,
            "clocks": clocks,
            "roofline": roof["spechub_verify_tree"],
            "kernels": roof,
            "special_function_pipe": {
                "note": ("3 ex2 per vocabulary pair per verified row (1 in pass A, over the target row; 2 in pass B); "
                         if hand_over else
                         "4 ex2 per vocabulary pair per verified row (2 in pass A, 2 in pass B); ")
                        + "B200 issues 16 ex2/clk/SM (measured)",
                "kernel": "spechub_verify_tree",
                "achieved_ex2_per_s": (3.0 if hand_over else 4.0) * B * (N - n_leaf) * V / (verify_ms * 1e-3),
                "peak_ex2_per_s": 148 * 16 * (clocks["sm_mhz"] or 1965.0) * 1e6,
            },
            "breakdown": {
                "spechub_only_step": {
                    "ms_per_step": call_ms["spechub_draft_sample"] + call_ms["spechub_verify_tree"],
                    "nodes_per_s": B * N * world / ((call_ms["spechub_draft_sample"]
                                                     + call_ms["spechub_verify_tree"]) * 1e-3),
                    "note": "spechub_draft_sample + spechub_verify_tree (verification and walk kernels) of the "
                            "timed steps: each node counted once"},
                "spechub_verify_nodes_per_s": B * N / (verify_ms * 1e-3),
                "spechub_verify_vocab_elements_per_s": B * N * V / (verify_ms * 1e-3),
                "step_vocab_elements_per_s": nodes_per_step * V * args.steps / (ms * 1e-3),
                "spechub_verify_without_probability_outputs": {
                    "ms_per_launch": lite_ms, "nodes_per_s": B * N / (lite_ms * 1e-3),
                    "note": "beta / rate not requested: rows whose first test accepts skip pass B; "
                            "not part of `value`"},
                "step_through_the_other_entry_points": {
                    "ms_per_step": other_ms, "nodes_per_s": len(METHODS) * B * N / (other_ms * 1e-3),
                    "note": ("the plain entry points (no hand-over of draft statistics)" if hand_over else
                             "the _stats entry points (draft statistics handed to verification)")
                            + "; this rank only; not part of `value`"},
                "step_as_cuda_graph": {
                    "ms_per_step": graph_ms,
                    "nodes_per_s": (len(METHODS) * B * N / (graph_ms * 1e-3)) if graph_ms else None,
                    "note": graph_note},
                "three_drafts_per_node": kary,
                "vocab_sharded_step": None if world == 1 else {"unavailable": vs_err} if not vs_ms else {
                    "ms_per_step": vs_ms, "nodes_per_s": B * N / (vs_ms * 1e-3), "ranks": world,
                    "nccl_version": ".".join(str(v) for v in torch.cuda.nccl.version()),
                    "note": "SpecHub draft + verify + walk of ONE batch of %d sequences whose vocabulary is sharded "
                            "over the ranks (strong scaling of one step); max over ranks; not part of `value`" % B},
                "step_through_three_method_calls": {
                    "ms_per_step": fused_ms, "nodes_per_s": len(METHODS) * B * N / (fused_ms * 1e-3),
                    "gpu_launches_per_step": 5,
                    "note": "mdsd_compare_draft_sample + mdsd_compare_verify_tree (their _stats forms with --draft-stats on): same outputs as the "
                            "nine launches of the timed step, bit for bit; this rank only; not part of `value`"},
            },
        }
        sfp = line["special_function_pipe"]
        sfp["frac"] = sfp["achieved_ex2_per_s"] / sfp["peak_ex2_per_s"]
        if not args.no_cpu_baseline and world == 1:
            v, desc, _ = oracle_sample(cfg, args.layout, args.cpu_seconds)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc}
            try:
                line["cpu_baseline_all_cores"] = oracle_all_cores(cfg, args.layout, v, args.cpu_seconds)
            except Exception as exc:   # reported, never fatal: the single-core baseline above stands
                line["cpu_baseline_all_cores"] = {"unavailable": str(exc).splitlines()[0][:160] if str(exc) else repr(exc)}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
