#!/usr/bin/env python
"""Benchmark of the DENSE sample + GraphSage forward hot path on synthetic paper-shaped graphs.

One step = one pass of the whole path (k-hop DENSE sampling, relabelling, feature gather +
segment-mean, linear layers) over one group of independent mini-batches through the C ABI.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2202_02365_b200 import inputs  # noqa: E402

CONFIGS = {
    # name: nodes, edges, graph kind, feature dim, hidden, fanouts, targets per mini-batch, partitions
    "config1_er_10k": dict(n=10_000, m=200_000, kind="er", dim=16, hidden=16, fanouts=[10, 5], batch=512, parts=1,
                           train=10_000),
    "config2_rmat_1m": dict(n=1_000_000, m=20_000_000, kind="rmat", dim=128, hidden=256, fanouts=[15, 10, 5],
                            batch=1000, parts=1, train=1_000_000),
    "config3_papers100m_shaped": dict(n=111_000_000, m=1_620_000_000, kind="rmat", dim=128, hidden=256,
                                      fanouts=[15, 10, 5], batch=1000, parts=16, train=1_100_000),
    # config 3's graph sampled from incoming AND outgoing edges, 15 / 10 / 5 neighbours per direction (the paper's
    # 30 / 20 / 10 over both directions, Section 7.1); mini-batches are ~20x larger, so a step takes 16 of them
    "config3_papers100m_shaped_inout": dict(n=111_000_000, m=1_620_000_000, kind="rmat", dim=128, hidden=256,
                                            fanouts=[15, 10, 5], batch=1000, parts=16, train=1_100_000, inout=True,
                                            group=16),
    # the setting of the paper's Table 6 at three layers: up to 10 incoming + 10 outgoing neighbours per node and layer
    # (the paper does not state its mini-batch size; 1,000 targets give mini-batches of its reported order, ~1M nodes)
    "table6_papers100m_shaped_3layers": dict(n=111_000_000, m=1_620_000_000, kind="rmat", dim=128, hidden=256,
                                             fanouts=[10, 10, 10], batch=1000, parts=16, train=1_100_000, inout=True,
                                             group=8),
    # a case small enough for ncu's counter passes whose feature table (4 GB) is still far larger than L2: the fused
    # layer-1 kernel's DRAM traffic per unit is captured here (profiles/k_sage_layer_fused_dram_traffic.md)
    "probe_rmat_8m_dim128": dict(n=8_000_000, m=160_000_000, kind="rmat", dim=128, hidden=256, fanouts=[15, 10, 5],
                                 batch=1000, parts=1, train=8_000_000),
    # the same idea for the fp16-operand variant of that kernel (half-precision rows of 1,536 bytes, 3 GB table)
    "probe_rmat_2m_fp16_768": dict(n=2_000_000, m=40_000_000, kind="rmat", dim=768, hidden=256, fanouts=[15, 10, 5],
                                   batch=1000, parts=1, train=2_000_000, fp16=True, group=32),
    # config 4's shapes at a tenth of its node count, whole fp16 table in HBM (no swaps): a throughput probe of the
    # wide fp16 layer-1 path, not the out-of-core configuration itself (that one is exercised by the tests)
    "config4_tenth_fp16_768_in_hbm": dict(n=12_200_000, m=130_000_000, kind="rmat", dim=768, hidden=256,
                                          fanouts=[15, 10, 5], batch=1000, parts=1, train=12_200_000, fp16=True),
}
# link prediction (config 5: Freebase86M-shaped), measured by run_lp: a step = one batch of 50,000 edges
LP_CONFIG = dict(n=86_000_000, m=338_000_000, dim=100, n_rel=14_824, parts=16, resident=8, edges=50_000, chunks=10,
                 negs=1000, fanout=20)
LP_WORKLOAD = "config5_freebase86m_shaped_lp"
# config 4 (Mag240M-Cites-shaped) out of core, measured by run_out_of_core: fp16 x 768 features in 32 partition blocks of
# 5.86 GB, a 10-partition HBM buffer, one block swapped in from pinned host memory per buffer state (side stream) while
# mini-batches run on the current state; the 187 GB table is never held: a block is a pure function of (seed, block)
OOC_CONFIG = dict(n=122_000_000, m=1_300_000_000, dim=768, hidden=256, fanouts=[15, 10, 5], batch=1000, parts=32, cap=10,
                  group=128, steps_per_state=25)
OOC_WORKLOAD = "config4_mag240m_shaped_out_of_core"
DEFAULT_WORKLOAD = "config3_papers100m_shaped"
HBM_NOMINAL_GBS = 8000.0
# DRAM traffic of the dominant kernel (fused layer 1) comes from a tracked ncu summary, not from a constant here: the
# summary gives, for a capture small enough for ncu's counter passes, DRAM bytes read per algorithmic byte and DRAM
# bytes written per output row; both scale with the units a launch processes
TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "k_sage_layer_fused_dram_traffic.md")


def traffic_model():
    """(dram read bytes per algorithmic byte, dram write bytes per output row, source) from the tracked summary."""
    import re
    try:
        text = open(TRAFFIC_PROFILE).read()
        r = re.search(r"dram_read_bytes_per_algorithmic_byte\s*[:=]\s*([0-9.]+)", text)
        w = re.search(r"dram_write_bytes_per_output_row\s*[:=]\s*([0-9.]+)", text)
        c = re.search(r"captured_at_commit\s*[:=]\s*([0-9a-f]+)", text)
        return float(r.group(1)), float(w.group(1)), f"profiles/k_sage_layer_fused_dram_traffic.md @ {c.group(1) if c else '?'}"
    except Exception:
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def build_workload(cfg, device, seed=0):
    t0 = time.time()
    if cfg["kind"] == "er":
        g = inputs.erdos_renyi_graph(cfg["n"], cfg["m"], seed, device)
    else:
        g = inputs.rmat_graph(cfg["n"], cfg["m"], seed, device)
    sync = torch.cuda.synchronize if torch.device(device).type == "cuda" else (lambda: None)
    sync()
    t1 = time.time()
    feats = inputs.normal_features(cfg["n"], cfg["dim"], seed + 1, device,
                                   dtype=torch.float16 if cfg.get("fp16") else torch.float32)
    sync()
    dims = [cfg["dim"]] + [cfg["hidden"]] * len(cfg["fanouts"])
    layers = inputs.glorot_layers(dims, seed + 2)
    return g, feats, layers, {"graph_s": round(t1 - t0, 1), "features_s": round(time.time() - t1, 1)}


def algorithmic_bytes(nodes, ents, cfg, feat_bytes=4):
    """Bytes the method must move for the sampled batches (per-unit figures of the scope table):
    sampling 12 E_s + 20 n_s + 4 V, features V d0 s, aggregation indices sum_l 4 (E_l + N_l),
    output n_k d_k 4.  nodes: [B, k+1] (hop 0 = targets), ents: [B, k]."""
    k = ents.shape[1]
    V = nodes.sum()
    n_s = nodes[:, :k].sum()
    E_s = ents.sum()
    a_s = 12 * E_s + 20 * n_s + 4 * V
    a_f = V * cfg["dim"] * feat_bytes
    a_i = 0
    for l in range(1, k + 1):                       # layer l aggregates hops 0 .. k-l
        a_i += 4 * (ents[:, :k - l + 1].sum() + nodes[:, :k - l + 1].sum())
    a_o = nodes[:, 0].sum() * cfg["hidden"] * 4
    flops = 0
    dims = [cfg["dim"]] + [cfg["hidden"]] * k
    for l in range(1, k + 1):
        flops += 2 * nodes[:, :k - l + 1].sum() * 2 * dims[l - 1] * dims[l]
    agg_l1 = a_f + 4 * (ents.sum() + nodes[:, :k].sum())
    flops_l1 = 2 * nodes[:, :k].sum() * 2 * dims[0] * dims[1]
    return {"sampling": int(a_s), "features": int(a_f), "agg_index": int(a_i), "output": int(a_o),
            "a_min": int(a_s + a_f + a_i + a_o), "flops": int(flops), "agg_l1": int(agg_l1), "flops_l1": int(flops_l1)}


_ORACLE_SHARED = {}


def _oracle_worker_init(folder, n_arrays, cfg, np_layers):
    """Runs once in every worker process: the graph arrays are memory-mapped from files the parent wrote (shared through
    the page cache), and the worker keeps to one core."""
    try:
        from threadpoolctl import threadpool_limits
        _ORACLE_SHARED["limit"] = threadpool_limits(1)   # the oracle's matmul must not spread over the other workers' cores
    except Exception:
        pass
    _ORACLE_SHARED.update(g_host=[np.load(os.path.join(folder, f"g{i}.npy"), mmap_mode="r") for i in range(n_arrays)],
                          cfg=cfg, np_layers=np_layers)


def _oracle_ready(_):
    return os.getpid()


def _oracle_sample(job):
    from oracle import dense_oracle as O
    tg, seed = job
    g_host, cfg = _ORACLE_SHARED["g_host"], _ORACLE_SHARED["cfg"]
    inout = len(g_host) > 2
    view = O.GraphView(g_host[0], g_host[1], out_row_offsets=g_host[2] if inout else None, out_nbrs=g_host[3] if inout else None)
    return O.sample_dense(view, tg, cfg["fanouts"], int(seed), "inout" if inout else "in")


def _oracle_forward(job):
    from oracle import dense_oracle as O
    ref, h0 = job
    O.forward(ref, h0, _ORACLE_SHARED["np_layers"])
    return len(ref["nbrs"])


def oracle_time(g_host, feats, layers, cfg, target_rows, seeds, limit_s=20.0, workers=None):
    """The CPU oracle as it stands on a bounded sample of the same mini-batches, one mini-batch per worker process
    over the host cores this job may use.  Rounds of `workers` mini-batches until the time limit: the workers sample
    (Algorithm 1), the parent hands each its H^0 rows (the feature table lives on the GPU), the workers run the layers.
    The workers are fresh processes (spawned, never forked from a process that holds a CUDA context); they map the graph
    arrays from files written once before the clock starts."""
    import multiprocessing as mp
    import shutil
    import tempfile
    cores = len(os.sched_getaffinity(0))
    workers = max(1, min(workers or cores, len(target_rows)))
    need = sum(int(a.nbytes) for a in g_host)
    base = "/dev/shm" if os.path.isdir("/dev/shm") and shutil.disk_usage("/dev/shm").free > 1.2 * need else None
    folder = tempfile.mkdtemp(prefix="mg_oracle_", dir=base)
    try:
        for i, a in enumerate(g_host):
            np.save(os.path.join(folder, f"g{i}.npy"), np.asarray(a))
        np_layers = [(w.numpy(), n.numpy(), b.numpy()) for w, n, b in layers]
        small_cfg = {"fanouts": list(cfg["fanouts"])}
        jobs = [(tg.tolist(), int(seed)) for tg, seed in zip(target_rows, seeds)]
        done, edges = 0, 0
        with mp.get_context("spawn").Pool(workers, initializer=_oracle_worker_init,
                                          initargs=(folder, len(g_host), small_cfg, np_layers)) as pool:
            pool.map(_oracle_ready, range(4 * workers), chunksize=1)      # every worker is up before the clock starts
            t0 = time.time()
            while done < len(jobs):
                chunk = jobs[done:done + workers]
                refs = pool.map(_oracle_sample, chunk, chunksize=1)
                h0s = [feats[torch.as_tensor(r["node_ids"], dtype=torch.int64).to(feats.device)].float().cpu().numpy() for r in refs]
                edges += sum(pool.map(_oracle_forward, list(zip(refs, h0s)), chunksize=1))
                done += len(chunk)
                if time.time() - t0 > limit_s:
                    break
            dt = time.time() - t0
    finally:
        shutil.rmtree(folder, ignore_errors=True)
    return {"batches": done, "seconds": dt, "batches_per_s": done / dt, "edges_per_s": edges / dt, "workers": workers,
            "cores_available": cores}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="mgdense", choices=["mgdense", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(CONFIGS) + [LP_WORKLOAD, OOC_WORKLOAD])
    ap.add_argument("--group", type=int, default=0, help="mini-batches per step (default: 128, or the workload's own)")
    ap.add_argument("--window", type=int, default=0, help="mini-batches per window of the layer schedule (0 = whole layers)")
    ap.add_argument("--lp-model", default="graphsage", choices=["graphsage", "gat"],
                    help="link-prediction workload only: the encoder layer (GraphSage mean or single-head graph attention)")
    ap.add_argument("--no-backward", action="store_true",
                    help="skip the timing of mg_backward on one group of mini-batches (reported beside the timed path, not in it)")
    ap.add_argument("--backward", action="store_true", help="(kept for old command lines: the backward pass is timed by default)")
    ap.add_argument("--steps-per-state", type=int, default=0,
                    help="out-of-core workload only: steps run on one buffer state while the next state's block loads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "mgdense" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    peaks = measured_peaks()
    if args.workload == OOC_WORKLOAD:
        if args.impl == "reference":
            if rank == 0:
                print(json.dumps({"impl": "reference", "unavailable": "the reference arm times the oracle on the default workload only"}))
            return
        run_out_of_core(args, peaks, rank, local_rank, world)
        return
    if args.workload == LP_WORKLOAD:
        if args.impl == "reference":
            if rank == 0:
                print(json.dumps({"impl": "reference", "unavailable": "the reference arm times the oracle on the default workload only"}))
            return
        run_lp(args, peaks, rank, local_rank, world)
        return
    cfg = CONFIGS[args.workload]

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, cfg)
        return

    import paper_2202_02365_b200 as mg
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    g, feats, layers, setup = build_workload(cfg, device, seed=0)
    ctx = mg.Context(local_rank)
    ctx.load_graph(g.row_offsets, g.nbrs)
    g_host = None
    if rank == 0 and not args.no_cpu_baseline:
        g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    n_edges = g.n_edges
    if cfg.get("inout"):
        gt = inputs.transpose_csr(g)
        ctx.load_out_graph(gt.row_offsets, gt.nbrs)
        ctx.set_sample_direction("inout")
        if g_host is not None:
            g_host = g_host + (gt.row_offsets.cpu().numpy(), gt.nbrs.cpu().numpy())
        del gt
    del g
    torch.cuda.empty_cache()
    if cfg["parts"] > 1:
        ctx.set_partitioning(cfg["parts"])
        ctx.load_features(feats, capacity_parts=cfg["parts"])
        ctx.set_resident(list(range(cfg["parts"])))
    else:
        ctx.load_features(feats)
    model = ctx.model(layers, mg.GEMM_TF32)
    dims_model = [cfg["dim"]] + [cfg["hidden"]] * len(cfg["fanouts"])
    ctx.set_layer_window(args.window)

    G, T, k = (args.group or cfg.get("group", 128)), cfg["batch"], len(cfg["fanouts"])
    n_steps_total = args.warmup + 2 * args.steps + 1
    # every rank draws its own mini-batches from the shuffled train set
    all_targets = inputs.train_set_batches(cfg["n"], cfg["train"], T, G * n_steps_total, seed=100 + rank)
    offs = torch.arange(0, G + 1, dtype=torch.int64) * T

    def step_targets(i):
        return all_targets[i * G:(i + 1) * G].reshape(-1)

    def step_seeds(i):
        return [(rank << 40) + i * G + b for b in range(G)]

    # capacities from a probe group (worst-case bounds would waste memory by ~10x)
    probe = ctx.sample_many(step_targets(0).to(device), offs, cfg["fanouts"], step_seeds(0),
                            caps=None if cfg["n"] < 2_000_000 else {"max_nodes_per_batch": 1 << (23 if cfg.get("inout") else 19)})
    nodes, ents = probe.counts()
    caps = {"max_nodes_total": int(nodes.sum() * 1.3) + 1024, "max_entries_total": int(ents.sum() * 1.3) + 1024,
            "max_nodes_per_batch": int(nodes.sum(1).max() * 1.5) + 64,
            "max_inner_nodes_per_batch": int(nodes[:, :-1].sum(1).max() * 1.5) + 64}
    probe.free()
    dense = ctx.sample_many(step_targets(0).to(device), offs, cfg["fanouts"], step_seeds(0), caps=caps)

    out_dev = torch.empty((G * T, cfg["hidden"]), dtype=torch.float32, device=device)
    out_host = torch.empty((G * T, cfg["hidden"]), dtype=torch.float32).pin_memory()
    dev_targets = [step_targets(i).to(device) for i in range(n_steps_total)]
    host_targets = [step_targets(i).pin_memory() for i in range(n_steps_total)]

    out_hosts = [out_host, torch.empty_like(out_host).pin_memory()]
    # three sample handles: two groups are always queued ahead of the one whose layers run, so that the GPU has
    # work while the host reads a finished sample's sizes and queues the next calls
    denses = [dense] + [ctx.sample_many(step_targets(0).to(device), offs, cfg["fanouts"], step_seeds(0), caps=caps)
                        for _ in range(2)]

    def begin(i, e2e):
        tg = host_targets[i] if e2e else dev_targets[i]
        ctx.sample_many_begin(tg, offs, cfg["fanouts"], step_seeds(i), caps=caps, out=denses[i % 3])

    def run_steps(first, count, e2e, export=False):
        """`count` steps, software-pipelined: groups i+1 and i+2 are sampled (sampling stream) while group i runs
        its layers (context stream); with e2e the host H^k of group i is copied out during group i+1; with export
        every group's DENSE is also laid out in the paper's canonical arrays (ascending ids inside each delta) for all
        of its mini-batches, on the sampling stream, before the next sample is queued there."""
        last = first + count
        begin(first, e2e)
        if first + 1 < last:
            begin(first + 1, e2e)
        for i in range(first, last):
            ctx.sample_many_end(denses[i % 3])
            if export:
                denses[i % 3].export_many()
            if i + 2 < last:
                begin(i + 2, e2e)
            if e2e:
                ctx.forward_host_async(model, denses[i % 3], out_hosts[i & 1])
            else:
                ctx.forward(model, denses[i % 3], out_dev)
        if e2e:
            ctx.wait_output()

    def run_step(i, e2e):
        run_steps(i, 1, e2e)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()

    for i in range(args.warmup):
        run_step(i, False)

    # ---- device-resident timing (no instrumentation inside the timed region) ----------------
    stats = {"nodes": [], "ents": []}
    launches0 = ctx.kernel_launches()
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    run_steps(args.warmup, args.steps, False)
    ev1.record()
    barrier()
    clocks = sampler.stop()
    ms_dev = ev0.elapsed_time(ev1)
    launches = ctx.kernel_launches() - launches0

    # ---- the same steps with the canonical export of every mini-batch inside the timed region -------------
    for i in range(2):
        run_steps(i, 1, False, export=True)      # allocates the export buffers
    barrier()
    ev4, ev5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev4.record()
    run_steps(args.warmup, args.steps, False, export=True)
    torch.cuda.synchronize()                     # the last export ends on the sampling stream
    ev5.record()
    barrier()
    ms_export = ev4.elapsed_time(ev5)

    # ---- the same steps with the intermediate layer outputs kept as fp16 (a model option; the headline keeps fp32) ----
    ms_f16 = None
    if all(w % 128 == 0 for w in dims_model[1:-1]) and k > 1:
        model16 = ctx.model(layers, mg.GEMM_TF32)
        model16.set_intermediates(torch.float16)
        model_main, model = model, model16
        for i in range(3):
            run_steps(i, 1, False)
        barrier()
        ev6, ev7 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev6.record()
        run_steps(args.warmup, args.steps, False)
        ev7.record()
        barrier()
        ms_f16 = ev6.elapsed_time(ev7)
        ctx.profile(True)
        ctx.profile_read(reset=True)
        for s_ in range(min(args.steps, 8)):
            run_step(args.warmup + s_, False)
        phases16 = ctx.profile_read(reset=True)
        ctx.profile(False)
        phases16 = {name: round(v["ms"] / min(args.steps, 8), 4) for name, v in phases16.items() if v["launches"] and name.startswith("aggregate")}
        model = model_main

    # ---- the same steps again with per-phase CUDA events on the library's stream ---------------
    ctx.profile(True)
    ctx.profile_read(reset=True)
    for s in range(args.steps):          # one group at a time here, so that the phase events do not overlap
        run_step(args.warmup + s, False)
        denses[(args.warmup + s) % 3].export_many()      # its kernels are the "sample_sort" phase
        n_, e_ = denses[(args.warmup + s) % 3].counts()
        stats["nodes"].append(n_); stats["ents"].append(e_)
    phases = ctx.profile_read(reset=True)
    ctx.profile(False)

    # ---- end to end: host targets in, host H^k out --------------------------------------
    barrier()
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record()
    run_steps(args.warmup + args.steps, args.steps, True)      # ends with the last H^k on the host
    ev3.record()
    barrier()
    ms_e2e = ev2.elapsed_time(ev3)

    # ---- latency of a single mini-batch (sample + all layers, device-resident, one call after the other) ----
    lat_dense = None
    lat_out = torch.empty((T, cfg["hidden"]), dtype=torch.float32, device=device)
    lat_targets = dev_targets[0][:T].contiguous()
    lat_ms = []
    for rep in range(3 + 20):
        torch.cuda.synchronize()
        t_lat = time.perf_counter()
        lat_dense = ctx.sample(lat_targets, cfg["fanouts"], seed=rep, out=lat_dense)
        ctx.forward(model, lat_dense, lat_out)      # synchronous: returns when H^k is in lat_out
        if rep >= 3:
            lat_ms.append((time.perf_counter() - t_lat) * 1e3)
    single_batch_latency_ms = float(np.median(lat_ms))

    # ---- the backward pass of one group (reported beside the timed path, not part of it) ----
    # gradients of the weights and biases alone (fixed features: node classification), and with the gradient of every
    # base-representation row as well (learnable base representations)
    backward_ms = backward_h0_ms = None
    if not args.no_backward:
        ctx.keep_layer_outputs(True)
        g_out = torch.randn_like(out_dev)
        for want_h0 in (False, True):
            bw = []
            for rep in range(4):
                ctx.forward(model, denses[0], out_dev)
                torch.cuda.synchronize()
                t_bw = time.perf_counter()
                res = ctx.backward(model, denses[0], g_out, want_h0_grad=want_h0)
                torch.cuda.synchronize()
                if rep:
                    bw.append((time.perf_counter() - t_bw) * 1e3)
                del res
            if want_h0:
                backward_h0_ms = float(np.median(bw))
            else:
                backward_ms = float(np.median(bw))
        del g_out
        ctx.keep_layer_outputs(False)

    if world > 1:
        t = torch.tensor([ms_dev, ms_e2e, ms_export], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_dev, ms_e2e, ms_export = float(t[0]), float(t[1]), float(t[2])

    nodes = torch.cat(stats["nodes"]).numpy()
    ents = torch.cat(stats["ents"]).numpy()
    alg = algorithmic_bytes(nodes, ents, cfg, feat_bytes=2 if cfg.get("fp16") else 4)
    n_batches = args.steps * G * world
    value = n_batches / (ms_dev / 1e3)
    e2e_value = n_batches / (ms_e2e / 1e3)
    sampled_edges = float(ents.sum()) * world

    # ---- rooflines (CUDA-event times of the library's own kernels, second pass) -----------------
    # The dominant kernel is the fused layer-1 kernel (k_sage_layer_fused<first>): it gathers the base
    # representations (the bulk of A_min), reduces them and runs the layer's GEMM on the tensor cores.
    # It is HBM-bound: achieved = its algorithmic bytes (V d0 s + 4 (E_1 + N_1)) over its event time.
    export_ms = phases["sample_sort"]["ms"]          # mg_dense_export_many's kernels; not part of sample_ms / path_hbm
    sample_ms = sum(v["ms"] for name, v in phases.items() if name.startswith("sample_") and name != "sample_sort")
    agg1 = phases["aggregate_l1"]
    rest = phases["aggregate_rest"]
    gemm = phases["gemm"]
    tf32_peak = peaks["bf16_tflops_sustained"] * 0.5     # nominal TF32 : bf16 dense ratio is 1 : 2
    fused = gemm["launches"] == 0
    n_l1 = max(1, agg1["launches"])
    roofline = {"kernel": "k_sage_layer_fused<layer 1> (feature gather + segment mean + tcgen05 TF32 GEMM)" if fused
                else "k_aggregate<layer 1> (feature gather + segment mean)",
                "bound": "hbm", "achieved": alg["agg_l1"] / (agg1["ms"] / 1e3) / 1e9 if agg1["ms"] else None,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "bytes_per_launch": alg["agg_l1"] / n_l1,
                "ms_per_launch": agg1["ms"] / n_l1, "launches": agg1["launches"], "peak_source": peaks["source"]}
    roofline["frac"] = roofline["achieved"] / roofline["peak"] if roofline["achieved"] else None
    # dram__bytes_read.sum + dram__bytes_write.sum per launch: the ncu capture of a smaller case of the same kernel
    # (feature table of a few GB, far above L2), scaled by the units this launch processes (fp32 x 128 features only)
    rows_out_l1 = float(nodes[:, :k].sum()) / n_l1
    roofline["rows_out_per_launch"] = rows_out_l1
    tm = traffic_model()
    if tm and cfg["dim"] == 128 and not cfg.get("fp16"):
        roofline["traffic"] = tm[0] * roofline["bytes_per_launch"] + tm[1] * rows_out_l1
        roofline["traffic_source"] = tm[2]
    else:
        roofline["traffic"] = None
    flops_l1 = alg["flops_l1"]
    tensor = {"what": "layer GEMM work inside the fused kernels (all layers)", "bound": "tensor",
              "achieved": alg["flops"] / ((agg1["ms"] + rest["ms"] + gemm["ms"]) / 1e3) / 1e12, "peak": tf32_peak,
              "unit": "TFLOP/s", "layer1_tflops": flops_l1 / (agg1["ms"] / 1e3) / 1e12 if agg1["ms"] else None}
    tensor["frac"] = tensor["achieved"] / tensor["peak"]
    mem_ms = sample_ms + agg1["ms"] + rest["ms"] + phases.get("other", {"ms": 0.0})["ms"]   # "other": the layers' row pre-pass
    path_gbs = alg["a_min"] / (mem_ms / 1e3) / 1e9 if mem_ms else None

    line = {
        "metric": "DENSE sample+aggregate mini-batches/s", "value": value, "unit": "mini-batches/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_dev / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 (TF32 tensor-core GEMM)",
        "data": "synthetic",
        "config": {"workload": args.workload, "nodes": cfg["n"], "edges": n_edges, "feature_dim": cfg["dim"],
                   "hidden": cfg["hidden"], "fanouts": cfg["fanouts"], "targets_per_batch": T,
                   "mini_batches_per_step": G, "partitions": cfg["parts"], "resident": cfg["parts"],
                   "l2": "inputs larger than L2 (feature table and CSR far exceed 126 MB; no flush)",
                   "setup_s": setup},
        "sampled_edges_per_s": sampled_edges / (ms_dev / 1e3),
        # the same steps with mg_dense_export_many for every group inside the timed region: the paper's arrays
        # (ascending ids inside each delta, repr_map in those rows) for all mini-batches of the group
        "value_with_canonical_export": n_batches / (ms_export / 1e3),
        "ms_per_step_with_canonical_export": ms_export / args.steps,
        "export_ms_per_step": export_ms / args.steps,
        # the same steps with H^1 .. H^{k-1} stored as fp16 (mg_model_set_intermediates; the same 10-bit mantissa the
        # TF32 layers round their inputs to): half the bytes and half the row requests between the layers
        "value_fp16_intermediates": (n_batches / (ms_f16 / 1e3)) if ms_f16 else None,
        "ms_per_step_fp16_intermediates": (ms_f16 / args.steps) if ms_f16 else None,
        "layer_phases_ms_per_step_fp16_intermediates": phases16 if ms_f16 else None,
        "per_batch": {"nodes": float(nodes.sum(1).mean()), "sampled_edges": float(ents.sum(1).mean()),
                      "algorithmic_bytes": alg["a_min"] / (args.steps * G),
                      "gemm_flops": alg["flops"] / (args.steps * G)},
        "e2e": {"value": e2e_value, "unit": "mini-batches/s", "h2d_bytes_per_step": int(G * T * 4),
                "d2h_bytes_per_step": int(G * T * cfg["hidden"] * 4), "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "single_batch_latency_ms": single_batch_latency_ms,
        "backward_ms_per_group": backward_ms,
        "backward_with_base_gradients_ms_per_group": backward_h0_ms,
        "clocks": clocks,
        "roofline": roofline,
        "tensor": tensor,
        "path_hbm": {"what": "A_min over the time of all sampling and layer kernels (the layer GEMMs run inside them)",
                     "achieved_gbs": path_gbs, "frac_of_measured": path_gbs / peaks["hbm_gbs"] if path_gbs else None,
                     "frac_of_8tbs": path_gbs / HBM_NOMINAL_GBS if path_gbs else None, "kernel_ms": mem_ms},
        "phases_ms_per_step": {name: round(v["ms"] / args.steps, 4) for name, v in phases.items() if v["launches"]},
    }
    if rank == 0:
        if g_host is not None:
            r = oracle_time(g_host, feats, layers, cfg, all_targets[args.warmup * G:], step_seeds(args.warmup),
                            limit_s=args.cpu_seconds)
            line["cpu_baseline"] = {"value": r["batches_per_s"], "unit": "mini-batches/s", "cores": r["workers"], "kind": "oracle",
                                    "sample": f"{r['batches']} mini-batches of the timed workload in {r['seconds']:.1f} s, one "
                                              f"mini-batch per worker process ({r['cores_available']} cores available to the job)",
                                    "sampled_edges_per_s": r["edges_per_s"]}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()



def run_out_of_core(args, peaks, rank, local_rank, world):
    """Config 4 as stated: R-MAT 122M nodes / 1.30B edges, fp16 features of width 768, 32 partitions, a 10-partition
    buffer in HBM.  Buffer states follow the random one-swap order (Section 5.2's fallback); while the mini-batches of
    a state run (sampling restricted to resident endpoints, three fused layers), the next state's incoming block is
    copied from a pinned host block on the side stream, then committed (slot map + in-buffer view of the graph).
    The timed region of a state = queueing the swap, its steps, and the commit; the incoming block is made in host
    memory before the region starts (it stands in for the table that is already there)."""
    import paper_2202_02365_b200 as mg
    c = OOC_CONFIG
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    t0 = time.time()
    g = inputs.rmat_graph(c["n"], c["m"], seed=40, device=device)
    n_edges = g.n_edges
    ctx = mg.Context(local_rank)
    ctx.load_graph(g.row_offsets, g.nbrs)
    del g
    torch.cuda.empty_cache()
    P, cap, dim, T, k = c["parts"], c["cap"], c["dim"], c["batch"], len(c["fanouts"])
    G = args.group or c["group"]
    S = args.steps_per_state or c["steps_per_state"]
    ctx.set_partitioning(P)
    ctx.load_features(None, capacity_parts=cap, backing=mg.BACKING_HOST, dtype=torch.float16, dim=dim)
    part_rows = inputs.contiguous_partition(c["n"], P)
    rows_of = lambda p: min(part_rows, c["n"] - p * part_rows)
    staging = [torch.empty((part_rows, dim), dtype=torch.float16).pin_memory() for _ in range(2)]
    feat_seed = 41 + 1000 * rank

    def stage(p, slot):
        inputs.block_features(rows_of(p), dim, feat_seed, p, device=device, dtype=torch.float16, out=staging[slot][:rows_of(p)])
        torch.cuda.synchronize()
        return staging[slot]

    states = inputs.swap_order(P, cap, seed=44 + rank)
    for i, p in enumerate(states[0]):                # fill the buffer, one block at a time through one staging block
        ctx.set_partition_source(p, stage(p, 0))
        ctx.set_resident(sorted(states[0][:i + 1]))
    layers = inputs.glorot_layers([dim] + [c["hidden"]] * k, seed=43)
    model = ctx.model(layers, mg.GEMM_TF32)
    setup_s = round(time.time() - t0, 1)
    offs = torch.arange(0, G + 1, dtype=torch.int64) * T
    n_states = max(1, min(len(states) - 1, (args.warmup + args.steps + S - 1) // S + 1))

    def state_targets(state, n_steps, seed):
        mask = inputs.resident_node_mask(c["n"], P, state, device=device)
        pool = torch.nonzero(mask).flatten().to(torch.int32)
        gen = torch.Generator(device=device); gen.manual_seed(seed)
        pick = torch.randperm(pool.numel(), generator=gen, device=device)[:n_steps * G * T]
        return pool[pick].reshape(n_steps, G * T).contiguous()

    tg0 = state_targets(states[0], 1, 7)
    seeds0 = [(rank << 40) + b for b in range(G)]
    probe = ctx.sample_many(tg0[0], offs, c["fanouts"], seeds0, caps={"max_nodes_per_batch": 1 << 19})
    nodes, ents = probe.counts()
    caps = {"max_nodes_total": int(nodes.sum() * 1.4) + 1024, "max_entries_total": int(ents.sum() * 1.4) + 1024,
            "max_nodes_per_batch": int(nodes.sum(1).max() * 1.6) + 64,
            "max_inner_nodes_per_batch": int(nodes[:, :-1].sum(1).max() * 1.6) + 64}
    probe.free()
    denses = [ctx.sample_many(tg0[0], offs, c["fanouts"], seeds0, caps=caps) for _ in range(3)]
    out_dev = torch.empty((G * T, c["hidden"]), dtype=torch.float32, device=device)
    out_hosts = [torch.empty((G * T, c["hidden"]), dtype=torch.float32).pin_memory() for _ in range(2)]

    def run_steps(tg, base_seed, e2e):
        """tg: one row of G x T targets per step (device rows, or pinned host rows with e2e)"""
        n = len(tg)
        src = list(tg)
        seeds = lambda i: [(rank << 40) + base_seed + i * G + b for b in range(G)]
        begin = lambda i: ctx.sample_many_begin(src[i], offs, c["fanouts"], seeds(i), caps=caps, out=denses[i % 3])
        begin(0)
        if n > 1:
            begin(1)
        for i in range(n):
            ctx.sample_many_end(denses[i % 3])
            if i + 2 < n:
                begin(i + 2)
            if e2e:
                ctx.forward_host_async(model, denses[i % 3], out_hosts[i & 1])
            else:
                ctx.forward(model, denses[i % 3], out_dev)
        if e2e:
            ctx.wait_output()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()

    # a swap with nothing else running, and a commit whose copies have long finished (slot map + view rebuild alone)
    incoming = lambda s: [p for p in states[s + 1] if p not in states[s]][0]
    swap_alone_ms = rebuild_alone_ms = None
    cur = 0
    run_steps(state_targets(states[0], max(args.warmup, 3), 8), 1 << 20, False)       # warm-up steps
    ctx.set_partition_source(incoming(0), stage(incoming(0), 1))
    barrier()
    t1 = time.perf_counter()
    ctx.set_resident(states[1], async_=True)
    ctx.commit_resident(120_000)
    torch.cuda.synchronize()
    swap_and_rebuild_ms = (time.perf_counter() - t1) * 1e3
    cur = 1
    # timed states
    sampler = ClockSampler(local_rank)
    launches0 = ctx.kernel_launches()
    seg_ms, commit_ms, done_steps, stats = [], [], 0, {"nodes": [], "ents": []}
    e2e_ms, e2e_steps = 0.0, 0
    sampler.start()
    while done_steps < args.steps and cur + 1 < len(states):
        n_here = min(S, args.steps - done_steps)
        tg = state_targets(states[cur], n_here, 100 + cur)
        q = incoming(cur)
        ctx.set_partition_source(q, stage(q, cur & 1))
        barrier()
        t1 = time.perf_counter()
        ctx.set_resident(states[cur + 1], async_=True)       # the incoming block starts loading on the side stream
        run_steps(tg, cur * 100_000, False)
        ev_steps = torch.cuda.Event()
        ev_steps.record()
        ev_steps.synchronize()                                # the steps are done; the copy on the side stream may not be
        t2 = time.perf_counter()
        ctx.commit_resident(120_000)                          # waits for what is left of the copy, flips the map, rebuilds the view
        torch.cuda.synchronize()
        t3 = time.perf_counter()
        barrier()
        seg_ms.append((t3 - t1) * 1e3)
        commit_ms.append((t3 - t2) * 1e3)
        done_steps += n_here
        cur += 1
    clocks = sampler.stop()
    launches = ctx.kernel_launches() - launches0
    # the same without a swap in flight: steps alone on the current state (also the phase profile), then end to end
    tg = state_targets(states[cur], min(S, args.steps), 999)
    barrier()
    t1 = time.perf_counter()
    run_steps(tg, 7 << 20, False)
    torch.cuda.synchronize()
    steps_alone_ms = (time.perf_counter() - t1) * 1e3 / tg.shape[0]
    ctx.profile(True)
    ctx.profile_read(reset=True)
    for i in range(tg.shape[0]):
        run_steps(tg[i:i + 1], (8 << 20) + i * G, False)
        n_, e_ = denses[0].counts()
        stats["nodes"].append(n_); stats["ents"].append(e_)
    phases = ctx.profile_read(reset=True)
    ctx.profile(False)
    tg_host = [t.cpu().pin_memory() for t in tg]
    barrier()
    t1 = time.perf_counter()
    run_steps(tg_host, 9 << 20, True)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t1) * 1e3 / len(tg_host)
    # a commit with its copy already complete: slot map + view rebuild alone
    if cur + 1 < len(states):
        q = incoming(cur)
        ctx.set_partition_source(q, stage(q, cur & 1))
        ctx.set_resident(states[cur + 1], async_=True)
        time.sleep(1.0)
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        ctx.commit_resident(120_000)
        torch.cuda.synchronize()
        rebuild_alone_ms = (time.perf_counter() - t1) * 1e3
        swap_alone_ms = swap_and_rebuild_ms - rebuild_alone_ms
    total_ms = float(sum(seg_ms))
    if world > 1:
        tt = torch.tensor([total_ms], device=device, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt[0])
    nodes = torch.cat(stats["nodes"]).numpy()
    ents = torch.cat(stats["ents"]).numpy()
    cfg_like = {"dim": dim, "hidden": c["hidden"]}
    alg = algorithmic_bytes(nodes, ents, cfg_like, feat_bytes=2)
    n_prof = tg.shape[0]
    agg1, rest = phases["aggregate_l1"], phases["aggregate_rest"]
    sample_ms = sum(v["ms"] for name, v in phases.items() if name.startswith("sample_"))
    block_bytes = rows_of(0) * dim * 2
    exposed = [max(0.0, cm - (rebuild_alone_ms or 0.0)) for cm in commit_ms]
    tf32_peak = peaks["bf16_tflops_sustained"] * 0.5
    line = {
        "metric": "DENSE sample+aggregate mini-batches/s", "value": done_steps * G * world / (total_ms / 1e3), "unit": "mini-batches/s",
        "n_gpus": world, "steps": done_steps, "warmup": args.warmup, "ms_per_step": total_ms / max(1, done_steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 (fp16 features, TF32 tensor-core GEMM)",
        "data": "synthetic",
        "config": {"workload": OOC_WORKLOAD, "nodes": c["n"], "edges": n_edges, "feature_dim": dim, "feature_dtype": "fp16",
                   "hidden": c["hidden"], "fanouts": c["fanouts"], "targets_per_batch": T, "mini_batches_per_step": G,
                   "partitions": P, "resident": cap, "steps_per_buffer_state": S, "buffer_states_timed": len(seg_ms),
                   "timed_region": "per buffer state: queue the swap of one 5.86 GB block from pinned host memory, run the state's "
                                   "steps, commit (wait for the copy, slot map, in-buffer view); summed over the states",
                   "l2": "inputs larger than L2 (58.6 GB of resident feature blocks; no flush)", "setup_s": setup_s},
        "sampled_edges_per_s": float(ents.sum()) / n_prof * done_steps * world / (total_ms / 1e3),
        "per_batch": {"nodes": float(nodes.sum(1).mean()), "sampled_edges": float(ents.sum(1).mean()),
                      "algorithmic_bytes": alg["a_min"] / (n_prof * G)},
        "swap": {"block_bytes": block_bytes, "swap_alone_ms": swap_alone_ms, "rebuild_alone_ms": rebuild_alone_ms,
                 "h2d_gbs_alone": block_bytes / (swap_alone_ms / 1e3) / 1e9 if swap_alone_ms else None,
                 "commit_ms_per_state": commit_ms, "exposed_swap_ms_per_state": exposed,
                 "fraction_of_swap_hidden": (1.0 - float(np.mean(exposed)) / swap_alone_ms) if swap_alone_ms else None,
                 "ms_per_step_without_a_swap_in_flight": steps_alone_ms},
        "e2e": {"value": G * world / (e2e_ms / 1e3), "unit": "mini-batches/s", "h2d_bytes_per_step": int(G * T * 4),
                "d2h_bytes_per_step": int(G * T * c["hidden"] * 4), "ms_per_step": e2e_ms,
                "note": "host targets in, host H^k out, no swap in flight"},
        "gpu_launches": int(launches), "clocks": clocks,
        "roofline": {"kernel": "k_sage_layer_fused<layer 1, fp16 features> (feature gather + segment mean + tcgen05 TF32 GEMM)",
                     "bound": "hbm", "achieved": alg["agg_l1"] / (agg1["ms"] / 1e3) / 1e9 if agg1["ms"] else None,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "bytes_per_launch": alg["agg_l1"] / max(1, agg1["launches"]),
                     "ms_per_launch": agg1["ms"] / max(1, agg1["launches"]), "peak_source": peaks["source"], "traffic": None},
        "tensor": {"bound": "tensor", "achieved": alg["flops"] / ((agg1["ms"] + rest["ms"]) / 1e3) / 1e12, "peak": tf32_peak, "unit": "TFLOP/s",
                   "layer1_tflops": alg["flops_l1"] / (agg1["ms"] / 1e3) / 1e12 if agg1["ms"] else None},
        "phases_ms_per_step": {name: round(v["ms"] / n_prof, 4) for name, v in phases.items() if v["launches"]},
    }
    if line["roofline"]["achieved"]:
        line["roofline"]["frac"] = line["roofline"]["achieved"] / peaks["hbm_gbs"]
    line["tensor"]["frac"] = line["tensor"]["achieved"] / tf32_peak
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_lp(args, peaks, rank, local_rank, world):
    """Link-prediction step at config 5's sizes: negatives + target union (mg_lp_prepare), a one-hop DENSE sample with
    fanout 20, one GraphSage layer 100 -> 100, DistMult scores of the positives and of both corrupted sides."""
    import paper_2202_02365_b200 as mg
    c = LP_CONFIG
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    t0 = time.time()
    g = inputs.rmat_graph(c["n"], c["m"], seed=5, device=device, n_relations=c["n_rel"])
    emb = inputs.normal_features(c["n"], c["dim"], seed=3, device=device, std=0.001)
    rel_emb = inputs.normal_features(c["n_rel"], c["dim"], seed=9, device=device)
    setup_s = round(time.time() - t0, 1)
    ctx = mg.Context(local_rank)
    ctx.load_graph(g.row_offsets, g.nbrs)
    ctx.set_partitioning(c["parts"])
    ctx.load_features(emb, capacity_parts=c["resident"])
    resident = [0, 2, 3, 5, 8, 9, 12, 15]
    ctx.set_resident(resident)
    mask = inputs.resident_node_mask(c["n"], c["parts"], resident)
    n_total = args.warmup + 2 * args.steps
    batches = [inputs.lp_edges(g, mask, c["edges"], seed=1000 * rank + i) for i in range(n_total)]
    n_edges_graph = g.n_edges
    del g, mask
    torch.cuda.empty_cache()
    layers = inputs.glorot_layers([c["dim"], c["dim"]], seed=8)
    model = ctx.model(layers, mg.GEMM_TF32)
    gat = None
    if args.lp_model == "gat":
        gen = torch.Generator().manual_seed(9)
        w = layers[0][0]
        gat = ctx.gat_model([(w, torch.randn(c["dim"], generator=gen) * 0.1, torch.randn(c["dim"], generator=gen) * 0.1,
                              torch.zeros(c["dim"]))], mg.GEMM_TF32)
    dense = None
    h = None
    stats = {"targets": [], "entries": []}

    def step(i, record=False):
        nonlocal dense, h
        src, rel, dst = batches[i]
        lp = ctx.lp_prepare(src, rel, dst, c["chunks"], c["negs"], seed=77 + i)
        targets = lp.targets()
        dense = ctx.sample(targets, [c["fanout"]], seed=i, out=dense)
        if h is None or h.shape[0] < targets.numel():
            h = torch.empty((int(targets.numel() * 1.2) + 16, c["dim"]), dtype=torch.float32, device=device)
        if gat is not None:
            ctx.gat_forward(gat, dense, h[:targets.numel()])
        else:
            ctx.forward(model, dense, h[:targets.numel()])
        scores = ctx.distmult_score(lp, h[:targets.numel()], rel_emb)
        if record:
            n_, e_ = dense.counts()
            stats["targets"].append(int(targets.numel())); stats["entries"].append(int(e_.sum()))
        lp.free()
        return scores

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()

    for i in range(args.warmup):
        step(i)
    sampler = ClockSampler(local_rank)
    launches0 = ctx.kernel_launches()
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(args.warmup, args.warmup + args.steps):
        step(i)
    ev1.record()
    barrier()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    launches = ctx.kernel_launches() - launches0
    # the same steps with the library's phase events: DistMult kernel time
    ctx.profile(True)
    ctx.profile_read(reset=True)
    for i in range(args.warmup + args.steps, args.warmup + 2 * args.steps):
        step(i, record=True)
    phases = ctx.profile_read(reset=True)
    ctx.profile(False)
    if world > 1:
        tt = torch.tensor([ms], device=device, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms = float(tt[0])
    B, negs, dim = c["edges"], c["negs"], c["dim"]
    dm_ms = phases["distmult"]["ms"] / args.steps
    score_bytes = 4.0 * B * (1 + 2 * negs)                       # compulsory score writes, both corrupted sides
    operand_bytes = 4.0 * (3 * B * dim + 2 * c["chunks"] * negs * dim)
    flops = 2.0 * B * negs * dim * 2 + 3.0 * B * dim
    line = {
        "metric": "link-prediction steps/s (negatives + DENSE sample + GraphSage layer + DistMult, 50,000 edges per step)",
        "value": args.steps * world / (ms / 1e3), "unit": "steps/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 (TF32 tensor-core GEMM)", "data": "synthetic",
        "config": {"workload": LP_WORKLOAD, "nodes": c["n"], "edges": n_edges_graph, "embedding_dim": dim,
                   "relations": c["n_rel"], "partitions": c["parts"], "resident": len(resident), "edges_per_step": B,
                   "chunks": c["chunks"], "negatives_per_chunk": negs, "fanouts": [c["fanout"]], "encoder": args.lp_model,
                   "l2": "inputs larger than L2 (embedding table 34 GB, scores 400 MB per step; no flush)",
                   "setup_s": {"graph_and_embeddings_s": setup_s}},
        "scored_pairs_per_s": args.steps * world * B * (1 + 2 * negs) / (ms / 1e3),
        "per_step": {"targets": float(np.mean(stats["targets"])), "sampled_edges": float(np.mean(stats["entries"]))},
        "gpu_launches": int(launches), "clocks": clocks,
        "roofline": {"kernel": "k_distmult_neg_tc (both corrupted sides) + k_distmult_pos", "bound": "hbm",
                     "achieved": (score_bytes + operand_bytes) / (dm_ms / 1e3) / 1e9 if dm_ms else None,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "bytes_per_step": score_bytes + operand_bytes,
                     "ms_per_step": dm_ms, "peak_source": peaks["source"], "traffic": None,
                     "tensor_tflops": flops / (dm_ms / 1e3) / 1e12 if dm_ms else None},
        "phases_ms_per_step": {k2: round(v2["ms"] / args.steps, 4) for k2, v2 in phases.items() if v2["ms"] > 0},
    }
    if line["roofline"]["achieved"]:
        line["roofline"]["frac"] = line["roofline"]["achieved"] / peaks["hbm_gbs"]
    if rank == 0:
        print(json.dumps(line))


def run_reference(args, cfg):
    """The CPU oracle on the host cores: a bounded sample of the same workload per step."""
    from oracle import dense_oracle as O  # noqa: F401
    device = torch.device("cuda", 0) if torch.cuda.is_available() else torch.device("cpu")
    g, feats, layers, _ = build_workload(cfg, device, seed=0)
    g_host = (g.row_offsets.cpu().numpy(), g.nbrs.cpu().numpy())
    n_edges = g.n_edges
    if cfg.get("inout"):
        gt = inputs.transpose_csr(g)
        g_host = g_host + (gt.row_offsets.cpu().numpy(), gt.nbrs.cpu().numpy())
        del gt
    del g
    cores = len(os.sched_getaffinity(0))
    per_step = cores                      # a step = one round of mini-batches, one per host core
    total = (args.warmup + args.steps) * per_step
    targets = inputs.train_set_batches(cfg["n"], cfg["train"], cfg["batch"], max(total, 1), seed=100)
    seeds = list(range(total))
    nw = args.warmup * per_step
    if nw:
        oracle_time(g_host, feats, layers, cfg, targets[:nw], seeds[:nw], limit_s=1e9)
    r = oracle_time(g_host, feats, layers, cfg, targets[nw:], seeds[nw:], limit_s=1e9)
    line = {
        "impl": "reference", "metric": "DENSE sample+aggregate mini-batches/s", "value": r["batches_per_s"],
        "unit": "mini-batches/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": r["seconds"] / max(1, args.steps) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "nodes": cfg["n"], "edges": n_edges, "feature_dim": cfg["dim"],
                   "hidden": cfg["hidden"], "fanouts": cfg["fanouts"], "targets_per_batch": cfg["batch"],
                   "mini_batches_per_step": per_step},
        "cpu_baseline": {"value": r["batches_per_s"], "unit": "mini-batches/s", "cores": r["workers"], "kind": "oracle",
                         "sample": f"{per_step} mini-batches per step (one per worker process), {args.steps} steps"},
        "e2e": {"value": r["batches_per_s"], "unit": "mini-batches/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "sampled_edges_per_s": r["edges_per_s"],
    }
    print(json.dumps(line))


if __name__ == "__main__":
    main()
