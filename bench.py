#!/usr/bin/env python
"""Benchmark of one-pass token-tree verification (mask slice -> tree attention over all layers -> accept/reject).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step = one verification pass of the whole path over one batch of the synthetic workload: the tree
attention of every layer (independent, seeded KV caches resident in HBM) followed by the accept/reject
walk.  The mask is built once before the timed region (the paper builds it at initialisation, Section 3.2)
and sliced per sequence by a row count.  The default workload is the long-context one (batch 16, 32 heads
x 128, 4096-token prefix, tree (1; 4,2,2,1), 32 layers).  With N > 1 (torchrun) every rank verifies its own
batch of the same size (weak scaling, no data-path collective).

`--impl reference` times the CPU oracle (fp64, numpy) on a bounded sample of the same workload.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree_verify_tree_tokens_per_s"
UNIT = "tree-tokens/s"
NOMINAL_HBM_GBS = 8000.0


def _traffic_for(w):
    """DRAM bytes per launch of the attention kernel from the tracked ncu capture (profiles/attention_traffic.json:
    dram__bytes_read.sum + dram__bytes_write.sum on a small batch; traffic grows in proportion to the batch).  The
    figure only holds for the kernel sources it was taken on: None once they have changed."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "attention_traffic.json")) as f:
            cap = json.load(f)
        h = hashlib.sha1()
        for name in cap["sources"]:
            with open(os.path.join(ROOT, "paper_2409_10644_b200", "csrc", name), "rb") as f:
                h.update(f.read())
    except (OSError, KeyError, ValueError):
        return None
    if h.hexdigest()[:12] != cap.get("source_sha1_12") or w.name != cap.get("workload"):
        return None
    return int(cap["bytes_per_launch"] * w.B / cap["batch"])


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except Exception:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _algorithmic_bytes_attention(H, D, lens, n_act, words, elt):
    """Bytes one tree-attention call must move: K and V rows of prefix and tree, Q read, O write, mask words."""
    kv = sum(H * (int(l) + int(n)) * D * 2 * elt for l, n in zip(lens, n_act))
    qo = sum(H * int(n) * D * 2 * elt for n in n_act)
    return kv + qo + sum(int(n) * words * 8 for n in n_act)


# ------------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample (reported baseline; also the `--impl reference` arm)
# ------------------------------------------------------------------------------------------------

_ORACLE_POOL = {}


def oracle_sample(w, budget_s=12.0, min_pairs=8):
    """Times the oracle, as it stands, on (sequence, head) attention problems and on verify sequences of
    workload `w`, and extrapolates to a full step.  Returns (tree-tokens/s, description, threads)."""
    import torch
    from mcsd_inputs import attention_inputs, gammas, parent_array, seq_lens, verify_inputs
    from oracle import mcsd_oracle as orc
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    lens = seq_lens(w)
    gam = gammas(w)
    n_act = np.array([orc.n_active_for_gamma(parent, int(g)) for g in gam])
    scale = 1.0 / np.sqrt(w.D)
    # attention: one (b, h) problem at a time, drawn with the workload's seeded generator
    t_attn, pairs = 0.0, 0
    wb = dataclasses.replace(w, B=1, H=1)
    # Generated problems are kept and taken in turn (drawing one costs more than solving it); 64 of them are a few
    # hundred MB, more than the host's caches hold, so every solve still streams its keys and values from memory.
    pool = _ORACLE_POOL.setdefault((w.name, w.B, w.H), {})
    while pairs < min_pairs or (t_attn < budget_s and pairs < w.B * w.H * w.n_layers):
        b = pairs % w.B
        slot = pairs % 64
        if slot not in pool:
            one = dataclasses.replace(wb, base_seed=w.seed(0, 0) + 7919 * slot, prefix=(int(lens[b]), int(lens[b])))
            pool[slot] = {k: v.float().numpy() for k, v in attention_inputs(one, 0, "cpu").items()}
        inp = pool[slot]
        t0 = time.perf_counter()
        orc.tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"], [int(lens[b])],
                           [int(n_act[b])], parent, scale)
        t_attn += time.perf_counter() - t0
        pairs += 1
    # verify: whole sequences
    nseq = min(w.B, 4)
    vin = verify_inputs(w, 0, "cpu", parent=parent, B=nseq)
    host = {k: v.numpy() for k, v in vin.items()}
    t0 = time.perf_counter()
    orc.verify_tree(host["p"], host["q"], host["tokens"], parent, gam[:nseq], host["u_accept"], host["u_bonus"])
    t_ver = time.perf_counter() - t0
    step_s = t_attn / pairs * (w.B * w.H * w.n_layers) + t_ver / nseq * w.B
    try:
        from threadpoolctl import threadpool_info
        threads = max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    sample = ("%d of %d (sequence, head, layer) attention problems (%.1f s; %d distinct seeded problems of the workload's "
              "shapes taken in turn) and %d of %d verify sequences (%.2f s), extrapolated to one full step"
              % (pairs, w.B * w.H * w.n_layers, t_attn, len(pool), nseq, w.B, t_ver))
    return float(n_act.sum()) / step_s, sample, threads, step_s


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from mcsd_inputs import workload
    w = workload(args.workload)
    vals = []
    for i in range(args.warmup + args.steps):
        v, sample, threads, step_s = oracle_sample(w, budget_s=max(2.0, args.oracle_seconds / max(1, args.warmup + args.steps)))
        if i >= args.warmup:
            vals.append((v, step_s))
    value = float(np.mean([v for v, _ in vals]))
    ms = float(np.mean([s for _, s in vals])) * 1e3
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": _config(w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def cpu_baseline_in_fresh_process(workload_name, seconds=24.0):
    """The oracle leg of the GPU arm: the same program as `--impl reference` with the same untimed first pass, started
    as a new interpreter.  (Timed cold, without that pass, the same sample reads 2.2 x slower: the first pass pays for
    the page faults of the problem pool and the start of the BLAS threads.)"""
    cmd = [sys.executable, os.path.abspath(__file__), "--impl", "reference", "--workload", workload_name, "--steps", "1",
           "--warmup", "1", "--oracle-seconds", str(seconds)]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, env=env)
    for ln in reversed(res.stdout.strip().splitlines()):
        try:
            return json.loads(ln)["cpu_baseline"]
        except (ValueError, KeyError):
            continue
    return {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": "oracle process failed: " + res.stderr[-300:]}


def torchrun_command(n, argv, port, script=None):
    """Command line that starts n ranks of this script on this node (one per GPU) the way the scaling runs do."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr",
            "127.0.0.1", "--master-port", str(port), script or os.path.abspath(__file__)] + list(argv)


def launch_ranks(n, argv, runner=subprocess.call, script=None):
    """`python bench.py --gpus N` outside torchrun: start the N ranks here and hand back their exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return runner(torchrun_command(n, argv, port, script))


def _config(w, n_gpus):
    return {"workload": w.name, "batch_per_gpu": w.B, "heads": w.H, "head_dim": w.D, "prefix": list(w.prefix),
            "tree": {"n_roots": w.n_roots, "branching": list(w.branching), "nodes": w.n_nodes},
            "layers": w.n_layers, "vocab": w.V, "parallelism": "batch-sharded x%d, no collective" % n_gpus,
            "l2": "inputs larger than L2: every layer reads its own %.0f MB KV cache" %
                  (2 * w.B * w.H * w.L_max * w.D * (4 if w.dtype == "f32" else 2) / 1e6)}


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def verify_rows_read(states, parent, n_act):
    """Probability rows (of V floats) the verify kernel reads, counted on the host from the node states it left in the
    workspace: an internal node's pair of rows once per rejected child (the first test needs two scalars only), and
    at the stop node of the winning path the target row, plus the draft row if a child was rejected there.  (The
    located range of the inverse CDF is read a second time: at most a sixteenth of a row, not counted.)"""
    parent = np.asarray(parent)
    N = len(parent)
    first = np.full(N, -1)
    cnt = np.zeros(N, dtype=np.int64)
    for c, u in enumerate(parent):
        if u >= 0:
            if first[u] < 0:
                first[u] = c
            cnt[u] += 1
    nxt = states["next_child"].cpu().numpy()
    cc = states["c"].cpu().numpy()
    rows = 0
    for b in range(nxt.shape[0]):
        for u in range(int(n_act[b])):
            if cnt[u] == 0 or first[u] >= n_act[b]:
                continue
            rej = cnt[u] if nxt[b, u] < 0 else nxt[b, u] - first[u]
            rows += 2 * int(rej)
    return rows, cc


def measure_workload(mcsd, name, dev, layers, steps, flush):
    """Attention per layer and the verify step of one workload, replayed from CUDA graphs after an L2 flush."""
    import torch
    from mcsd_inputs import attention_inputs, gammas, parent_array, seq_lens, verify_inputs, workload
    w = dataclasses.replace(workload(name), n_layers=layers)
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    elt = 4 if w.dtype == "f32" else 2
    code = mcsd.MCSD_F32 if w.dtype == "f32" else mcsd.MCSD_BF16
    tm = mcsd.mcsd_build_mask(parent, device=dev)
    lens, gam = seq_lens(w), gammas(w)
    n_act = mcsd.n_active_from_gamma(tm.level_start_host, gam)
    lens_d, nact_d, gam_d = (torch.from_numpy(x).to(dev) for x in (lens, n_act, gam))
    lay = [attention_inputs(w, l, dev) for l in range(layers)]
    outs = [torch.empty_like(l["q"]) for l in lay]
    vin = verify_inputs(w, 0, dev, parent=parent)
    ws_a = mcsd.new_workspace(mcsd.mcsd_tree_attention_workspace_bytes(w.B, w.H, N, w.D, w.L_max, code), dev)
    ws_v = mcsd.new_workspace(mcsd.mcsd_verify_tree_workspace_bytes(w.B, N, w.V), dev)
    scale = 1.0 / float(np.sqrt(w.D))

    def attn():
        for inp, o in zip(lay, outs):
            mcsd.mcsd_tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"], lens_d, nact_d, tm,
                                     out=o, softmax_scale=scale, workspace=ws_a)
    vout = mcsd.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"], workspace=ws_v)

    def ver():
        mcsd.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"], workspace=ws_v, out=vout)
    attn()
    torch.cuda.synchronize()
    ga, gv = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
    with torch.cuda.graph(ga):
        attn()
    with torch.cuda.graph(gv):
        ver()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for k in range(-3, steps):
        flush.zero_()
        e = ev[max(k, 0)]
        e[0].record(); ga.replay(); e[1].record(); gv.replay(); e[2].record()
    torch.cuda.synchronize()
    a_ms = float(np.median([e[0].elapsed_time(e[1]) for e in ev])) / layers
    v_ms = float(np.median([e[1].elapsed_time(e[2]) for e in ev]))
    if mcsd.mcsd_workspace_status(ws_a) != 0 or mcsd.mcsd_workspace_status(ws_v) != 0:
        raise SystemExit("a device-side wait timed out in workload %s" % name)
    abytes = _algorithmic_bytes_attention(w.H, w.D, lens, n_act, tm.words, elt)
    rows, _ = verify_rows_read(mcsd.verify_node_states(ws_v, w.B, N), parent, n_act)
    rows += 2 * w.B                                    # stop node: target row, and (upper bound) the draft row
    peak, _ = _peaks()
    return {"workload": w.name, "layers_timed": layers, "tree_tokens": int(n_act.sum()), "attention_ms_per_layer": a_ms,
            "attention_GBs": abytes / (a_ms * 1e-3) / 1e9, "frac": abytes / (a_ms * 1e-3) / 1e9 / peak,
            "attention_algorithmic_bytes": int(abytes), "verify_ms": v_ms,
            "verify_nodes_per_s": float(n_act.sum()) / (v_ms * 1e-3),
            "verify_lazy_bytes": int(rows) * w.V * 4, "verify_lazy_GBs": rows * w.V * 4 / (v_ms * 1e-3) / 1e9,
            "verify_all_rows_bytes": int(n_act.sum()) * w.V * 4 * 2}


WORKLOAD_LAYERS = {"tiny_fp32": 8, "llama7b_b1": 8, "dynamic_slice_b8": 8, "long_context_b16": 8, "target_init_b32": 8,
                   "paper_static_2_4_3_1_1": 8, "paper_fork_w16_d5": 8}


def run_ours(args):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    import paper_2409_10644_b200 as mcsd
    from paper_2409_10644_b200.dist import aggregate
    from mcsd_inputs import attention_inputs, gammas, parent_array, seq_lens, verify_inputs, workload

    w0 = workload(args.workload)
    if args.batch > 0:
        w0 = dataclasses.replace(w0, B=args.batch)
    if args.layers > 0:
        w0 = dataclasses.replace(w0, n_layers=args.layers)
    w = dataclasses.replace(w0, base_seed=1000 * w0.index + 100000 * rank)
    parent = parent_array(w.n_roots, w.branching)
    N = len(parent)
    elt = 4 if w.dtype == "f32" else 2
    code = mcsd.MCSD_F32 if w.dtype == "f32" else mcsd.MCSD_BF16

    # ---- init (untimed): mask once, resident KV caches, per-step inputs staged in pinned host memory ----
    tm = mcsd.mcsd_build_mask(parent, device=dev)
    lens = seq_lens(w)
    gam = gammas(w)
    n_act = mcsd.n_active_from_gamma(tm.level_start_host, gam)
    lens_d = torch.from_numpy(lens).to(dev)
    nact_d = torch.from_numpy(n_act).to(dev)
    gam_d = torch.from_numpy(gam).to(dev)
    layers = [attention_inputs(w, l, dev) for l in range(w.n_layers)]
    vin = verify_inputs(w, 0, dev, parent=parent)
    outs = [torch.empty_like(l["q"]) for l in layers]
    ws_attn = mcsd.new_workspace(mcsd.mcsd_tree_attention_workspace_bytes(w.B, w.H, N, w.D, w.L_max, code), dev)
    ws_ver = mcsd.new_workspace(mcsd.mcsd_verify_tree_workspace_bytes(w.B, N, w.V), dev)
    vout = mcsd.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"],
                                 workspace=ws_ver)
    scale = 1.0 / float(np.sqrt(w.D))

    def step(timed_events=None):
        for l, (inp, o) in enumerate(zip(layers, outs)):
            if timed_events is not None:
                timed_events[l][0].record()
            mcsd.mcsd_tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"], lens_d,
                                     nact_d, tm, out=o, softmax_scale=scale, workspace=ws_attn)
            if timed_events is not None:
                timed_events[l][1].record()
        mcsd.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"],
                              workspace=ws_ver, out=vout)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    sync_all()
    if mcsd.mcsd_workspace_status(ws_attn) != 0 or mcsd.mcsd_workspace_status(ws_ver) != 0:
        raise SystemExit("a device-side wait timed out during warm-up; results would be invalid")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in layers]
          for _ in range(args.steps)]
    ver_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph:
        # The same launches replayed from two CUDA graphs (all attention layers; the verify step), so that the host's
        # launch path (25-50 us per call from Python) is not in the numbers of workloads whose kernels are shorter.
        def attn_layers():
            for inp, o in zip(layers, outs):
                mcsd.mcsd_tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"], lens_d,
                                         nact_d, tm, out=o, softmax_scale=scale, workspace=ws_attn)

        def verify_only():
            mcsd.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"],
                                  workspace=ws_ver, out=vout)
        l0 = mcsd.mcsd_launch_count()
        g_attn, g_ver = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_attn):
            attn_layers()
        with torch.cuda.graph(g_ver):
            verify_only()
        per_step = mcsd.mcsd_launch_count() - l0
        for _ in range(3):
            g_attn.replay()
            g_ver.replay()
        mid = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
        beg = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
        sync_all()
        t_start.record()
        for k in range(args.steps):
            beg[k].record()
            g_attn.replay()
            mid[k].record()
            g_ver.replay()
            ver_ev[k][1].record()
        t_end.record()
        sync_all()
        launches = per_step * args.steps
        clocks = sampler.stop() if rank == 0 else None
        ms_local = t_start.elapsed_time(t_end) / args.steps
        attn_ms = float(np.mean([beg[k].elapsed_time(mid[k]) for k in range(args.steps)])) / len(layers)
        ver_ms = float(np.mean([mid[k].elapsed_time(ver_ev[k][1]) for k in range(args.steps)]))
    else:
        sync_all()
        launches0 = mcsd.mcsd_launch_count()
        t_start.record()
        for k in range(args.steps):
            step(ev[k])
            ver_ev[k][1].record()
        t_end.record()
        sync_all()
        launches = mcsd.mcsd_launch_count() - launches0
        clocks = sampler.stop() if rank == 0 else None
        ms_local = t_start.elapsed_time(t_end) / args.steps
        attn_ms = float(np.mean([a.elapsed_time(b) for per in ev for (a, b) in per]))
        ver_ms = float(np.mean([ev[k][-1][1].elapsed_time(ver_ev[k][1]) for k in range(args.steps)]))
    if mcsd.mcsd_workspace_status(ws_attn) != 0:
        raise SystemExit("a device-side wait timed out; results are invalid")

    units, ms = aggregate(float(n_act.sum()), ms_local, device=dev)
    value = units / (ms * 1e-3)

    # ---- end to end: per-step inputs come from pinned host memory, results go back to the host ----
    pin = lambda t: t.detach().cpu().pin_memory()
    h_layers = [{k: pin(l[k]) for k in ("q", "k_tree", "v_tree")} for l in layers]
    h_vin = {k: pin(v) for k, v in vin.items()}
    h_lens, h_gam, h_nact = pin(lens_d), pin(gam_d), pin(nact_d)
    h_outs = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs]
    h_vout = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in vout.items() if v is not None}
    h2d = sum(t.numel() * t.element_size() for l in h_layers for t in l.values()) + \
        sum(t.numel() * t.element_size() for t in h_vin.values()) + 3 * 4 * w.B
    d2h = sum(t.numel() * t.element_size() for t in h_outs) + sum(t.numel() * t.element_size() for t in h_vout.values())

    # Copies and kernels are pipelined the way a serving loop would do it: one stream uploads (lengths first, then the
    # tree tensors layer after layer, then the verify inputs), the compute stream starts a layer as soon as its
    # tensors have landed, a third stream reads each layer's output back while later layers run.  PCIe carries both
    # directions at once.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in layers]
    ev_done = [torch.cuda.Event() for _ in layers]
    ev_vin, ev_ver = torch.cuda.Event(), torch.cuda.Event()

    def e2e_step():
        cur = torch.cuda.current_stream()
        s_in.wait_stream(cur)                  # the previous step no longer reads the input buffers
        with torch.cuda.stream(s_in):
            lens_d.copy_(h_lens, non_blocking=True)
            gam_d.copy_(h_gam, non_blocking=True)
            nact_d.copy_(h_nact, non_blocking=True)
            for i, (l, hl) in enumerate(zip(layers, h_layers)):
                for k, t in hl.items():
                    l[k].copy_(t, non_blocking=True)
                ev_in[i].record(s_in)
            for k, t in h_vin.items():
                vin[k].copy_(t, non_blocking=True)
            ev_vin.record(s_in)
        for i, (inp, o) in enumerate(zip(layers, outs)):
            cur.wait_event(ev_in[i])
            mcsd.mcsd_tree_attention(inp["q"], inp["k_cache"], inp["v_cache"], inp["k_tree"], inp["v_tree"], lens_d,
                                     nact_d, tm, out=o, softmax_scale=scale, workspace=ws_attn)
            ev_done[i].record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                h_outs[i].copy_(o, non_blocking=True)
        cur.wait_event(ev_vin)
        mcsd.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"],
                              workspace=ws_ver, out=vout)
        ev_ver.record(cur)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_ver)
            for k, t in h_vout.items():
                t.copy_(vout[k], non_blocking=True)
        cur.wait_stream(s_out)                 # the step ends when its last result is on the host

    e2e_steps = max(2, min(args.steps, 5))
    e2e_step()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    sync_all()
    e2e_units, e2e_ms = aggregate(float(n_act.sum()), e0.elapsed_time(e1) / e2e_steps, device=dev)
    e2e_value = e2e_units / (e2e_ms * 1e-3)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    peak, peak_kind = _peaks()
    abytes = _algorithmic_bytes_attention(w.H, w.D, lens, n_act, tm.words, elt)
    achieved = abytes / (attn_ms * 1e-3) / 1e9
    ver_rows_bytes = int(n_act.sum()) * w.V * 4 * 2
    lazy_rows, _ = verify_rows_read(mcsd.verify_node_states(ws_ver, w.B, N), parent, n_act)
    lazy_bytes = int(lazy_rows + 2 * w.B) * w.V * 4
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": _config(w, world), "launch": "cuda graphs" if args.graph else "stream launches",
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": e2e_ms,
                "note": "per step the tree's q/k/v of every layer, p, q, tokens, uniforms, lengths and gammas are copied "
                        "from pinned host memory and every layer's attention output plus the verify results are read "
                        "back, with uploads, kernels and read-backs pipelined on three streams; the prefix KV cache is "
                        "decode state and stays resident in HBM"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "tree attention (one layer: main kernel + split-KV combine)",
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": int(abytes), "avg_launch_ms": attn_ms, "traffic": _traffic_for(w0)},
        "breakdown": {"attention_ms_per_layer": attn_ms, "verify_ms": ver_ms,
                      "verify_nodes_per_s": float(n_act.sum()) / (ver_ms * 1e-3),
                      "verify_all_rows_GBs": ver_rows_bytes / (ver_ms * 1e-3) / 1e9,
                      "verify_lazy_bytes": lazy_bytes, "verify_lazy_GBs": lazy_bytes / (ver_ms * 1e-3) / 1e9,
                      "verify_bytes_note": "lazy = rows the kernel reads (a node's p and q rows once per rejected child, the "
                                           "stop node's rows), counted from the node states; all_rows = every active node's "
                                           "two rows, an upper bound the kernel does not move",
                      "tree_tokens_per_s_per_layer": float(n_act.sum()) / (attn_ms * 1e-3),
                      "mean_accept_len": float(vout["accept_len"].float().mean().item())},
    }
    if world == 1 and args.workloads:
        # the other workloads on the same box and clock record: a few layers each, graph replay after an L2 flush
        del h_layers, h_outs
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        table = []
        for name, nl in WORKLOAD_LAYERS.items():
            table.append(measure_workload(mcsd, name, dev, nl, 7, flush))
            torch.cuda.empty_cache()
        line["breakdown"]["workloads"] = table
        line["breakdown"]["workloads_note"] = ("every workload of the input table, eight layers each with their own KV caches, "
                                               "launches replayed from CUDA graphs, L2 flushed before each replay, medians of 7")
    if world == 1 and args.vocab_shards > 1:
        line["breakdown"]["vocab_sharded_verify"] = _time_vocab_sharded_verify(mcsd, w, vin, tm, gam_d, parent,
                                                                               args.vocab_shards, vout)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline_in_fresh_process(w0.name)
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def _time_vocab_sharded_verify(mcsd, w, vin, tm, gam_d, parent, R, vout):
    """Kernel time of the vocabulary-sharded verify step with the R ranks' column slices all on this GPU: the ranks'
    launches run one after the other in one stream, the all-reduces are replaced by combining the exchange buffers
    on the device, and the whole sequence is replayed from a CUDA graph so that the host's launch path is not in the
    number.  `ms_per_rank` = total / R still contains the stand-in reductions, so it bounds one rank's kernels from
    above; a real job adds k + 3 small all-reduces."""
    import torch
    from paper_2409_10644_b200 import dist as mdist
    k = mdist.max_children(parent)
    shards = []
    for r in range(R):
        v0, v1 = mdist.vocab_shard_range(w.V, r, R)
        shards.append(mcsd.VocabShard(vin["p"][:, :, v0:v1].contiguous(), vin["q"][:, :, v0:v1].contiguous(), v0, w.V,
                                      r, R, vin["tokens"], tm, gam_d, vin["u_accept"], vin["u_bonus"]))
    l0 = mcsd.mcsd_launch_count()
    outs = mdist.drive_vocab_shards(shards, mdist.reduce_on_one_device, k)
    launches = mcsd.mcsd_launch_count() - l0
    torch.cuda.synchronize()
    same = all(bool(torch.equal(o[key], vout[key])) for o in outs
               for key in ("accept_len", "out_tokens", "out_nodes", "best_root"))
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        mdist.drive_vocab_shards(shards, mdist.reduce_on_one_device, k)
    for _ in range(3):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 20
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    total = e0.elapsed_time(e1) / reps
    return {"ranks_on_one_gpu": R, "rounds": k + 1, "all_reduces_per_step": k + 3, "launches_all_ranks": int(launches),
            "ms_all_ranks": total, "ms_per_rank": total / R, "matches_single_gpu_outputs": same}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long_context_b16")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (profiling of a smaller case only)")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling only)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="issue the step's launches one by one from Python instead of replaying them from CUDA graphs "
                         "(the host's launch path, 25-50 us per call, then bounds workloads with shorter kernels)")
    ap.add_argument("--no-workloads", dest="workloads", action="store_false",
                    help="skip the per-workload table (breakdown.workloads) of the default run")
    ap.add_argument("--oracle-seconds", type=float, default=60.0, help="--impl reference: oracle time in total")
    ap.add_argument("--vocab-shards", type=int, default=0,
                    help="also time the vocabulary-sharded verify step with this many ranks' column slices on one GPU")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand with --gpus N: become the launcher of N ranks (torchrun sets WORLD_SIZE for them)
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
