#!/usr/bin/env python
"""Benchmark of the sparse-attention layer over a synthetic And-Inverter Graph.

One step = one pass of the whole hot path over the 10M-node workload (50 000 primary inputs + 10 000 000
gates, log-uniform locality window, 2-hop cones, d = 128, 8 heads, bf16):
    device graph prep (neighbourhood CSR, level buckets, class orderings)
    + 3 layers all-nodes-parallel (QKV projection, fused sparse attention, output projection + residual)
    + 3 layers levelised (the same layer in topological level order).
The metric is AIG nodes per second per sparse-attention layer: nodes x layer passes / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--shrink S]
    python bench.py --per-config [--configs 1,2,3] [--cpu-only --cpu-threads T]    (a table, see run_per_config)

With N > 1 (under torchrun) every rank runs its own circuit of the same shape (weak scaling, no collective
on the data path); the reported time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "AIG nodes/s per sparse-attention layer"
UNIT = "nodes/s"
FALLBACK_HBM_GBS = 6650.0


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def workload_config(w, n_levels=None, n_nbr=None):
    c = {"workload": w.name, "n_pi": w.n_pi, "n_gates": w.n_gates, "hops": w.hops, "d": w.d, "heads": w.heads,
         "layers": w.layers, "modes": list(w.modes), "window_log2": list(w.win_exp), "not_ratio": w.not_ratio,
         "residual": w.residual, "l2": "inputs larger than L2 (no flush)"}
    if n_levels is not None:
        c["n_levels"] = int(n_levels)
    if n_nbr is not None:
        c["n_nbr"] = int(n_nbr)
    return c


# --------------------------------------------------------------------------------------------------
# CPU checker timed on a bounded sample (reported baseline; also the --impl reference arm)
# --------------------------------------------------------------------------------------------------

def cpu_sample_problem(w, sample_nodes):
    """A circuit of about `sample_nodes` nodes from the workload's own generator (same primary-input share,
    window distribution, NOT ratio, hops and tensor recipe; node counts divided), small enough for the CPU."""
    from oracle import oracle as orc
    from paper_2502_01681_b200 import synth
    ws = synth.workload(5, max(1, round(w.n / sample_nodes)))
    g = ws.graph()
    sample_nodes = g.n
    ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)
    lptr, lnodes = orc.level_buckets(g.level)
    x = synth.bf16_bits_to_f32(w.x_bf16_bits(sample_nodes)).astype(np.float64)
    wq = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(w.w_qkv_f32(0))).astype(np.float64)
    wo = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(w.w_o_f32(0))).astype(np.float64)
    return g, ptr, idx, lptr, lnodes, x, wq, wo


def sample_text(prob):
    g = prob[0]
    return (f"the workload's generator at {g.n} nodes ({len(prob[3]) - 1} levels): graph prep + 1 parallel layer "
            f"+ 1 levelised layer, fp64")


def cpu_step(w, prob):
    """One parallel + one levelised layer of the checker on the sample; returns seconds."""
    from oracle import oracle as orc
    g, ptr, idx, lptr, lnodes, x, wq, wo = prob
    t0 = time.perf_counter()
    orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)
    orc.level_buckets(g.level)
    orc.layer_parallel(x, wq, wo, ptr, idx, w.heads, w.scale, residual=w.residual, rounding="bf16")
    orc.layer_levelised(x, wq, wo, ptr, idx, lptr, lnodes, w.heads, w.scale, residual=w.residual, rounding="bf16")
    return time.perf_counter() - t0


def cpu_baseline(w, sample_nodes=100_000, target_s=15.0):
    """Times the checker on a sample sized for roughly `target_s` seconds of CPU work on this host."""
    from oracle import oracle as orc
    prob = cpu_sample_problem(w, sample_nodes)
    dt = cpu_step(w, prob)
    if dt < target_s / 3:                      # fast host: scale the sample up once (at most 1M nodes)
        bigger = int(min(1_000_000, sample_nodes * target_s / max(dt, 1e-3)))
        prob = cpu_sample_problem(w, bigger)
        dt = cpu_step(w, prob)
    return {"value": prob[0].n * 2 / dt, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": sample_text(prob) + f", {dt:.1f} s"}


def run_reference(args, w):
    """--impl reference: the CPU checker as it stands, on the host cores, on a bounded sample per step."""
    from oracle import oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_nodes = 50_000
    prob = cpu_sample_problem(w, sample_nodes)
    for _ in range(args.warmup):
        cpu_step(w, prob)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        cpu_step(w, prob)
    dt = (time.perf_counter() - t0) / args.steps
    value = prob[0].n * 2 / dt
    sample = "per step: " + sample_text(prob)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(workload_config(w), sample_nodes=int(prob[0].n), sample_levels=int(len(prob[3]) - 1),
                           sample=("each step runs the CPU checker on a circuit of sample_nodes nodes drawn by this "
                                   "workload's generator, not on the full n_pi + n_gates nodes")),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.idx = device_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            sm, mx, reasons = [], [], set()
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            if sm:
                out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                       "samples": len(sm)}
        finally:
            try:
                os.unlink(self.path)
            except OSError:
                pass
        return out


# --------------------------------------------------------------------------------------------------
# aggregation over ranks (weak scaling: every rank runs its own circuit; no collective on the data path)
# --------------------------------------------------------------------------------------------------

def reduce_over_ranks(dist, device, seconds, units):
    """Whole-job figures from per-rank ones: the time is the MAXIMUM over ranks, the work the SUM over ranks.
    `dist` is torch.distributed (initialised) or None for a single process."""
    if dist is None:
        return float(seconds), float(units)
    import torch
    t = torch.tensor([float(seconds)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------------------------------------
# the GPU arm
# --------------------------------------------------------------------------------------------------

def run_ours(args, w):
    import torch
    from paper_2502_01681_b200 import dg4, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # every rank its own circuit of the same shape (weak scaling)
    w.seed = w.seed + 1000 * rank
    g = w.graph()
    n = g.n
    x_host = torch.empty((n, w.d), dtype=torch.int16).pin_memory()
    w.x_bf16_bits(out=x_host.numpy().view(np.uint16))
    wq = [torch.from_numpy(synth.f32_to_bf16_bits(w.w_qkv_f32(l)).view(np.int16)).cuda().view(torch.bfloat16)
          for l in range(w.layers)]
    wo = [torch.from_numpy(synth.f32_to_bf16_bits(w.w_o_f32(l)).view(np.int16)).cuda().view(torch.bfloat16)
          for l in range(w.layers)]
    out_host = torch.empty((n, w.d), dtype=torch.int16).pin_memory()

    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0, local)
    info = gr.info
    dsc = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=w.residual)
    ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc), dg4.dg4_layers_workspace_bytes(gr, dsc, w.layers)),
                     dtype=torch.uint8, device="cuda")
    x_dev = x_host.cuda().view(torch.bfloat16)
    h_par = torch.empty_like(x_dev)
    h_lev = torch.empty_like(x_dev)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # views into the workspace, laid out as the layer calls lay it out: Q [n,128] | KV [n,256] | O [n,128]
    wsb = ws.view(torch.bfloat16)
    q_v = wsb[: n * 128].view(n, 128)
    kv_v = wsb[n * 128: n * 384].view(n, 256)
    o_v = wsb[n * 384: n * 512].view(n, 128)
    stream = torch.cuda.current_stream()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    stage_ev = []          # (name, start, stop) per step

    def step(record):
        marks = []

        def mark(name, fn):
            if record:
                a, b = ev(), ev()
                a.record(stream)
                fn()
                b.record(stream)
                marks.append((name, a, b))
            else:
                fn()

        mark("graph_prep", lambda: dg4.dg4_graph_rebuild(gr))
        h_par.copy_(x_dev)
        for l in range(w.layers):
            mark("qkv", lambda: dg4.dg4_qkv_project(gr, dsc, h_par, wq[l], q_v, kv_v[:, :128], kv_v[:, 128:]))
            mark("attn", lambda: dg4.dg4_sparse_attn_fwd(gr, dsc, q_v, kv_v[:, :128], kv_v[:, 128:], o_v))
            mark("out", lambda: dg4.dg4_out_project(gr, dsc, o_v, wo[l], h_par, h_par))
        h_lev.copy_(x_dev)
        if not args.no_levelised:        # all layers in one call: they run as a wavefront over the levels
            mark("levelised", lambda: dg4.dg4_layers_fwd_levelised(gr, dsc, h_lev, wq, wo, ws, status))
        if record:
            stage_ev.append(marks)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step(False)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = dg4.dg4_launch_count()
    t_start, t_stop = ev(), ev()
    barrier()
    t_start.record(stream)
    for _ in range(args.steps):
        step(True)
    t_stop.record(stream)
    barrier()
    launches = dg4.dg4_launch_count() - launches0
    clocks = sampler.stop()
    assert int(status.item()) == 0, "device status reported an error"
    layer_passes = w.layers * 2
    total_s, total_units = reduce_over_ranks(dist, "cuda", t_start.elapsed_time(t_stop) * 1e-3,
                                             float(n) * layer_passes * args.steps)
    ms_per_step = total_s * 1e3 / args.steps
    value = total_units / total_s

    stages = {}
    for marks in stage_ev:
        for name, a, b in marks:
            stages.setdefault(name, []).append(a.elapsed_time(b))
    attn_ms = float(np.mean(stages["attn"]))
    alg_bytes = 516.0 * n + 516.0 * info.n_nbr
    peak, peak_kind = measured_hbm_peak()
    achieved = alg_bytes / (attn_ms * 1e-3) / 1e9
    per_step = lambda name: float(np.sum(stages.get(name, [float("nan")]))) / args.steps
    stage_report = {
        "graph_prep_ms": per_step("graph_prep"),
        "qkv_ms_per_layer": per_step("qkv") / w.layers,
        "attn_ms_per_layer": attn_ms,
        "out_ms_per_layer": per_step("out") / w.layers,
        "levelised_ms_per_layer": per_step("levelised") / w.layers,
        "parallel_layer_nodes_per_s": n / ((per_step("qkv") + per_step("attn") + per_step("out")) / w.layers * 1e-3),
        "levelised_layer_nodes_per_s": n / (per_step("levelised") / w.layers * 1e-3),
        "attn_kernel_nodes_per_s": n / (attn_ms * 1e-3),
    }

    # ---- outside the timed region: the additive-score variant of the attention kernel on the same circuit
    extras = {}
    if world == 1:
        s_dst = torch.randn(n, w.heads, device="cuda")
        s_src = torch.randn(n, w.heads, device="cuda")
        for _ in range(2):
            dg4.dg4_sparse_attn_additive_fwd(gr, dsc, s_dst, s_src, 0.2, kv_v[:, 128:], o_v)
        a0, a1 = ev(), ev()
        a0.record(stream)
        for _ in range(3):
            dg4.dg4_sparse_attn_additive_fwd(gr, dsc, s_dst, s_src, 0.2, kv_v[:, 128:], o_v)
        a1.record(stream)
        torch.cuda.synchronize()
        add_ms = a0.elapsed_time(a1) / 3
        add_bytes = (256.0 + 4 * w.heads + 36.0) * n + (256.0 + 4 * w.heads) * info.n_nbr
        extras = {"attn_additive_ms": add_ms, "attn_additive_algorithmic_gbs": add_bytes / (add_ms * 1e-3) / 1e9}
        del s_dst, s_src
        # the rest of the Transformer block on the same rows: feed-forward sub-layer (fused, tensor cores) and LayerNorm
        w1 = (torch.randn(512, 128, device="cuda") * 0.05).to(torch.bfloat16)
        w2 = (torch.randn(128, 512, device="cuda") * 0.05).to(torch.bfloat16)
        b1, b2 = torch.randn(512, device="cuda") * 0.1, torch.randn(128, device="cuda") * 0.1
        gam, bet = torch.ones(128, device="cuda"), torch.zeros(128, device="cuda")

        def timed3(fn):
            for _ in range(2):
                fn()
            t0, t1 = ev(), ev()
            t0.record(stream)
            for _ in range(3):
                fn()
            t1.record(stream)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / 3

        ffn_ms = timed3(lambda: dg4.dg4_ffn_fwd(gr, dsc, x_dev, w1, b1, w2, b2, gam, bet, 1e-5, o_v))
        ln_ms = timed3(lambda: dg4.dg4_layernorm_fwd(gr, dsc, x_dev, gam, bet, 1e-5, o_v))
        blk_ms = timed3(lambda: dg4.dg4_block_fwd_parallel(gr, dsc, x_dev, wq[0], wo[0], gam, bet, w1, b1, w2, b2, gam,
                                                           bet, 1e-5, h_par, ws))
        # the all-parallel layer in its opt-in one-kernel form (K|V projection + fused kernel), for comparison
        # with the three kernels timed inside the step
        dsc_fused = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=w.residual, fused_layer=True)
        fused_ms = timed3(lambda: dg4.dg4_layer_fwd_parallel(gr, dsc_fused, x_dev, wq[0], wo[0], h_par, ws))
        # the whole block level by level: one block, and three blocks as one wavefront (persistent kernel whose
        # attention-stage and feed-forward-stage CTAs hand the levels to one another), in place on a copy of X
        blocks3 = [(wq[l], wo[l], gam, bet, w1, b1, w2, b2, gam, bet) for l in range(3)]
        ws_blk = torch.empty(max(dg4.dg4_blocks_workspace_bytes(gr, dsc, 3), dg4.dg4_layer_workspace_bytes(gr, dsc)),
                             dtype=torch.uint8, device="cuda")

        def timed1(fn):
            h_par.copy_(x_dev)
            fn()
            h_par.copy_(x_dev)
            t0, t1 = ev(), ev()
            t0.record(stream)
            fn()
            t1.record(stream)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1)

        block_lev_ms = timed1(lambda: dg4.dg4_block_fwd_levelised(gr, dsc, h_par, *blocks3[0], 1e-5, ws_blk))
        blocks3_lev_ms = timed1(lambda: dg4.dg4_blocks_fwd_levelised(gr, dsc, h_par, blocks3, 1e-5, ws_blk))
        del ws_blk
        extras.update({"block_levelised_ms": block_lev_ms, "blocks3_levelised_ms": blocks3_lev_ms})
        extras.update({"ffn_ms": ffn_ms, "ffn_tflops": 4.0 * 128 * 512 * n / (ffn_ms * 1e-3) / 1e12,
                       "layernorm_ms": ln_ms, "layernorm_gbs": 512.0 * n / (ln_ms * 1e-3) / 1e9,
                       "block_parallel_ms": blk_ms, "parallel_layer_fused_ms": fused_ms})
        del w1, w2
        # the paper's cone depth (k = 8) on the 1M-node circuit: the warp-per-node kernel for wider cones
        w3 = synth.workload(3)
        g3 = w3.graph()
        gr3 = dg4.dg4_graph_create(g3.row_ptr, g3.col_idx, g3.level, 8, 0, local)
        q3, k3, v3 = ((torch.randn(g3.n, 128, device="cuda") * sdev).to(torch.bfloat16) for sdev in (0.5, 0.5, 1.0))
        o3 = torch.empty_like(q3)
        wide_ms = timed3(lambda: dg4.dg4_sparse_attn_fwd(gr3, dsc, q3, k3, v3, o3))
        extras.update({"wide8_nodes": g3.n, "wide8_entries_per_node": gr3.info.n_nbr / g3.n, "wide8_attn_ms": wide_ms,
                       "wide8_gather_tbs": gr3.info.n_nbr * 512.0 / (wide_ms * 1e-3) / 1e12})
        dg4.dg4_graph_destroy(gr3)
        del q3, k3, v3, o3

    # ---- end to end through the C ABI from host buffers -----------------------------------------
    # Every step uploads its circuit (pageable CSR arrays, through dg4_graph_create) and its features (pinned),
    # runs 3 parallel + 3 levelised layers and reads the result back into pinned memory.  Steps are pipelined
    # the way a serving loop would be: while step i computes, the host validates and uploads circuit i+1 on a
    # second stream, and the result of step i-1 drains on a third one.
    e2e_steps = max(2, min(16, args.steps))     # as many as the timed steps (at most 16): the three-stage pipeline's fill and drain amortise over them
    h2d = x_host.numel() * 2 + (g.row_ptr.nbytes + g.col_idx.nbytes + g.level.nbytes)
    d2h = out_host.numel() * 2 * (1 if args.no_levelised else 2)      # the parallel and the levelised result
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    out_hosts = [out_host, torch.empty_like(out_host).pin_memory()]
    out_par_host = torch.empty_like(out_host).pin_memory()
    x_slots = [torch.empty_like(x_dev), torch.empty_like(x_dev)]      # device buffers of two steps in flight
    hp = torch.empty_like(x_dev)
    drained = [None, None]                                # read-back of the step that last used a slot

    def stage_in(i):
        with torch.cuda.stream(up):
            if drained[i % 2] is not None:
                up.wait_event(drained[i % 2])
            x_slots[i % 2].view(torch.int16).copy_(x_host, non_blocking=True)
            arrived = torch.cuda.Event()
            arrived.record(up)
        gr2 = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0, local)
        return x_slots[i % 2], gr2, arrived

    # one untimed round fills the library's memory pool, as a serving loop's first request would
    for gr2 in [dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0, local) for _ in range(2)]:
        dg4.dg4_graph_destroy_async(gr2, stream)
    barrier()
    par_drained = None
    t0 = time.perf_counter()
    staged = stage_in(0)
    for i in range(e2e_steps):
        x2, gr2, arrived = staged
        stream.wait_event(arrived)
        if par_drained is not None:
            stream.wait_event(par_drained)                # the previous step's parallel result has left `hp`
        hp.copy_(x2)
        for l in range(w.layers):
            dg4.dg4_layer_fwd_parallel(gr2, dsc, hp, wq[l], wo[l], hp, ws)
        par_done = torch.cuda.Event()
        par_done.record(stream)
        with torch.cuda.stream(down):                     # the parallel result drains while the levelised layers run
            down.wait_event(par_done)
            out_par_host.copy_(hp.view(torch.int16), non_blocking=True)
            par_drained = torch.cuda.Event()
            par_drained.record(down)
        if not args.no_levelised:
            dg4.dg4_layers_fwd_levelised(gr2, dsc, x2, wq, wo, ws, status)
        done = torch.cuda.Event()
        done.record(stream)
        dg4.dg4_graph_destroy_async(gr2, stream)          # freed once this step's kernels have run
        with torch.cuda.stream(down):
            down.wait_event(done)
            if not args.no_levelised:
                out_hosts[i % 2].copy_(x2.view(torch.int16), non_blocking=True)
            drained[i % 2] = torch.cuda.Event()
            drained[i % 2].record(down)
        if i + 1 < e2e_steps:
            staged = stage_in(i + 1)
    torch.cuda.synchronize()
    barrier()
    e2e_total_s, e2e_units = reduce_over_ranks(dist, "cuda", time.perf_counter() - t0,
                                               float(n) * layer_passes * e2e_steps)
    e2e_s = e2e_total_s / e2e_steps
    e2e_value = e2e_units / e2e_total_s

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "valid": not (args.no_levelised or args.shrink != 1),
            "config": workload_config(w, info.n_levels, info.n_nbr),
            "stages": stage_report,
            "extras": extras,
            "roofline": {"bound": "hbm", "kernel": "sparse_attn_kernel", "achieved": achieved, "peak": peak,
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_nominal_8000": achieved / 8000.0,
                         "algorithmic_bytes_per_launch": alg_bytes,
                         "unique_row_floor_bytes": 4.0 * 256 * n + 4.0 * (info.n_nbr + n),
                         "traffic": TRAFFIC["bytes_per_node"] * n if args.shrink == 1 and TRAFFIC["bytes_per_node"] else None,
                         "traffic_source": TRAFFIC},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": e2e_s * 1e3, "steps": e2e_steps,
                    "note": "steps pipelined: upload of step i+1 and read-back of step i-1 overlap the compute of step i; "
                            "both results (parallel and levelised stack) are read back every step"},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# --per-config: the attention step on each of the five workloads (a table, not the benchmark line)
# --------------------------------------------------------------------------------------------------

def run_per_config(args):
    """Times the fused sparse-attention kernel on each workload: 20 repetitions back to back (warm L2) and 20
    with a 512 MB scratch write in between (cold L2), median and minimum; the layer and the levelised mode
    where the workload has them; the CPU checker's attention on the same circuit beside it.  Prints a
    markdown table."""
    cfgs = [int(c) for c in args.configs.split(",")]
    rows = []
    if not args.cpu_only:
        import torch
        from paper_2502_01681_b200 import dg4
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: the product has no CPU path")
        torch.cuda.set_device(0)
        stream = torch.cuda.current_stream()
        scratch = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    from paper_2502_01681_b200 import synth
    peak, peak_kind = measured_hbm_peak()

    def timed(fn, reps, between=None):
        import torch
        ts = []
        for _ in range(reps):
            if between is not None:
                between()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return float(np.median(ts)), float(np.min(ts))

    for cfg in cfgs:
        w = synth.workload(cfg)
        g = w.graph()
        n = g.n
        r = {"cfg": cfg, "name": w.name, "n": n, "dtype": w.dtype}
        esz = 4 if w.dtype == "f32" else 2
        if not args.cpu_only:
            import torch
            t0 = time.perf_counter()
            gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0, 0)
            torch.cuda.synchronize()
            r["create_ms"] = (time.perf_counter() - t0) * 1e3
            r["prep_ms"] = timed(lambda: dg4.dg4_graph_rebuild(gr), 5)[0]
            info = gr.info
            r["n_nbr"], r["levels"] = int(info.n_nbr), int(info.n_levels)
            tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
            dsc = dg4.desc(w.heads, dg4.DG4_F32 if w.dtype == "f32" else dg4.DG4_BF16, w.scale, residual=w.residual)

            def dev(bits):
                return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

            if w.with_projection:
                x = dev(w.x_bf16_bits())
                wq = [dev(synth.f32_to_bf16_bits(w.w_qkv_f32(l))) for l in range(w.layers)]
                wo = [dev(synth.f32_to_bf16_bits(w.w_o_f32(l))) for l in range(w.layers)]
                q, k, v = (torch.empty_like(x) for _ in range(3))
                dg4.dg4_qkv_project(gr, dsc, x, wq[0], q, k, v)
            elif w.dtype == "f32":
                q, k, v = (torch.from_numpy(t).cuda() for t in w.qkv_f32())
            else:
                q, k, v = (dev(t) for t in w.qkv_bf16_bits())
            o = torch.empty_like(q)
            attn = lambda: dg4.dg4_sparse_attn_fwd(gr, dsc, q, k, v, o)
            for _ in range(3):
                attn()
            r["warm"] = timed(attn, 20)
            r["cold"] = timed(attn, 20, between=lambda: scratch.zero_())
            r["bytes"] = (2 * w.d * esz + 4) * n + (2 * w.d * esz + 4) * r["n_nbr"]
            if w.with_projection:
                ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc),
                                     dg4.dg4_layers_workspace_bytes(gr, dsc, w.layers)),
                                 dtype=torch.uint8, device="cuda")
                status = torch.zeros(1, dtype=torch.int32, device="cuda")
                h = torch.empty_like(x)
                if "parallel" in w.modes:
                    par = lambda: dg4.dg4_layer_fwd_parallel(gr, dsc, x, wq[0], wo[0], h, ws)
                    for _ in range(3):
                        par()
                    r["layer"] = timed(par, 20)
                    # the workload's whole stack of parallel layers: eager launches, then captured once in a CUDA graph
                    def stack():
                        h.copy_(x)
                        for l in range(w.layers):
                            dg4.dg4_layer_fwd_parallel(gr, dsc, h, wq[l], wo[l], h, ws)
                    r["stack"] = timed(stack, 20)
                    side = torch.cuda.Stream()
                    side.wait_stream(stream)
                    cg = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(cg, stream=side):
                        stack()
                    stream.wait_stream(side)
                    cg.replay()
                    r["stack_graph"] = timed(cg.replay, 20)
                    del cg
                if "levelised" in w.modes:
                    lev = lambda: dg4.dg4_layers_fwd_levelised(gr, dsc, h, wq, wo, ws, status)
                    h.copy_(x)
                    lev()
                    r["lev"] = timed(lev, 5, between=lambda: h.copy_(x))
                    dsl = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=w.residual, level_launches=True)
                    r["lev_launches"] = timed(lambda: dg4.dg4_layer_fwd_levelised(gr, dsl, h, wq[0], wo[0], ws, status),
                                              2, between=lambda: h.copy_(x))
                    assert int(status.item()) == 0
                del ws, h
            dg4.dg4_graph_destroy(gr)
            del q, k, v, o
            torch.cuda.empty_cache()
        if not args.no_cpu_baseline:
            from oracle import oracle as orc
            wc = synth.workload(cfg, 10) if cfg == 5 else w       # the 10M-node circuit: a tenth of it
            gc = wc.graph() if cfg == 5 else g
            ptr, idx = orc.neighbourhood(gc.row_ptr, gc.col_idx, w.hops)
            if w.dtype == "f32":
                qc, kc, vc = (t.astype(np.float64) for t in wc.qkv_f32())
            else:
                qc, kc, vc = (synth.bf16_bits_to_f32(t).astype(np.float64) for t in wc.qkv_bf16_bits())
            t0 = time.perf_counter()
            orc.attention(qc, kc, vc, ptr, idx, w.heads, w.scale)
            r["cpu_s"], r["cpu_n"], r["cpu_threads"] = time.perf_counter() - t0, gc.n, orc.num_threads()
        rows.append(r)

    print(f"HBM peak used: {peak:.0f} GB/s ({peak_kind}); nominal 8000 GB/s.  Times in ms as median / minimum.")
    if not args.cpu_only:
        print("\n| cfg | nodes | neighbour entries | levels | graph create (host+device) | device prep | attention, warm L2 "
              "| attention, cold L2 | nodes/s (cold median) | algorithmic GB/s | of measured | of 8000 |")
        print("|---|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|")
        for r in rows:
            t = r["cold"][0] * 1e-3
            gbs = r["bytes"] / t / 1e9
            print(f"| {r['cfg']} {r['name']} ({r['dtype']}) | {r['n']} | {r['n_nbr']} | {r['levels']} | {r['create_ms']:.2f} "
                  f"| {r['prep_ms']:.3f} | {r['warm'][0]:.4f} / {r['warm'][1]:.4f} | {r['cold'][0]:.4f} / {r['cold'][1]:.4f} "
                  f"| {r['n'] / t:.3e} | {gbs:.0f} | {100 * gbs / peak:.0f} % | {100 * gbs / 8000:.0f} % |")
        print("\n| cfg | parallel layer (QKV + attention + output) | all parallel layers, eager launches | the same as one "
              "CUDA graph | levelised, all layers in one launch | per layer "
              "| us per wavefront step (levels + layers - 1 steps) | levelised, one layer as per-level launches |")
        print("|---|---:|---:|---:|---:|---:|---:|---:|")
        for r in rows:
            if "layer" in r or "lev" in r:
                L = synth.workload(r["cfg"]).layers
                lay = (f"{r['layer'][0]:.3f} / {r['layer'][1]:.3f} | {r['stack'][0]:.3f} / {r['stack'][1]:.3f} "
                       f"| {r['stack_graph'][0]:.3f} / {r['stack_graph'][1]:.3f}") if "layer" in r else "- | - | -"
                if "lev" in r:
                    lev = (f"{r['lev'][0]:.2f} / {r['lev'][1]:.2f} | {r['lev'][0] / L:.2f} "
                           f"| {1e3 * r['lev'][0] / (r['levels'] + L - 1):.2f} | {r['lev_launches'][0]:.1f}")
                else:
                    lev = "- | - | - | -"
                print(f"| {r['cfg']} | {lay} | {lev} |")
    if not args.no_cpu_baseline:
        print("\n| cfg | CPU checker, attention only: nodes | threads | seconds | nodes/s |")
        print("|---|---:|---:|---:|---:|")
        for r in rows:
            print(f"| {r['cfg']} | {r['cpu_n']} | {r['cpu_threads']} | {r['cpu_s']:.3f} | {r['cpu_n'] / r['cpu_s']:.3e} |")


# DRAM bytes (read + write) per node of one launch of the roofline kernel, from the ncu capture summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum of one launch / the nodes of that launch; traffic per
# node does not depend on the circuit's size because the window distribution does not).  "bytes_per_node" must be
# set to None whenever the kernel named here changes, until its counters have been taken again.
TRAFFIC = {"kernel": "sparse_attn_kernel<true, 2, 7>", "capture": "profiles/sparse_attn_kernel_cfg5_quarter.md",
           "capture_nodes": 2_512_500, "capture_dram_bytes": 4.149e9, "bytes_per_node": 4.149e9 / 2_512_500}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--shrink", type=int, default=1, help="divide the workload's node counts (profiling only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-levelised", action="store_true",
                    help="profiling only: leave the levelised layers out of the step (the printed value is then "
                         "not a benchmark result)")
    ap.add_argument("--per-config", action="store_true",
                    help="time the attention step on each of the five workloads and print a table instead of "
                         "the benchmark line")
    ap.add_argument("--configs", default="1,2,3,4,5", help="with --per-config: which workloads")
    ap.add_argument("--cpu-only", action="store_true", help="with --per-config: only the CPU checker's column")
    ap.add_argument("--cpu-threads", type=int, default=0, help="with --per-config: OpenMP threads of the CPU checker")
    args = ap.parse_args()
    if args.cpu_threads > 0:
        os.environ["OMP_NUM_THREADS"] = str(args.cpu_threads)
    if args.per_config:
        run_per_config(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" and args.shrink == 1 else args.warmup
    from paper_2502_01681_b200 import synth
    w = synth.workload(5, args.shrink)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
