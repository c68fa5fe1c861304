#!/usr/bin/env python
"""Benchmark of the per-rank MoE expert block on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3-uniform|...] [--impl reference]
    python bench.py --sweep            # cost-profile sweep (G, N grid) + max-affine fit -> n*

One "step" is one pass of the whole hot path (count+dispatch, permute+quantise, the fused gate/up + SwiGLU +
down FFN kernel, combine) over one seeded synthetic routed batch, replayed as one CUDA graph.  Weight copies
rotate through a pool larger than L2 so no step finds its weights cached (the paper's calibration
protocol, Appendix B).  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_expert_block_us"          # step time / activated expert instances (lower is better)
UNIT = "us_per_expert_block"
L2_BYTES = 126 * 1024 * 1024
NOMINAL_FP8_OVER_BF16 = 2.0             # dense fp8 peak = 2 x dense bf16 peak on this part

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused FFN kernel from the committed ncu
# capture (profiles/), keyed by workload; None until a capture exists for that workload.
NCU_TRAFFIC_BYTES = {
    "cfg2": 395.02e6,          # profiles/ffn_kernel_cfg2_flat_decode.md (391.08 MB read + 3.9 MB written)
    "cfg5-8-1024": 231.6e6,    # profiles/ffn_kernel_cfg5_G8_N1024_linear.md
}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def make_workload(name: str, rank: int = 0):
    from paper_2608_13057_b200 import workloads as W
    if name == "cfg1":
        return W.config1(seed=0 + 101 * rank)
    if name == "cfg2":
        return W.config2(seed=1 + 101 * rank)
    if name.startswith("cfg2-T"):                      # cfg2-T512: the same rank with another decode batch size
        return W.config2(seed=1 + 101 * rank, T=int(name[6:]))
    if name.startswith("cfg3-"):
        return W.config3(name[5:].replace("-", "_"), seed=2 + 101 * rank)
    if name == "cfg4":
        return W.config4(seed=3 + 101 * rank)
    if name.startswith("cfg5s-"):                      # cfg5s-G-N: same totals, uneven rows per instance
        _, G, N = name.split("-")
        return W.config5_skewed(int(G), int(N))
    if name.startswith("cfg5-"):                       # cfg5-G-N
        _, G, N = name.split("-")
        return W.config5_point(int(G), int(N))
    raise ValueError(name)


def workload_stats(wl):
    """Units of one step, from the routing and the quota table alone (host tally, not timed)."""
    live = wl.topk_ids[:wl.n_valid].reshape(-1)
    counts = np.bincount(live[(live >= 0) & (live < wl.E)], minlength=wl.E)
    rows = []
    for e in range(wl.E):
        for r in range(wl.R_max):
            if wl.replica_map[e, r] >= 0:
                rows.append(int(wl.quota[e, r]))
    rows = [m for m in rows if m > 0]
    tiles = sum(-(-m // 128) for m in rows)
    return dict(G_act=len(rows), N_local=sum(rows), tiles=tiles, M_pad=128 * tiles,
                weight_bytes=len(rows) * 3 * wl.d * wl.f, padded_flops=128 * tiles * 6 * wl.d * wl.f,
                n_valid=int(wl.n_valid), counts_total=int(counts.sum()))


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled in the background while the GPU is timed."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(gpu_index), "-lms", "100"], stdout=self.file,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.file:
            c = [v.strip() for v in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        busy = [v for v in sm if v >= 0.5 * max(sm)] or sm
        return dict(sm_mhz=float(np.median(busy)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))


# --------------------------------------------------------------------------------------------------
# CPU oracle legs (the only places bench.py touches oracle/)
# --------------------------------------------------------------------------------------------------

def oracle_sample_us_per_block(wl, budget_s: float = 15.0):
    """Times the oracle as it stands on a bounded sample: all of steps 1-2, the FFN of the first few
    activated instances (until budget_s), extrapolated over instances; plus the combine."""
    from oracle import tempo_oracle as O
    t0 = time.perf_counter()
    disp = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, wl.M_cap)
    a_q, a_s = O.permute_pad(wl.x, disp["row_pair"], disp["m_pad"], wl.k)
    t_head = time.perf_counter() - t0
    act = [i for i in range(wl.G_max) if disp["inst_count"][i] > 0]
    done, rows_done, t_ffn = 0, 0, 0.0
    y = np.zeros((len(disp["row_pair"]), wl.d), np.float32)
    for i in act:
        lo, hi = int(disp["inst_off"][i]), int(disp["inst_off"][i + 1])
        w = wl.expert_weights(int(wl.slot_expert[i]))
        t1 = time.perf_counter()
        _, _, y[lo:hi] = O.expert_ffn(a_q[lo:hi], a_s[lo:hi], w.w13_q, w.w13_s, w.w2_q, w.w2_s)
        t_ffn += time.perf_counter() - t1
        done += 1
        rows_done += hi - lo
        if t_ffn > budget_s and done >= 2:
            break
    t2 = time.perf_counter()
    O.combine(y, disp["pair_row"], wl.topk_w, min(wl.n_valid, 256), wl.T, wl.k)
    t_comb = (time.perf_counter() - t2) * max(1.0, wl.n_valid / 256.0)
    total = t_head + t_ffn * (len(act) / max(done, 1)) + t_comb
    sample = (f"steps 1-2 in full, FFN of {done} of {len(act)} activated instances ({rows_done} padded rows) "
              f"scaled by instance count, combine of {min(wl.n_valid, 256)} rows scaled by rows")
    return total * 1e6 / max(len(act), 1), sample


def run_reference(args):
    """--impl reference: the CPU oracle, timed on the host cores, same metric and workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args.workload, 0)
    wl.slot_weights()
    st = workload_stats(wl)
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample_us_per_block(wl, budget_s=2.0)
    vals, sample = [], ""
    for _ in range(max(1, min(args.steps, 3))):
        v, sample = oracle_sample_us_per_block(wl, budget_s=8.0)
        vals.append(v)
    v = float(np.mean(vals))
    cores = os.cpu_count()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
        "warmup": min(args.warmup, 1), "ms_per_step": v * st["G_act"] / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "G_act": st["G_act"], "N_local": st["N_local"]},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------------

def _capture_graphs(torch, buf, pools, run=None):
    run = buf.run_block if run is None else run
    graphs = []
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for blob in pools:
            run(packed=blob)                            # warm the launch path outside capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for blob in pools:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            run(packed=blob)
        graphs.append(g)
    return graphs


def _capture_chain(torch, buf, pools, steps, run=None):
    """One graph holding `steps` consecutive steps (weight copies in rotation), as a serving stack captures
    a whole forward pass: step i+1's first kernel launches programmatically behind step i's last one."""
    run = buf.run_block if run is None else run
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(steps):
            run(packed=pools[i % len(pools)])
    return g


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2608_13057_b200 import binding as B
    from paper_2608_13057_b200.ranks import reduce_step

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    wl = make_workload(args.workload, rank)
    st = workload_stats(wl)
    max_m = args.max_m                                 # > 0: the masked layout, instance i at rows [i*max_m, (i+1)*max_m)
    buf = B.RankBuffers.for_workload(wl, M_cap=wl.G_max * max_m if max_m else None)
    weight_bytes_all = buf.packed.numel()
    n_pools = max(2, math.ceil((1 << 30) / max(weight_bytes_all, 1)))
    n_pools = min(n_pools, 64)
    pools = [buf.packed] + [buf.packed.clone() for _ in range(n_pools - 1)]
    run_fn = (lambda packed: buf.run_block_masked(max_m, packed=packed)) if max_m else None
    graphs = _capture_graphs(torch, buf, pools, run_fn)
    K, Wm = args.steps, args.warmup

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None

    # ---- region A: the whole block as one graph replay per step, inputs resident in HBM ------------
    for i in range(Wm):
        graphs[i % n_pools].replay()
    barrier()
    # K steps exactly: whole chains of `chain_steps` steps, then single-step graphs for the remainder
    chain_steps = n_pools * max(1, 12 // n_pools)
    chain = _capture_chain(torch, buf, pools, chain_steps, run_fn) if K >= chain_steps else None
    if chain is not None:
        chain.replay()
        barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    done = 0
    while chain is not None and K - done >= chain_steps:
        chain.replay()
        done += chain_steps
    for i in range(K - done):
        graphs[i % n_pools].replay()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    status = int(buf.status.item())

    # ---- region B: the same steps launched call by call with events between the kernels -----------
    Kb = min(K, 200)
    names = ["count_dispatch", "permute_pad", "grouped_ffn", "unpermute_combine"]
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(Kb)]
    s = buf.shape
    torch.cuda._sleep(int(4e7))                        # keep the GPU busy so every launch is queued ahead
    for i in range(Kb):
        blob = pools[i % n_pools]
        ev[i][0].record()
        if max_m:
            B.tempo_count_dispatch_masked(s, max_m, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts,
                                          buf.counts, buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair,
                                          buf.tile_inst, buf.m_pad, buf.status)
            ev[i][1].record()
            B.tempo_permute_pad_masked(s, buf.x, buf.row_pair, buf.pair_row, buf.tile_inst, buf.m_pad, buf.a_q, buf.a_sf,
                                       buf.status)
            ev[i][2].record()
            B.tempo_grouped_ffn_masked(s, max_m, buf.a_q, buf.a_sf, blob, buf.inst_count, buf.h_q, buf.h_sf, buf.y,
                                       buf.status, buf.workspace)
        else:
            B.tempo_count_dispatch(s, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts, buf.counts,
                                   buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair, buf.tile_inst, buf.m_pad,
                                   buf.status)
            ev[i][1].record()
            B.tempo_permute_pad(s, buf.x, buf.row_pair, buf.m_pad, buf.a_q, buf.a_sf, buf.status, pair_row=buf.pair_row)
            ev[i][2].record()
            B.tempo_grouped_ffn(s, buf.a_q, buf.a_sf, blob, buf.inst_off, buf.m_pad, buf.h_q, buf.h_sf, buf.y,
                                buf.status, buf.workspace)
        ev[i][3].record()
        B.tempo_unpermute_combine(s, buf.y, buf.pair_row, buf.topk_w, buf.n_valid, buf.out, buf.status)
        ev[i][4].record()
    torch.cuda.synchronize()
    kern_us = {n: float(np.mean([ev[i][j].elapsed_time(ev[i][j + 1]) for i in range(Kb)])) * 1e3
               for j, n in enumerate(names)}

    # ---- e2e: host buffers in, host result out, every step ------------------------------------------
    h_ids = torch.from_numpy(wl.topk_ids).pin_memory()
    h_w = torch.from_numpy(wl.topk_w).pin_memory()
    h_x = torch.from_numpy(wl.x).to(torch.bfloat16).pin_memory()
    h_out = [torch.empty(wl.T, wl.d, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    h2d = h_ids.numel() * 4 + h_w.numel() * 4 + h_x.numel() * 2
    d2h = h_out[0].numel() * 2
    # Two sets of device buffers and three streams, as a serving loop would run it: step i+1's inputs come in
    # and step i-1's result goes out while step i computes.  Every step still pays its own copies inside the
    # timed region; PCIe carries both directions at once.
    buf2 = B.RankBuffers.for_workload(wl, M_cap=buf.M_cap, with_weights=False)
    run_fn2 = (lambda packed: buf2.run_block_masked(max_m, packed=packed)) if max_m else None
    sets = [(buf, graphs), (buf2, _capture_graphs(torch, buf2, pools, run_fn2))]
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_cmp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(i):
        j = i & 1
        b, gs = sets[j]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_cmp[j])                  # this set's previous step has read its inputs
            b.topk_ids.copy_(h_ids, non_blocking=True)
            b.topk_w.copy_(h_w, non_blocking=True)
            b.x.copy_(h_x, non_blocking=True)
            ev_in[j].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(ev_in[j])                  # the inputs are there
            s_cmp.wait_event(ev_out[j])                 # and the previous result of this set has left
            gs[i % n_pools].replay()
            ev_cmp[j].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[j])
            h_out[j].copy_(b.out, non_blocking=True)
            ev_out[j].record(s_out)

    # The same pipeline captured once: a graph of `ce` consecutive steps over the three streams (every step's
    # copies are nodes of the graph), so the host issues one launch per `ce` steps and its timing drops out.
    def capture_e2e(ce):
        g = torch.cuda.CUDAGraph()
        gi = [torch.cuda.Event() for _ in range(ce)]
        gc = [torch.cuda.Event() for _ in range(ce)]
        go = [torch.cuda.Event() for _ in range(ce)]
        with torch.cuda.graph(g):
            cur = torch.cuda.current_stream()
            s_in.wait_stream(cur)
            s_out.wait_stream(cur)
            for i in range(ce):
                b = sets[i & 1][0]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(gc[i - 2])     # this set's previous step has read its inputs
                    b.topk_ids.copy_(h_ids, non_blocking=True)
                    b.topk_w.copy_(h_w, non_blocking=True)
                    b.x.copy_(h_x, non_blocking=True)
                    gi[i].record(s_in)
                cur.wait_event(gi[i])
                if i >= 2:
                    cur.wait_event(go[i - 2])          # and its previous result has left
                if max_m:
                    b.run_block_masked(max_m, packed=pools[i % n_pools])
                else:
                    b.run_block(packed=pools[i % n_pools])
                gc[i].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(gc[i])
                    h_out[i & 1].copy_(b.out, non_blocking=True)
                    go[i].record(s_out)
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)
        return g

    Ke = min(K, 480)
    ce = 2 * n_pools * max(1, 24 // n_pools)               # steps per captured graph (even: the buffer sets alternate)
    for i in range(min(Wm, 5) + 1):
        e2e_step(i)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if Ke >= ce:
        g_e2e = capture_e2e(ce)
        g_e2e.replay()
        barrier()
        Ke = (Ke // ce) * ce
        f0.record()
        for _ in range(Ke // ce):
            g_e2e.replay()
        f1.record()
        e2e_mode = f"{ce} steps per CUDA graph, copies included"
    else:
        f0.record(s_in)
        for i in range(Ke):
            e2e_step(i)
        f1.record(s_out)
        e2e_mode = "launched step by step"
    barrier()
    ms_e2e = f0.elapsed_time(f1) / Ke
    e2e_ok = bool(torch.equal(h_out[0], h_out[1]) and torch.equal(h_out[0], buf.out.cpu()))

    clocks = sampler.stop() if sampler is not None else None

    ms_step, units = reduce_step(ms_total / K, float(st["G_act"]), "cuda" if world > 1 else None)
    ms_e2e_max, _ = reduce_step(ms_e2e, float(st["G_act"]), "cuda" if world > 1 else None)
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    peaks = _peaks()
    us_step = ms_step * 1e3
    hbm_time = st["weight_bytes"] / (peaks["hbm_gbs"] * 1e9) * 1e6
    fp8_peak = peaks["bf16_tflops_sustained"] * NOMINAL_FP8_OVER_BF16
    tensor_time = st["padded_flops"] / (fp8_peak * 1e12) * 1e6
    bound = "hbm" if hbm_time >= tensor_time else "tensor"
    # dominant kernel: the fused FFN kernel (both GEMMs of every activated instance in one launch)
    ffn_us = kern_us["grouped_ffn"]
    if bound == "hbm":
        alg = st["weight_bytes"]                                   # bytes: 3*d*f per activated instance
        achieved = alg / (ffn_us * 1e-6) / 1e9
        roof = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], traffic=NCU_TRAFFIC_BYTES.get(args.workload))
    else:
        alg = st["padded_flops"]                                   # flops: 6*d*f per padded row
        achieved = alg / (ffn_us * 1e-6) / 1e12
        roof = dict(bound="tensor", achieved=achieved, peak=fp8_peak, unit="TFLOP/s", frac=achieved / fp8_peak,
                    traffic=NCU_TRAFFIC_BYTES.get(args.workload))
    roof.update(kernel="ffn_kernel (gate/up + SwiGLU + down, one launch)", kernel_us=ffn_us, peak_source=peaks["source"] +
                (" HBM copy" if bound == "hbm" else " bf16 sustained x 2 (nominal fp8/bf16 ratio)"))

    out = {
        "metric": METRIC, "value": us_step / units, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3",
        "data": "synthetic",
        "config": {"workload": args.workload, "T": wl.T, "top_k": wl.k, "E": wl.E, "d": wl.d, "f": wl.f,
                   "G_act": st["G_act"], "N_local": st["N_local"], "M_pad": st["M_pad"],
                   "layout": f"masked, max_m={max_m}" if max_m else "grouped",
                   "graph": f"{chain_steps} consecutive steps per CUDA graph (weight copies in rotation), single-step graphs for the remainder",
                   "l2": f"weights rotate through {n_pools} copies ({n_pools * weight_bytes_all / 1e9:.2f} GB >> L2)",
                   "parallelism": f"{world} independent rank(s), no collective"},
        "block_us": us_step, "tokens_per_s": st["n_valid"] * world / (us_step * 1e-6),
        "block_roofline": {"weight_us": hbm_time, "padded_flop_us": tensor_time,
                           "frac": max(hbm_time, tensor_time) / us_step,
                           "ffn_frac": max(hbm_time, tensor_time) / kern_us["grouped_ffn"]},
        "kernel_us": kern_us, "gpu_launches": 4 * K, "device_status": status,
        "roofline": roof, "clocks": clocks,
        "e2e": {"value": ms_e2e_max * 1e3 / units, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": "two buffer sets, copy-in / compute / copy-out streams; " + e2e_mode, "steps": Ke,
                "results_identical": e2e_ok},
    }
    if world == 1 and not args.no_cpu_baseline:
        v, sample = oracle_sample_us_per_block(wl, budget_s=12.0)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample}
    print(json.dumps(out))


# --------------------------------------------------------------------------------------------------
# cost-profile sweep (config 5) and fit
# --------------------------------------------------------------------------------------------------

def run_sweep(args):
    import torch
    from paper_2608_13057_b200 import binding as B
    from paper_2608_13057_b200 import costmodel as C
    from paper_2608_13057_b200 import workloads as W

    torch.cuda.set_device(0)
    d, f = 4096, 1536
    Gs = [int(g) for g in args.sweep_G.split(",")] if args.sweep_G else list(W.SWEEP_G)
    Ns = [int(n) for n in args.sweep_N.split(",")] if args.sweep_N else list(W.SWEEP_N)
    replays = args.replays
    rows = []
    gen = torch.Generator(device="cuda").manual_seed(4)
    for G in Gs:
        # one weight set per G, copied into a rotation pool >> L2
        wl0 = W.config5_point(G, 1, with_x=False)
        probe = B.RankBuffers(G, 1, G, G, 1, d, f)
        bf16 = args.variant == "bf16"
        packed = probe.pack_weights_bf16(*wl0.slot_weights_bf16()) if bf16 else probe.pack_weights(*wl0.slot_weights())
        n_pools = min(64, max(2, math.ceil((1 << 30) / packed.numel())))
        pools = [packed] + [packed.clone() for _ in range(n_pools - 1)]
        del probe
        for N in Ns:
            T = G * N
            buf = B.RankBuffers(T, 1, G, G, 1, d, f)
            buf.topk_ids.copy_((torch.arange(T, device="cuda", dtype=torch.int32) % G).view(T, 1))
            buf.topk_w.fill_(1.0)
            buf.replica_map.copy_(torch.arange(G, device="cuda", dtype=torch.int32).view(G, 1))
            buf.quota.fill_(N)
            buf.x.copy_(torch.randn(T, d, generator=gen, device="cuda").to(torch.bfloat16))
            if bf16:
                buf.alloc_bf16()
            graphs = _capture_graphs(torch, buf, pools, buf.run_block_bf16 if bf16 else None)
            s = buf.shape
            ffn_graphs = []
            for blob in pools:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    if bf16:
                        B.tempo_grouped_ffn_bf16(s, buf.a_bf16, blob, buf.inst_off, buf.m_pad, buf.h_bf16, buf.y,
                                                 buf.status, buf.workspace)
                    else:
                        B.tempo_grouped_ffn(s, buf.a_q, buf.a_sf, blob, buf.inst_off, buf.m_pad, buf.h_q, buf.h_sf,
                                            buf.y, buf.status, buf.workspace)
                ffn_graphs.append(g)

            def med(gs):
                ts = []
                for i in range(3):
                    gs[i % n_pools].replay()
                for i in range(replays):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    gs[i % n_pools].replay()
                    b.record()
                    b.synchronize()
                    ts.append(a.elapsed_time(b) * 1e3)
                return float(np.median(ts)), float(np.percentile(ts, 10)), float(np.percentile(ts, 90))

            t_block, b10, b90 = med(graphs)
            t_ffn, f10, f90 = med(ffn_graphs)
            tiles = G * (-(-N // 128))
            rows.append(dict(G=G, n=N, N=G * N, tiles=tiles, t_block_us=t_block, t_ffn_us=t_ffn, block_p10=b10,
                             block_p90=b90, ffn_p10=f10, ffn_p90=f90, status=int(buf.status.item())))
            print(json.dumps(rows[-1]), file=sys.stderr, flush=True)
            del buf, graphs, ffn_graphs
            torch.cuda.empty_cache()
        del pools, packed
        torch.cuda.empty_cache()
    G = np.array([r["G"] for r in rows])
    N = np.array([r["N"] for r in rows])
    tiles = np.array([r["tiles"] for r in rows])
    result = {"sweep": {"d": d, "f": f, "points": len(rows), "replays": replays, "variant": args.variant}, "rows": rows}
    for scope in ("ffn", "block"):
        t = np.array([r[f"t_{scope}_us"] for r in rows])
        result[f"fit_{scope}"] = C.fit_max_affine(G, N, t)
        result[f"fit_{scope}_tile"] = C.fit_max_affine(G, N, t, tiles=tiles, tile_aware=True)
    print(json.dumps(result))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--sweep-G", default="")
    ap.add_argument("--sweep-N", default="")
    ap.add_argument("--replays", type=int, default=30)
    ap.add_argument("--variant", default="fp8", choices=["fp8", "bf16"], help="--sweep only: which steps 2 and 3")
    ap.add_argument("--max-m", type=int, default=0, help="> 0: run the block in the masked layout with this row stride")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
