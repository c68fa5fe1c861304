#!/usr/bin/env python
"""Benchmark of the per-rank MoE expert block on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3-uniform|cfg4|...] [--impl reference]
    python bench.py --sweep            # full cost-profile sweep (G, N grid) + max-affine fit -> n*

One "step" is one pass of the whole hot path (count+dispatch, activation quantise/permute, the fused gate/up +
SwiGLU + down FFN kernel, combine) over one seeded synthetic routed batch, replayed from CUDA graphs.  Weight
copies rotate through a pool larger than L2 so no step finds its weights cached (the paper's calibration
protocol, Appendix B).  Rank 0 prints ONE JSON line.  The default line is quoted on config 2 (the flat,
HBM-bound regime) and, at one GPU, carries the rest of the metric as well: `regimes.linear` (config 4, the
tensor-bound regime), `fit` (Eq. 1 / Eq. 3 fitted to a reduced in-run sweep, with the B200 n*), and a dense fp8
GEMM rate measured in the same run as the tensor-bound denominator.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import re
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
NOMINAL_FP8_TFLOPS = 4500.0
POOL_BYTES = 1 << 30                    # weight copies rotate through at least this much (>> L2)
FIT_G = (4, 16, 64)                     # reduced in-run sweep behind `fit` (the full grid: --sweep)
FIT_N = (64, 128, 129, 256, 1024, 4096)

# ncu summary (profiles/) that holds dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant
# kernel for a workload, on a line "dram_bytes_per_launch: <number>"; None where no capture exists.
NCU_SUMMARY = {
    "cfg2": "ffn_kernel_cfg2_flat_decode.md",
    "cfg5-8-1024": "ffn_kernel_cfg5_G8_N1024_linear.md",
}


def ncu_traffic_bytes(workload: str):
    name = NCU_SUMMARY.get(workload)
    if name is None:
        return None
    try:
        text = open(os.path.join(ROOT, "profiles", name)).read()
    except OSError:
        return None
    m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", text)
    return float(m.group(1)) if m else None


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


def n_pools_for(weight_bytes_all: int) -> int:
    return min(64, max(2, math.ceil(POOL_BYTES / max(weight_bytes_all, 1))))


def workload_config(name, wl, st, world, max_m=0):
    """The `config` object of the JSON line: the workload and how L2 is defeated.  Both arms print the same."""
    packed_bytes = wl.G_max * 3 * wl.d * wl.f            # + 0.8 % scale atoms
    pools = n_pools_for(packed_bytes)
    return {"workload": name, "T": wl.T, "top_k": wl.k, "E": wl.E, "d": wl.d, "f": wl.f, "G_act": st["G_act"],
            "N_local": st["N_local"], "M_pad": st["M_pad"], "layout": f"masked, max_m={max_m}" if max_m else "grouped",
            "l2": f"weights rotate through {pools} copies of {packed_bytes / 1e9:.2f} GB each (>> 126 MB L2)",
            "parallelism": f"{world} independent rank(s), no collective"}


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled in the background while the GPU is timed."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(gpu_index), "-lms", "20"], stdout=self.file,
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
        sm, mx, pw, reasons = [], [], [], set()
        for line in self.file:
            c = [v.strip() for v in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
                pw.append(float(c[3]))
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
        return dict(sm_mhz=float(np.median(busy)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm),
                    power_w_max=float(max(pw)) if pw else None)


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
        "config": workload_config(args.workload, wl, st, max(1, args.gpus), args.max_m),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------------

def _pct(ts):
    return dict(p10=float(np.percentile(ts, 10)), p50=float(np.percentile(ts, 50)), p90=float(np.percentile(ts, 90)))


def _capture_graphs(torch, pools, run):
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


def _capture_chain(torch, pools, steps, run):
    """One graph holding `steps` consecutive steps (weight copies in rotation), as a serving stack captures
    a whole forward pass: step i+1's first kernel launches programmatically behind step i's last one."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(steps):
            run(packed=pools[i % len(pools)])
    return g


def measure_fp8_peak(torch, seconds: float = 3.0):
    """Dense e4m3 GEMM rate of the vendor library (torch._scaled_mm, 8192^3, per-tensor scales, bf16 out):
    best of 10 launches (burst) and a back-to-back loop of about `seconds` (sustained, under the power cap).
    A denominator for the tensor-bound roofline only; nothing on the hot path calls it."""
    try:
        n = 8192
        a = (torch.randn(n, n, device="cuda") * 0.5).to(torch.float8_e4m3fn)
        b = (torch.randn(n, n, device="cuda") * 0.5).to(torch.float8_e4m3fn).t()      # column-major operand
        one = torch.ones((), device="cuda", dtype=torch.float32)

        def mm():
            return torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)

        for _ in range(3):
            mm()
        torch.cuda.synchronize()
        flops = 2.0 * n ** 3
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            mm()
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        reps = max(10, int(seconds * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            mm()
        e1.record()
        e1.synchronize()
        sustained = e0.elapsed_time(e1) / reps
        return dict(fp8_tflops=flops / best / 1e9, fp8_tflops_sustained=flops / sustained / 1e9,
                    how=f"torch._scaled_mm e4m3 x e4m3 -> bf16, {n}^3, best of 10 and {reps} back to back "
                        f"({e0.elapsed_time(e1) / 1e3:.1f} s)")
    except Exception as exc:                             # no fp8 GEMM in this torch build: fall back to 2 x bf16
        return dict(fp8_tflops=None, fp8_tflops_sustained=None, how=f"unavailable: {type(exc).__name__}: {exc}"[:200])


def tensor_denominators(peaks, fp8):
    """TFLOP/s figures a tensor-bound fraction can be quoted against; the first available one is primary."""
    d = {}
    if fp8 and fp8.get("fp8_tflops_sustained"):
        d["fp8_measured_sustained"] = fp8["fp8_tflops_sustained"]
        d["fp8_measured_burst"] = fp8["fp8_tflops"]
    d["bf16_sustained_x2"] = peaks["bf16_tflops_sustained"] * NOMINAL_FP8_OVER_BF16
    d["bf16_burst_x2"] = peaks["bf16_tflops"] * NOMINAL_FP8_OVER_BF16
    d["nominal_dense_fp8"] = NOMINAL_FP8_TFLOPS
    return d


class Leg:
    """One workload on the device: buffers, weight copies, graphs, and the timed regions."""

    def __init__(self, torch, B, name, wl, max_m=0, device_weights=False, path="permute"):
        from paper_2608_13057_b200 import workloads as W
        self.torch, self.B, self.name, self.wl, self.max_m = torch, B, name, wl, max_m
        self.path = "permute" if max_m else path         # "gather": tempo_quantize_tokens + tempo_grouped_ffn_gather
        self.st = workload_stats(wl)
        M_cap = wl.G_max * max_m if max_m else None
        if device_weights:
            self.buf = B.RankBuffers.for_workload(wl, M_cap=M_cap, with_weights=False)
            self.buf.pack_weights(*W.slot_weights_cuda(wl))
            torch.cuda.empty_cache()
        else:
            self.buf = B.RankBuffers.for_workload(wl, M_cap=M_cap)
        buf = self.buf
        self.n_pools = n_pools_for(buf.packed.numel())
        self.pools = [buf.packed] + [buf.packed.clone() for _ in range(self.n_pools - 1)]
        self.run = self.runner(buf)
        self.graphs = _capture_graphs(torch, self.pools, self.run)
        self.chain_steps = self.n_pools * max(1, 12 // self.n_pools)
        self.chain = None

    def runner(self, buf):
        if self.max_m:
            return lambda packed: buf.run_block_masked(self.max_m, packed=packed)
        return buf.run_block_gather if self.path == "gather" else buf.run_block

    def replay_steps(self, K):
        """Exactly K steps: whole chains of `chain_steps` steps, then single-step graphs for the remainder."""
        done = 0
        while self.chain is not None and K - done >= self.chain_steps:
            self.chain.replay()
            done += self.chain_steps
        for i in range(K - done):
            self.graphs[i % self.n_pools].replay()

    def time_regions(self, K, warmup, regions, barrier):
        torch = self.torch
        for i in range(warmup):
            self.graphs[i % self.n_pools].replay()
        barrier()
        if K >= self.chain_steps and self.chain is None:
            self.chain = _capture_chain(torch, self.pools, self.chain_steps, self.run)
            self.chain.replay()
            barrier()
        ms = []
        for _ in range(regions):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record()
            self.replay_steps(K)
            e1.record()
            barrier()
            ms.append(e0.elapsed_time(e1))
        return ms

    def kernel_pass(self, Kb):
        """The same steps launched call by call with events between the kernels (queued behind a spin kernel so
        that no launch is late): per-kernel CUDA-event durations on the launching stream."""
        torch, B, buf, max_m = self.torch, self.B, self.buf, self.max_m
        gather = self.path == "gather"
        names = ["count_dispatch", "quantize_tokens" if gather else "permute_pad", "grouped_ffn", "unpermute_combine"]
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(Kb)]
        s = buf.shape
        torch.cuda._sleep(int(4e7))
        for i in range(Kb):
            blob = self.pools[i % self.n_pools]
            ev[i][0].record()
            if max_m:
                B.tempo_count_dispatch_masked(s, max_m, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota,
                                              buf.cum_counts, buf.counts, buf.inst_count, buf.inst_off, buf.pair_row,
                                              buf.row_pair, buf.tile_inst, buf.m_pad, buf.status)
                ev[i][1].record()
                B.tempo_permute_pad_masked(s, buf.x, buf.row_pair, buf.pair_row, buf.tile_inst, buf.m_pad, buf.a_q,
                                           buf.a_sf, buf.status)
                ev[i][2].record()
                B.tempo_grouped_ffn_masked(s, max_m, buf.a_q, buf.a_sf, blob, buf.inst_count, buf.h_q, buf.h_sf, buf.y,
                                           buf.status, buf.workspace)
            else:
                B.tempo_count_dispatch(s, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts,
                                       buf.counts, buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair,
                                       buf.tile_inst, buf.m_pad, buf.status)
                ev[i][1].record()
                if gather:
                    B.tempo_quantize_tokens(s, buf.x, buf.n_valid, buf.x_q, buf.x_sf, buf.status)
                    ev[i][2].record()
                    B.tempo_grouped_ffn_gather(s, buf.x_q, buf.x_sf, buf.row_pair, blob, buf.inst_off, buf.m_pad,
                                               buf.h_q, buf.h_sf, buf.y, buf.status, buf.workspace)
                else:
                    B.tempo_permute_pad(s, buf.x, buf.row_pair, buf.m_pad, buf.a_q, buf.a_sf, buf.status,
                                        pair_row=buf.pair_row)
                    ev[i][2].record()
                    B.tempo_grouped_ffn(s, buf.a_q, buf.a_sf, blob, buf.inst_off, buf.m_pad, buf.h_q, buf.h_sf, buf.y,
                                        buf.status, buf.workspace)
            ev[i][3].record()
            B.tempo_unpermute_combine(s, buf.y, buf.pair_row, buf.topk_w, buf.n_valid, buf.out, buf.status)
            ev[i][4].record()
        torch.cuda.synchronize()
        return {n: float(np.median([ev[i][j].elapsed_time(ev[i][j + 1]) for i in range(Kb)])) * 1e3
                for j, n in enumerate(names)}

    def ffn_chained(self, regions, barrier):
        """The dominant kernel alone, the way it runs inside the block: a CUDA graph of `chain_steps` consecutive
        FFN launches (weight copies in rotation, the block's own activations), each launch's prologue overlapping
        its predecessor's tail by programmatic dependent launch; events bracket the whole graph, so the per-launch
        figure carries no event or launch gap.  Median over `regions` replays of (graph time / launches)."""
        torch, B, buf, s = self.torch, self.B, self.buf, self.buf.shape
        gather = self.path == "gather"

        def ffn(blob):
            if self.max_m:
                B.tempo_grouped_ffn_masked(s, self.max_m, buf.a_q, buf.a_sf, blob, buf.inst_count, buf.h_q, buf.h_sf,
                                           buf.y, buf.status, buf.workspace)
            elif gather:
                B.tempo_grouped_ffn_gather(s, buf.x_q, buf.x_sf, buf.row_pair, blob, buf.inst_off, buf.m_pad, buf.h_q,
                                           buf.h_sf, buf.y, buf.status, buf.workspace)
            else:
                B.tempo_grouped_ffn(s, buf.a_q, buf.a_sf, blob, buf.inst_off, buf.m_pad, buf.h_q, buf.h_sf, buf.y,
                                    buf.status, buf.workspace)

        n = self.chain_steps
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n):
                ffn(self.pools[i % self.n_pools])
        g.replay()
        barrier()
        us = []
        for _ in range(regions):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            e1.synchronize()
            us.append(e0.elapsed_time(e1) * 1e3 / n)
        return float(np.median(us))

    def rooflines(self, us_step, kern_us, peaks, fp8):
        """`roofline` (the dominant kernel) and `block_roofline` (the whole step) of this leg."""
        st = self.st
        denoms = tensor_denominators(peaks, fp8)
        primary = next(iter(denoms))
        fp8_peak = denoms[primary]
        hbm_time = st["weight_bytes"] / (peaks["hbm_gbs"] * 1e9) * 1e6
        tensor_time = st["padded_flops"] / (fp8_peak * 1e12) * 1e6
        bound = "hbm" if hbm_time >= tensor_time else "tensor"
        ffn_us = kern_us.get("grouped_ffn_chained", kern_us["grouped_ffn"])
        if bound == "hbm":
            achieved = st["weight_bytes"] / (ffn_us * 1e-6) / 1e9             # bytes: 3*d*f per activated instance
            roof = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=achieved / peaks["hbm_gbs"], traffic=ncu_traffic_bytes(self.name),
                        peak_source=peaks["source"] + " HBM copy (MEASURED_PEAKS.json)")
        else:
            achieved = st["padded_flops"] / (ffn_us * 1e-6) / 1e12            # flops: 6*d*f per padded row
            roof = dict(bound="tensor", achieved=achieved, peak=fp8_peak, unit="TFLOP/s", frac=achieved / fp8_peak,
                        traffic=ncu_traffic_bytes(self.name),
                        peak_source=f"{primary}: " + (fp8["how"] if primary.startswith("fp8_measured") else
                                                      peaks["source"] + " bf16 GEMM rate x 2 (nominal fp8/bf16 ratio)"),
                        frac_vs={k: achieved / v for k, v in denoms.items()})
        roof.update(kernel="ffn_kernel (gate/up + SwiGLU + down, one launch)", kernel_us=ffn_us,
                    kernel_us_how="graph of consecutive launches of this kernel, events around the graph, per launch"
                    if "grouped_ffn_chained" in kern_us else "one launch between two events")
        block = {"weight_us": hbm_time, "padded_flop_us": tensor_time, "bound": bound,
                 "frac": max(hbm_time, tensor_time) / us_step, "ffn_frac": max(hbm_time, tensor_time) / ffn_us,
                 "tensor_peak": primary}
        if bound == "tensor":
            block["frac_vs"] = {k: max(hbm_time, st["padded_flops"] / (v * 1e12) * 1e6) / us_step
                                for k, v in denoms.items()}
        return roof, block


def measure_e2e(torch, B, leg, K, warmup, barrier):
    """Host buffers in, host result out, every step: two sets of device buffers and three streams, as a serving
    loop would run it (step i+1's inputs come in and step i-1's result goes out while step i computes), captured
    into CUDA graphs of `ce` steps, copies included.  Every step pays its own copies inside the timed region."""
    wl, buf, pools, n_pools, max_m = leg.wl, leg.buf, leg.pools, leg.n_pools, leg.max_m
    h_ids = torch.from_numpy(wl.topk_ids).pin_memory()
    h_w = torch.from_numpy(wl.topk_w).pin_memory()
    h_x = torch.from_numpy(wl.x).to(torch.bfloat16).pin_memory()
    h_out = [torch.empty(wl.T, wl.d, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    h2d = h_ids.numel() * 4 + h_w.numel() * 4 + h_x.numel() * 2
    d2h = h_out[0].numel() * 2
    buf2 = B.RankBuffers.for_workload(wl, M_cap=buf.M_cap, with_weights=False)
    sets = [buf, buf2]
    runs = [leg.runner(buf), leg.runner(buf2)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def capture(ce):
        g = torch.cuda.CUDAGraph()
        gi = [torch.cuda.Event() for _ in range(ce)]
        gc = [torch.cuda.Event() for _ in range(ce)]
        go = [torch.cuda.Event() for _ in range(ce)]
        with torch.cuda.graph(g):
            cur = torch.cuda.current_stream()
            s_in.wait_stream(cur)
            s_out.wait_stream(cur)
            for i in range(ce):
                b = sets[i & 1]
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
                runs[i & 1](packed=pools[i % n_pools])
                gc[i].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(gc[i])
                    h_out[i & 1].copy_(b.out, non_blocking=True)
                    go[i].record(s_out)
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)
        return g

    Ke = max(2, min(K, 480))
    ce = min(2 * n_pools * max(1, 24 // n_pools), (Ke // 2) * 2)     # steps per graph, even: the buffer sets alternate
    # warm the launch path of the second buffer set outside capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        runs[1](packed=pools[0])
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g_e2e = capture(ce)
    for _ in range(max(1, min(warmup, 3))):
        g_e2e.replay()
    barrier()
    Ke = (Ke // ce) * ce
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(Ke // ce):
        g_e2e.replay()
    f1.record()
    barrier()
    ms = f0.elapsed_time(f1) / Ke
    ok = bool(torch.equal(h_out[0], h_out[1]) and torch.equal(h_out[0], buf.out.cpu()))
    del buf2
    return dict(ms=ms, steps=Ke, h2d=h2d, d2h=d2h, identical=ok,
                mode=f"two buffer sets, copy-in / compute / copy-out streams; {ce} steps per CUDA graph, copies included")


def sweep_rows(torch, B, Gs, Ns, replays, variant="fp8", device_weights=False, log=None):
    """(G, N) points of config 5: G instances of the Qwen3-235B expert shape with N rows each; per point the
    median / p10 / p90 over `replays` single-step graph replays of the whole block and of the FFN kernel alone."""
    from paper_2608_13057_b200 import workloads as W
    d, f = 4096, 1536
    bf16 = variant == "bf16"
    rows = []
    gen = torch.Generator(device="cuda").manual_seed(4)
    for G in Gs:
        wl0 = W.config5_point(G, 1, with_x=False)        # one weight set per G, copied into a rotation pool >> L2
        probe = B.RankBuffers(G, 1, G, G, 1, d, f)
        if bf16:
            packed = probe.pack_weights_bf16(*wl0.slot_weights_bf16())
        elif device_weights:
            packed = probe.pack_weights(*W.slot_weights_cuda(wl0))
        else:
            packed = probe.pack_weights(*wl0.slot_weights())
        n_pools = n_pools_for(packed.numel())
        pools = [packed] + [packed.clone() for _ in range(n_pools - 1)]
        del probe
        torch.cuda.empty_cache()
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
            graphs = _capture_graphs(torch, pools, buf.run_block_bf16 if bf16 else buf.run_block)
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
            if log is not None:
                print(json.dumps(rows[-1]), file=log, flush=True)
            del buf, graphs, ffn_graphs
            torch.cuda.empty_cache()
        del pools, packed
        torch.cuda.empty_cache()
    return rows


def fit_rows(rows):
    from paper_2608_13057_b200 import costmodel as C
    G = np.array([r["G"] for r in rows])
    N = np.array([r["N"] for r in rows])
    tiles = np.array([r["tiles"] for r in rows])
    out = {}
    for scope in ("ffn", "block"):
        t = np.array([r[f"t_{scope}_us"] for r in rows])
        out[f"fit_{scope}"] = C.fit_max_affine(G, N, t)
        out[f"fit_{scope}_tile"] = C.fit_max_affine(G, N, t, tiles=tiles, tile_aware=True)
    return out


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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K, Wm, R = args.steps, args.warmup, max(1, args.replays)
    wl = make_workload(args.workload, rank)
    leg = Leg(torch, B, args.workload, wl, max_m=args.max_m, path=args.path, device_weights=args.device_weights)
    st = leg.st
    sampler = ClockSampler(local) if rank == 0 else None

    # ---- region A: R timed regions of exactly K steps each, inputs resident in HBM ------------------
    ms_regions = leg.time_regions(K, Wm, R, barrier)
    status = int(leg.buf.status.item())
    # ---- region B: per-kernel durations ---------------------------------------------------------------
    kern_us = leg.kernel_pass(min(K, 200))
    kern_us["grouped_ffn_chained"] = leg.ffn_chained(R, barrier)
    # ---- e2e ------------------------------------------------------------------------------------------------
    try:
        e2e = measure_e2e(torch, B, leg, K, Wm, barrier)
    except Exception as exc:                              # keep the resident-input figure if the host path fails
        e2e = dict(ms=float("nan"), steps=0, h2d=0, d2h=0, identical=False, mode=f"failed: {type(exc).__name__}: {exc}"[:300])
    clocks = sampler.stop() if sampler is not None else None

    step_ms = [m / K for m in ms_regions]
    ms_step, units = reduce_step(float(np.median(step_ms)), float(st["G_act"]), "cuda" if world > 1 else None)
    ms_e2e_max, _ = reduce_step(e2e["ms"], float(st["G_act"]), "cuda" if world > 1 else None)

    extras = world == 1 and not args.no_extras and args.workload == "cfg2" and not args.max_m
    linear = fit = fp8 = None
    extras_errors = {}
    if extras:
        # Each extra leg stands on its own: a failure in one is reported in the line, it does not cost the others
        # or the headline figure measured above.
        del leg.graphs, leg.chain, leg.pools
        torch.cuda.empty_cache()
        try:        # ---- the tensor-bound regime: config 4, the largest single-GPU configuration
            wl4 = make_workload("cfg4", 0)
            leg4 = Leg(torch, B, "cfg4", wl4, device_weights=True, path=args.path)
            sampler4 = ClockSampler(local)
            K4 = leg4.chain_steps
            ms4 = leg4.time_regions(K4, 3, R, barrier)
            kern4 = leg4.kernel_pass(24)
            kern4["grouped_ffn_chained"] = leg4.ffn_chained(R, barrier)
            clocks4 = sampler4.stop()
            status4 = int(leg4.buf.status.item())
            linear = dict(leg=leg4, ms=ms4, K=K4, kern=kern4, clocks=clocks4, status=status4)
            del leg4.graphs, leg4.chain, leg4.pools
            torch.cuda.empty_cache()
        except Exception as exc:
            extras_errors["linear"] = f"{type(exc).__name__}: {exc}"[:300]
        try:        # ---- reduced cost-profile sweep -> fit
            rows = sweep_rows(torch, B, FIT_G, FIT_N, max(10, min(R, 30)), device_weights=True)
            fit = dict(rows=rows, **fit_rows(rows))
        except Exception as exc:
            extras_errors["fit"] = f"{type(exc).__name__}: {exc}"[:300]
        fp8 = measure_fp8_peak(torch)        # dense fp8 GEMM rate of the vendor library, as a denominator
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    peaks = _peaks()
    us_step = ms_step * 1e3
    roof, block = leg.rooflines(us_step, kern_us, peaks, fp8)
    pct = _pct([m * 1e3 for m in step_ms])
    out = {
        "metric": METRIC, "value": us_step / units, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3",
        "data": "synthetic",
        "config": workload_config(args.workload, wl, st, world, args.max_m),
        "path": leg.path,
        "timing": {"regions": R, "steps_per_region": K, "statistic": "median over regions of (region time / K)",
                   "graph": f"{leg.chain_steps} consecutive steps per CUDA graph (weight copies in rotation), "
                            "single-step graphs for the remainder"},
        "block_us": us_step, "block_us_percentiles": pct, "tokens_per_s": st["n_valid"] * world / (us_step * 1e-6),
        "block_roofline": block, "kernel_us": kern_us, "gpu_launches": 4 * K, "device_status": status,
        "roofline": roof, "clocks": clocks,
        "e2e": {"value": None if math.isnan(ms_e2e_max) else ms_e2e_max * 1e3 / units, "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                "d2h_bytes_per_step": e2e["d2h"], "pipeline": e2e["mode"], "steps": e2e["steps"],
                "results_identical": e2e["identical"]},
    }
    if extras_errors:
        out["extras_errors"] = extras_errors
    if extras and linear is not None:
        l4 = linear["leg"]
        step4 = [m / linear["K"] * 1e3 for m in linear["ms"]]
        us4 = float(np.median(step4))
        roof4, block4 = l4.rooflines(us4, linear["kern"], peaks, fp8)
        out["regimes"] = {
            "flat": {"workload": args.workload, "block_us": us_step, "bound": block["bound"], "block_frac": block["frac"],
                     "ffn_frac": roof["frac"]},
            "linear": {"workload": "cfg4", "config": workload_config("cfg4", l4.wl, l4.st, 1),
                       "weights": "drawn on the device (same distribution and scale rule; timing only)",
                       "value": us4 / l4.st["G_act"], "unit": UNIT, "block_us": us4, "block_us_percentiles": _pct(step4),
                       "steps_per_region": linear["K"], "regions": R, "tokens_per_s": l4.st["n_valid"] / (us4 * 1e-6),
                       "kernel_us": linear["kern"], "roofline": roof4, "block_roofline": block4,
                       "clocks": linear["clocks"], "device_status": linear["status"]},
        }
    if extras and fit is not None:
        keep = ("a", "b", "b2", "c", "beta", "n_star", "fit_err", "n_flat", "n_linear")
        out["fit"] = {"grid": {"G": list(FIT_G), "N_per_instance": list(FIT_N), "d": 4096, "f": 1536,
                               "replays": max(10, min(R, 30))},
                      "n_star": fit["fit_ffn_tile"]["n_star"],
                      **{k: {kk: fit[k][kk] for kk in keep} for k in ("fit_ffn", "fit_ffn_tile", "fit_block", "fit_block_tile")},
                      "points": [{k: r[k] for k in ("G", "n", "t_ffn_us", "t_block_us")} for r in fit["rows"]]}
    if extras:
        out["measured_fp8"] = fp8
    if world == 1 and not args.no_cpu_baseline and not args.device_weights:
        v, sample = oracle_sample_us_per_block(wl, budget_s=12.0)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample}
    print(json.dumps(out))


# --------------------------------------------------------------------------------------------------
# cost-profile sweep (config 5) and fit
# --------------------------------------------------------------------------------------------------

def run_sweep(args):
    import torch
    from paper_2608_13057_b200 import binding as B
    from paper_2608_13057_b200 import workloads as W

    torch.cuda.set_device(0)
    Gs = [int(g) for g in args.sweep_G.split(",")] if args.sweep_G else list(W.SWEEP_G)
    Ns = [int(n) for n in args.sweep_N.split(",")] if args.sweep_N else list(W.SWEEP_N)
    rows = sweep_rows(torch, B, Gs, Ns, args.replays, args.variant, device_weights=args.variant == "fp8", log=sys.stderr)
    result = {"sweep": {"d": 4096, "f": 1536, "points": len(rows), "replays": args.replays, "variant": args.variant},
              "rows": rows}
    result.update(fit_rows(rows))
    print(json.dumps(result))


# --------------------------------------------------------------------------------------------------
# dispatch policies on the mixed-regime batch: modelled against measured (closes the solver loop)
# --------------------------------------------------------------------------------------------------

def run_policies(args):
    """Config 3's routed batch under five dispatch policies (uniform, token-balanced, keep-hot-whole, the table
    tempo_fast builds from the cost profile fitted IN THIS RUN, and the same solved on the previous window's counts
    as the deployed system does): for each, the block time of the rank
    that holds all 20 slots and of the two virtual GPUs (16 primaries / 4 replica slots) the solver balances,
    measured on this GPU one after the other, next to what the fitted Eq. 3 profile predicts."""
    import torch
    from paper_2608_13057_b200 import binding as B
    from paper_2608_13057_b200 import policies as P
    from paper_2608_13057_b200 import solver as S

    torch.cuda.set_device(0)

    def barrier():
        torch.cuda.synchronize()

    if args.fit_json:
        fit = json.load(open(args.fit_json))
        fit = fit.get("fit", fit)["fit_block_tile"]
    else:
        rows = sweep_rows(torch, B, FIT_G, FIT_N, max(10, min(args.replays, 30)), device_weights=True)
        fit = fit_rows(rows)["fit_block_tile"]
    params = S.CostParams(a=fit["a"], b=fit["b"], c=fit["c"], beta=fit["beta"], b2=fit["b2"])
    K, R = args.steps, max(1, args.replays)
    out = {"policies": [], "fit_block_tile": {k: fit[k] for k in ("a", "b", "b2", "c", "beta", "n_star", "fit_err")},
           "workload": "cfg3 routed batch (T=4096, top-8, Zipf 1.2), 16 primaries on virtual GPU A, replicas of the "
                       "4 hottest on virtual GPU B", "steps_per_region": K, "regions": R}
    for case in P.build_cases(params):
        m = P.modeled(case.x, params)
        meas = {}
        for key, wl in (("rank", case.rank), ("gpu_a", case.gpus[0]), ("gpu_b", case.gpus[1])):
            leg = Leg(torch, B, wl.name, wl, device_weights=True, path=args.path)
            ms = leg.time_regions(K, 3, R, barrier)
            status = int(leg.buf.status.item())
            # the quota table is honoured exactly: every instance holds the rows the policy gave it
            want = np.zeros(wl.G_max, np.int64)
            if key == "rank":
                want[:] = case.rank_rows                # what the (renormalised, if stale) table must give
            else:
                for e in range(wl.E):
                    if wl.replica_map[e, 0] >= 0:
                        want[wl.replica_map[e, 0]] = wl.quota[e, 0]
            exact = bool(np.array_equal(leg.buf.inst_count.cpu().numpy(), want))
            meas[key] = dict(us=float(np.median(ms)) / K * 1e3, status=status, quotas_exact=exact, G_act=leg.st["G_act"],
                             N=leg.st["N_local"], tiles=leg.st["tiles"])
            del leg
            torch.cuda.empty_cache()
        hot = [[int(a), int(b)] for a, b in case.x if b > 0]
        out["policies"].append(dict(policy=case.name, hot_splits=hot, modeled_us=m,
                                    measured_us=dict(gpu_us=[meas["gpu_a"]["us"], meas["gpu_b"]["us"]],
                                                     makespan_us=max(meas["gpu_a"]["us"], meas["gpu_b"]["us"]),
                                                     rank_us=meas["rank"]["us"]),
                                    detail=meas))
    # Does the offline profile transfer to these deployment-like batches?  (Section 5.2: the paper refits the profile on
    # the records of its microbenchmark and compares it with the offline one.)
    from paper_2608_13057_b200 import costmodel as C
    legs = [v for p in out["policies"] for v in p["detail"].values() if v["G_act"] > 0]
    Gs, Ns, Ts, ts = (np.array([v[k] for v in legs], dtype=np.float64) for k in ("G_act", "N", "tiles", "us"))
    pred = C.block_time(params.a, params.b, params.c, params.beta, Gs, Ns, params.b2, Ts)
    out["transfer"] = {"legs": len(legs), "offline_profile_mean_abs_err": float(np.mean(np.abs(pred - ts) / ts)),
                       "offline_profile_mean_signed_err": float(np.mean((pred - ts) / ts)),
                       "records": [dict(G=int(g), N=int(n), tiles=int(t_), us=float(u)) for g, n, t_, u in zip(Gs, Ns, Ts, ts)]}
    mk = [p["measured_us"]["makespan_us"] for p in out["policies"]]
    md = [p["modeled_us"]["makespan_us"] for p in out["policies"]]
    out["spread"] = {"measured_worst_over_best": max(mk) / min(mk), "modeled_worst_over_best": max(md) / min(md),
                     "measured_best": out["policies"][int(np.argmin(mk))]["policy"],
                     "modeled_best": out["policies"][int(np.argmin(md))]["policy"]}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the linear-regime leg, the in-run fit and the fp8 GEMM rate of the default line")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--policies", action="store_true",
                    help="config 3 under four dispatch policies: modelled (fit of this run) against measured")
    ap.add_argument("--fit-json", default="", help="--policies: take fit_block_tile from this bench line instead")
    ap.add_argument("--sweep-G", default="")
    ap.add_argument("--sweep-N", default="")
    ap.add_argument("--replays", type=int, default=30, help="timed regions of K steps each (sweep: replays per point)")
    ap.add_argument("--variant", default="fp8", choices=["fp8", "bf16"], help="--sweep only: which steps 2 and 3")
    ap.add_argument("--path", default="permute", choices=["permute", "gather"],
                    help="steps 2-3: tempo_permute_pad + tempo_grouped_ffn, or tempo_quantize_tokens + "
                         "tempo_grouped_ffn_gather (same results bit for bit)")
    ap.add_argument("--device-weights", action="store_true",
                    help="draw the weights on the device (timing only; minutes faster for the large shapes)")
    ap.add_argument("--max-m", type=int, default=0, help="> 0: run the block in the masked layout with this row stride")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    elif args.policies:
        run_policies(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
