#!/usr/bin/env python
"""Benchmark of the RMM hot path on B200.

A step is one pass of the whole hot path over one product: scores of A, top-k selection, gathers and the
reduced product Y = A[:, I] B[I, :] (rmm_product).  Workload at N = 1: the 70B-class MLP down projection, the
largest single-GPU product of the benchmark configurations (A 32768 tokens x 28672 intermediate activations
with 1 % heavy-tailed channels, B 28672 x 8192 weight, bf16), headline retention ratio rho = 0.5; the other
ratios, the 1B-class product (2048 x 8192 x 2048) and the other 70B-class products are reported beside it.
With N > 1 every rank runs the same workload on its own GPU (independent replicas, no data-path collective).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

prints ONE JSON line.  `--impl reference` times the CPU oracle (the slow fp64 checker) on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

M, K, N = 32768, 28672, 8192          # headline product: 70B-class down projection
M1, K1, N1 = 2048, 8192, 2048         # the 1B-class down projection (reported in `mlp_1b`)
RHO = 0.5
RHOS = (0.25, 0.5, 0.75, 1.0)
METRIC = "reduced-GEMM retained TFLOP/s (whole RMM op: score + select + reduced product)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0          # dense bf16 tensor peak of a B200 as specified (context beside the measured peaks)
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the GEMM kernel on the headline workload at rho = 0.5,
# from the one-pass ncu capture summarised in profiles/reduced_gemm_tc_kernel_down_proj_28672x8192_rho0.5.md
GEMM_DRAM_TRAFFIC_BYTES = 7609957888 + 536464128
WORKLOAD = ("70B-class MLP down-projection: A 32768x28672 bf16 N(0,1) with 1% Student-t(3) channels, "
            "B 28672x8192 bf16 N(0,0.02^2)")


def keep(rho: float, k_axis: int) -> int:
    return max(1, math.ceil(rho * k_axis - 1e-9))


def retained_flops(rho: float, m: int = M, k_axis: int = K, n: int = N) -> float:
    return 2.0 * m * keep(rho, k_axis) * n


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"bf16_burst": float(d["bf16_tflops"]), "bf16_sustained": float(d["bf16_tflops_sustained"]),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x: float, world: int) -> float:
    """The slowest rank's time (replicas are independent: the job is as slow as its slowest replica)."""
    if world == 1:
        return x
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(ms_step: float, world: int, rho: float = RHO) -> float:
    """TFLOP/s of the whole job: every replica retains the same FLOPs per step; ms_step is the max over ranks."""
    return world * retained_flops(rho) / (ms_step * 1e-3) / 1e12


def gemm_roofline(achieved_tflops: float, kernel_ms: float, peaks: dict, clocks: dict, traffic):
    """Roofline entry of the tensor-core GEMM.  The denominator is the measured cuBLAS bf16 rate that matches the clocks
    the kernel actually ran at: the sustained figure when the SM clock sampled during the timed region sagged under the
    power cap (median below 85 % of the maximum), the burst figure otherwise."""
    sm, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    sagged = bool(sm and mx and sm < 0.85 * mx)
    peak = peaks["bf16_sustained"] if sagged else peaks["bf16_burst"]
    return {"bound": "tensor", "kernel": "reduced_gemm_tc_kernel", "achieved": achieved_tflops, "peak": peak, "unit": "TFLOP/s",
            "frac": achieved_tflops / peak, "traffic": traffic,
            "peak_source": f"{peaks['source']} cuBLAS bf16, {'sustained (SM clock sagged under load)' if sagged else 'burst (SM clock stayed near maximum)'}",
            "frac_of_burst_peak": achieved_tflops / peaks["bf16_burst"],
            "frac_of_sustained_peak": achieved_tflops / peaks["bf16_sustained"],
            "frac_of_nominal_peak": achieved_tflops / NOMINAL_BF16_TFLOPS,
            "kernel_ms": kernel_ms, "sm_mhz_x_kernel_ms": (sm * kernel_ms) if sm else None}


def time_region(fn, steps: int, world: int) -> float:
    """ms per step over exactly `steps` calls, device-timed, barrier + synchronize on both sides, max over ranks."""
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    barrier(world)
    return max_over_ranks(e0.elapsed_time(e1), world) / steps


def interleaved_rho_sweep(rmm, binding, A, B, Y, rhos, rounds: int = 6):
    """Whole reduced product per rho and the dense cuBLAS product of the same shape, timed call by call in rotation
    (each call bracketed by its own events): under the power cap the SM clock drifts by a quarter over seconds of
    tensor-core load, so variants timed one after the other are not comparable, variants that take turns are.
    Returns ({rho: (whole_op_ms, gemm_kernel_ms)}, dense_ms)."""
    Kx = A.shape[-1]
    idx = {rho: torch.empty(rmm.rmm_keep_count(rho, Kx), dtype=torch.int32, device=A.device) for rho in rhos}
    calls = [lambda: torch.matmul(A, B, out=Y)] + [(lambda rho=rho: rmm.rmm_product(A, B, rho=rho, out=Y, idx=idx[rho])) for rho in rhos]
    for c in calls:
        c()
        c()
    nv = len(calls)
    total, gemm, order = [0.0] * nv, [0.0] * nv, []
    kt = binding.KernelTimer(rounds * nv, "reduced_gemm_tc_kernel")
    with kt:
        for r in range(rounds):
            for j in range(nv):
                jj = (j + r) % nv
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                calls[jj]()
                e1.record()
                e1.synchronize()
                total[jj] += e0.elapsed_time(e1)
                if jj > 0:
                    order.append(jj)
    times = [t for _, t in kt.times_ms()]
    assert len(times) == len(order)
    for jj, t in zip(order, times):
        gemm[jj] += t
    return {rho: (total[j + 1] / rounds, gemm[j + 1] / rounds) for j, rho in enumerate(rhos)}, total[0] / rounds


def cpu_oracle_sample(A_rows, B, rho: float, m_total: int, target_s: float = 12.0):
    """Time the oracle as it stands on a bounded sample of the headline workload: the score pass on `A_rows` (a slice of
    the activations), the selection at full width, the product on as many of those rows as fit the time target.  The
    whole-workload figure is an extrapolation to all m_total rows (score and product are row-separable) and says so."""
    import oracle
    oracle.build()
    cores = oracle.num_threads()
    R, k_axis = A_rows.shape
    n = B.shape[1]
    t0 = time.perf_counter()
    e, _ = oracle.score(A_rows)
    t_score = time.perf_counter() - t0
    t0 = time.perf_counter()
    idx, _ = oracle.select(e, oracle.keep_count(rho, k_axis))
    t_sel = time.perf_counter() - t0
    probe = min(R, cores)
    t0 = time.perf_counter()
    oracle.reduced_gemm(A_rows, B, idx, rows=(0, probe))
    t_probe = time.perf_counter() - t0
    rows = int(max(probe, min(R, target_s / max(t_probe / probe, 1e-9))))
    rows = max(cores, rows // cores * cores)
    t0 = time.perf_counter()
    oracle.reduced_gemm(A_rows, B, idx, rows=(0, rows))
    t_rows = time.perf_counter() - t0
    # time of the whole workload, extrapolated: score on m_total rows, one selection, product on m_total rows
    t_full = t_score * m_total / R + t_sel + t_rows * m_total / rows
    flops = 2.0 * m_total * len(idx) * n
    return {"value": flops / t_full / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"extrapolated from a sample: score on {R} of {m_total} rows ({t_score:.2f} s), selection over {k_axis} keys "
                      f"({t_sel:.3f} s), product on {rows} rows at rho={rho} ({t_rows:.2f} s); whole workload would take {t_full:.0f} s",
            "seconds": t_score + t_sel + t_probe + t_rows}


def run_reference(args):
    """Reference arm: the CPU oracle, timed on this machine's host cores; rank 0 only.  Every step is a bounded sample of the
    headline workload: score, selection and product on `cores` rows of activations of the same width."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2608_13426_b200 import synth
    import oracle
    oracle.build()
    cores = oracle.num_threads()
    rows = cores                             # one row per thread
    A = synth.heavy_tailed_activations(rows, K, seed=0)
    B = synth.weight(K, N, seed=1)
    k = oracle.keep_count(RHO, K)
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        e, _ = oracle.score(A)
        idx, _ = oracle.select(e, k)
        oracle.reduced_gemm(A, B, idx, rows=(0, rows))
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = 2.0 * rows * k * N / (ms / 1e3) / 1e12
    sample = f"{rows} rows of {M} per step (score, selection and product on that sample), rho={RHO}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "rho": RHO, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def attention_case(rmm, binding, synth, dev, heads, seq, head_dim=128, reps=10, ratios=((0.5, 1.0), (0.75, 1.0), (0.5, 0.5), (0.5, 0.25))):
    """Reduced attention on a prefill shape (heads x seq x head_dim, causal): feature reduction only (one fused pass) and
    feature + token reduction (three fused sweeps: row normalisers, token scores, gathered P V); S~ and P stay on the SM
    in both.  torch's dense scaled_dot_product_attention at the same shape is context, not a target."""
    Qa, Ka, Va = synth.attention_qkv(1, heads, heads, seq, seq, head_dim, seed=0, device=str(dev))
    for _ in range(3):
        torch.nn.functional.scaled_dot_product_attention(Qa, Ka, Va, is_causal=True)
    dense = time_region(lambda i: torch.nn.functional.scaled_dot_product_attention(Qa, Ka, Va, is_causal=True), reps, 1)
    out = []
    for rho_d, rho_t in ratios:
        for _ in range(2):
            rmm.rmm_reduced_attn(Qa, Ka, Va, True, rho_d, rho_t)
        t = time_region(lambda i: rmm.rmm_reduced_attn(Qa, Ka, Va, True, rho_d, rho_t), reps, 1)
        kt = binding.KernelTimer(64)
        with kt:
            rmm.rmm_reduced_attn(Qa, Ka, Va, True, rho_d, rho_t)
        parts = {}
        for name, x in kt.times_ms():
            parts[name] = parts.get(name, 0.0) + 1e3 * x
        kd = rmm.rmm_keep_count(rho_d, head_dim)
        # causal flops actually needed: (kd + Dh * rho_t) multiply-adds per visible (query, key) pair
        fl = 2.0 * heads * (seq * (seq + 1) / 2) * (kd + head_dim * rho_t)
        out.append({"rho_d": rho_d, "rho_t": rho_t, "shape": [heads, seq, head_dim], "causal": True, "ms": t,
                    "retained_tflops": fl / t / 1e9, "kernels_us": parts, "dense_sdpa_ms": dense,
                    "speedup_vs_dense_sdpa": dense / t,
                    "path": ("composed (S~ and P in memory)" if kd > 128 else "fused, ") +
                            ("" if kd > 128 else ("one pass" if rho_t >= 1.0 else "three sweeps")) +
                            ("" if kd > 128 or head_dim <= 128 else ", two passes over the columns of V")})
    return out


def layer_sweep_70b(rmm, binding, synth, dev, peaks, tokens=32768, hidden=8192, inter=28672, reps=5):
    """Whole reduced product (score + select + gathers + GEMM) per projection shape and rho, dense cuBLAS beside it."""
    # (Q, K and V read the same activations, hence the same index set: fused into one product they share the selection
    # and the gather of A, which the narrow K/V projection alone cannot repay)
    shapes = [("q_o_proj", tokens, hidden, hidden), ("k_v_proj", tokens, hidden, 1024), ("qkv_fused_proj", tokens, hidden, hidden + 2048),
              ("gate_up_proj", tokens, hidden, inter), ("down_proj", tokens, inter, hidden)]
    out = []
    for name, m, kk, n in shapes:
        A = synth.heavy_tailed_activations(m, kk, seed=7, device=str(dev))
        B = synth.weight(kk, n, seed=8, device=str(dev))
        Y = torch.empty(m, n, dtype=torch.bfloat16, device=dev)
        res, dense = interleaved_rho_sweep(rmm, binding, A, B, Y, RHOS, rounds=reps)
        rows = []
        for rho in RHOS:
            t = res[rho][0]
            fl = 2.0 * m * rmm.rmm_keep_count(rho, kk) * n
            rows.append({"layer": name, "shape": [m, kk, n], "rho": rho, "whole_op_ms": t, "whole_op_tflops": fl / t / 1e9,
                         "frac_of_sustained_peak": fl / t / 1e9 / peaks["bf16_sustained"],
                         "frac_of_burst_peak": fl / t / 1e9 / peaks["bf16_burst"],
                         "dense_cublas_ms": dense, "dense_cublas_tflops": 2.0 * m * kk * n / dense / 1e9,
                         "speedup_vs_dense_cublas": dense / t, "timing": "variants interleaved call by call"})
        out += rows
        del A, B, Y
    # attention of one layer: 64 query heads on 8 kv heads, causal
    Q, Kx, V = synth.attention_qkv(1, 64, 8, tokens, tokens, 128, seed=0, device=str(dev))
    for _ in range(2):
        torch.nn.functional.scaled_dot_product_attention(Q, Kx, V, is_causal=True, enable_gqa=True)
    dense = time_region(lambda i: torch.nn.functional.scaled_dot_product_attention(Q, Kx, V, is_causal=True, enable_gqa=True), reps, 1)
    for rho_d, rho_t in ((0.5, 1.0), (0.5, 0.5), (0.5, 0.25)):
        rmm.rmm_reduced_attn(Q, Kx, V, True, rho_d, rho_t)
        t = time_region(lambda i: rmm.rmm_reduced_attn(Q, Kx, V, True, rho_d, rho_t), reps, 1)
        out.append({"layer": "attention", "shape": [64, 8, tokens, 128], "rho_d": rho_d, "rho_t": rho_t, "ms": t,
                    "dense_sdpa_ms": dense, "speedup_vs_dense_sdpa": dense / t})
    return out


def chained_mlp_70b(rmm, synth, dev, tokens=32768, hidden=8192, inter=28672, rho=RHO, reps=5):
    """Up projection followed by the reduced down projection of a 70B-class MLP.  The up projection's epilogue leaves
    the column energies of the activations it writes, so the down projection selects its index set from them and needs
    no pass over the 1.9 GB of activations: times with and without that pass, and what the epilogue sums cost."""
    X = synth.heavy_tailed_activations(tokens, hidden, seed=11, device=str(dev))
    W_up = synth.weight(hidden, inter, seed=12, device=str(dev))
    W_down = synth.weight(inter, hidden, seed=13, device=str(dev))
    H = torch.empty(tokens, inter, dtype=torch.bfloat16, device=dev)
    Y = torch.empty(tokens, hidden, dtype=torch.bfloat16, device=dev)
    k = rmm.rmm_keep_count(rho, inter)
    idx = torch.empty(k, dtype=torch.int32, device=dev)
    keep = {}

    def up_plain(i):
        rmm.rmm_reduced_gemm(X, W_up, None, out=H)

    def up_scored(i):
        keep["e"] = rmm.rmm_reduced_gemm(X, W_up, None, out=H, want_energy=True)[1]

    def down_from_energies(i):
        sel = rmm.rmm_select(keep["e"], k=k)
        rmm.rmm_reduced_gemm(H, W_down, sel, out=Y)

    def down_with_score_pass(i):
        rmm.rmm_product(H, W_down, rho=rho, out=Y, idx=idx)

    def dense_block(i):
        torch.matmul(X, W_up, out=H)
        torch.matmul(H, W_down, out=Y)

    # The SM clock under the power cap drifts by a quarter over a few seconds of tensor-core load, so the variants are
    # interleaved call by call (each call bracketed by its own events) instead of being timed one after the other.
    names = ["up_ms", "up_with_epilogue_energies_ms", "down_selected_from_epilogue_energies_ms", "down_with_score_pass_ms",
             "block_ms_dense_cublas"]
    fns = [up_plain, up_scored, down_from_energies, down_with_score_pass, dense_block]
    for fn in fns:
        fn(0)
    total = [0.0] * len(fns)
    for r in range(reps):
        for j in range(len(fns)):
            jj = (j + r) % len(fns)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if jj in (2, 3):
                up_scored(r)          # the down projection under test reads H and its energies fresh
            e0.record()
            fns[jj](r)
            e1.record()
            e1.synchronize()
            total[jj] += e0.elapsed_time(e1)
    res = {"shape_up": [tokens, hidden, inter], "shape_down": [tokens, inter, hidden], "rho_down": rho,
           "timing": "variants interleaved call by call"}
    for n, t in zip(names, total):
        res[n] = t / reps
    res["block_ms_epilogue_energies"] = res["up_with_epilogue_energies_ms"] + res["down_selected_from_epilogue_energies_ms"]
    res["block_ms_score_pass"] = res["up_ms"] + res["down_with_score_pass_ms"]
    del X, W_up, W_down, H, Y
    return res


def paper_table5_case(rmm, synth, dev, reps=10):
    """The setting of the paper's kernel-latency table (8B-class attention: 32 heads, head_dim 128, batch 1, rho = 0.8
    on both axes, L = 1024 / 2048 / 4096).  The paper's A100 figures (RMM QK^T kernel + RMM AV kernel, each with its
    norm and top-k) are quoted beside ours as context: other hardware, other software."""
    paper_ms = {1024: (0.089, 0.039), 2048: (0.336, 0.114), 4096: (1.071, 0.399)}
    out = []
    for L, (qk, av) in paper_ms.items():
        Q, Kx, V = synth.attention_qkv(1, 32, 32, L, L, 128, seed=0, device=str(dev))
        for _ in range(3):
            rmm.rmm_reduced_attn(Q, Kx, V, True, 0.8, 0.8)
        t = time_region(lambda i: rmm.rmm_reduced_attn(Q, Kx, V, True, 0.8, 0.8), reps, 1)
        out.append({"seq": L, "rho_d": 0.8, "rho_t": 0.8, "causal": True, "ms": t,
                    "paper_a100_rmm_qk_plus_av_ms": qk + av, "note": "paper figure: A100, Triton, layout and mask not stated"})
    return out


def gemm_framed_attention(rmm, synth, dev, peaks, reps=5):
    """The attention products as stand-alone reduced GEMMs with their operands in memory: QK^T with head_dim reduction
    (32 heads, 4096 tokens; S~ is written, so the product is bound by that write) and PV with sequence-axis reduction
    on a given causal P (16384 tokens, 4 of the 32 heads: P alone is 0.5 GB per head)."""
    out = []
    H, L, Dh = 32, 4096, 128
    Q, Kx, _ = synth.attention_qkv(1, H, H, L, L, Dh, seed=0, device=str(dev))
    Qd, Kd = Q[0], Kx[0]
    S = torch.empty(H, L, L, dtype=torch.bfloat16, device=dev)
    for _ in range(2):
        torch.bmm(Qd, Kd.transpose(1, 2), out=S)
    dense = time_region(lambda i: torch.bmm(Qd, Kd.transpose(1, 2), out=S), reps, 1)
    for rho in (0.5, 0.75):
        idx, _, _, _ = rmm.rmm_score_select(Qd, rho=rho)

        def op(i):
            rmm.rmm_score_select(Qd, rho=rho, idx=idx)
            rmm.rmm_reduced_gemm(Qd, Kd.transpose(1, 2), idx, scale=Dh ** -0.5, out=S)

        op(0)
        t = time_region(op, reps, 1)
        out.append({"product": "QK^T, head_dim reduction", "shape": [H, L, Dh], "rho": rho, "whole_op_ms": t,
                    "s_written_gbs": S.numel() * 2 / t / 1e6, "frac_of_hbm_peak": S.numel() * 2 / t / 1e6 / peaks["hbm_gbs"],
                    "dense_bmm_ms": dense, "speedup_vs_dense": dense / t})
    del S, Q, Kx
    H, L = 4, 16384
    P = synth.attention_probs(L, H, Dh, seed=3, causal=True, device=str(dev))
    V = synth.gaussian((H, L, Dh), 1.0, seed=5).to(dev)
    O = torch.empty(H, L, Dh, dtype=torch.bfloat16, device=dev)
    for _ in range(2):
        torch.bmm(P, V, out=O)
    dense = time_region(lambda i: torch.bmm(P, V, out=O), reps, 1)
    for rho in (0.25, 0.5):
        idx, _, _, _ = rmm.rmm_score_select(P, rho=rho)
        sel = time_region(lambda i: rmm.rmm_score_select(P, rho=rho, idx=idx), reps, 1)
        rmm.rmm_reduced_gemm(P, V, idx, out=O)
        g = time_region(lambda i: rmm.rmm_reduced_gemm(P, V, idx, out=O), reps, 1)
        out.append({"product": "PV, sequence-axis reduction on a given P", "shape": [H, L, Dh], "rho": rho,
                    "score_select_ms": sel, "score_select_gbs": P.numel() * 2 / sel / 1e6,
                    "score_select_frac_of_hbm": P.numel() * 2 / sel / 1e6 / peaks["hbm_gbs"], "gather_gemm_ms": g,
                    "whole_op_ms": sel + g, "dense_bmm_ms": dense, "speedup_vs_dense": dense / (sel + g)})
    return out


def low_bit_sweep(rmm, binding, synth, dev, peaks, reps=10):
    """The reduced product with 8-bit operands (e4m3 activations quantised on the fly, e4m3 weight) beside the bf16 one, on
    the 1B-class and the 70B-class down projection at rho = 0.5: gathers + product, and the product kernel alone."""
    out = []
    for (m, kk, n) in ((M1, K1, N1), (M, K, N)):
        A = synth.heavy_tailed_activations(m, kk, seed=5, device=str(dev))
        W = synth.weight(kk, n, seed=6, device=str(dev))
        b_scale = float(W.abs().max()) / 448.0
        Bq = (W.t().float() / b_scale).to(torch.float8_e4m3fn).contiguous()
        Y = torch.empty(m, n, dtype=torch.bfloat16, device=dev)
        idx, _, _, _ = rmm.rmm_score_select(A, rho=RHO)
        row = {"shape": [m, kk, n], "rho": RHO, "k": int(idx.numel())}
        for name, fn in (("bf16", lambda i: rmm.rmm_reduced_gemm(A, W, idx, out=Y)),
                         ("e4m3", lambda i: rmm.rmm_reduced_gemm_q8(A, Bq, b_scale, idx, out=Y))):
            for i in range(3):
                fn(i)
            t = time_region(fn, reps, 1)
            kt = binding.KernelTimer(reps, "reduced_gemm_tc_kernel")
            with kt:
                time_region(fn, reps, 1)
            g = sum(x for _, x in kt.times_ms()) / reps
            fl = 2.0 * m * idx.numel() * n
            row[name] = {"gathers_and_product_ms": t, "product_kernel_ms": g, "product_kernel_tflops": fl / g / 1e9}
        row["e4m3_speedup_product_kernel"] = row["bf16"]["product_kernel_ms"] / row["e4m3"]["product_kernel_ms"]
        row["e4m3_speedup_with_gathers"] = row["bf16"]["gathers_and_product_ms"] / row["e4m3"]["gathers_and_product_ms"]
        out.append(row)
        del A, W, Bq, Y
    return out


def run_mlp_1b_only(args):
    """Only the 1B-class product at rho = 0.5 (a few dozen launches: for profiler captures of the one-launch front end
    and of the single-tile GEMM); prints its own JSON line."""
    import paper_2608_13426_b200 as rmm
    from paper_2608_13426_b200 import binding, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    res = small_product_sweep(rmm, binding, synth, dev, measured_peaks(), 0, reps=max(3, args.steps), rhos=(RHO,))
    assert rmm.rmm_status_read() == 0
    print(json.dumps({"mlp_1b": res}))


def run_phase_stamps(args):
    """Per-phase timelines from a library built with the debug time stamps
    (RMM_NVCC_EXTRA="-DRMM_GEMM_STAMPS -DRMM_FRONT_STAMPS -DRMM_ATTN_STAMPS" python -m paper_2608_13426_b200.build):
    the one-launch front end and the GEMM of the 1B-class product (microseconds from the first block's start; maxima over
    blocks), and the clocks per phase of the fused attention kernel's MMA-issuing thread and of one softmax warp.  The
    shipped library has no stamps; rebuild without the flags afterwards."""
    import ctypes
    import paper_2608_13426_b200 as rmm
    from paper_2608_13426_b200 import binding, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    L = binding.lib()
    have = {n: hasattr(L, n) for n in ("rmm_debug_front_stamps", "rmm_debug_gemm_stamps", "rmm_debug_attn_stamps")}
    if not any(have.values()):
        print(json.dumps({"phase_stamps": None, "why": "the library was built without -DRMM_*_STAMPS"}))
        return
    buf = (ctypes.c_ulonglong * 16)()
    out = {}
    A, B = synth.mlp_product(M1, K1, N1, seed=0)
    A, B = A.to(dev), B.to(dev)
    front_names = ["stream_end", "energies_published", "barrier_passed", "selected", None, "a_gathered_b_copied"]
    gemm_names = ["setup_done", "first_mma", "last_main_loop_issued", "last_accumulator_complete", "last_epilogue_done", "last_thread_out"]
    reps = max(5, args.steps)
    for rho in (0.25, 0.5):
        for _ in range(3):
            rmm.rmm_product(A, B, rho=rho)
        torch.cuda.synchronize()
        for n in ("rmm_debug_front_stamps", "rmm_debug_gemm_stamps"):
            if have[n]:
                getattr(L, n)(buf)
        acc_f, acc_g = [0.0] * 6, [0.0] * 6
        for _ in range(reps):
            rmm.rmm_product(A, B, rho=rho)
            torch.cuda.synchronize()
            if have["rmm_debug_front_stamps"]:
                L.rmm_debug_front_stamps(buf)
                for j in range(6):
                    acc_f[j] += (buf[j + 1] - buf[0]) / 1e3
            if have["rmm_debug_gemm_stamps"]:
                L.rmm_debug_gemm_stamps(buf)
                for j in range(6):
                    acc_g[j] += (buf[j + 1] - buf[0]) / 1e3
        e = {}
        if have["rmm_debug_front_stamps"]:
            e["front_us_from_start"] = {n: round(v / reps, 2) for n, v in zip(front_names, acc_f) if n}
        if have["rmm_debug_gemm_stamps"]:
            e["gemm_us_from_start"] = {n: round(v / reps, 2) for n, v in zip(gemm_names, acc_g)}
        out[f"mlp_1b_rho{rho}"] = e
    if have["rmm_debug_attn_stamps"]:
        Q, Kk, V = synth.attention_qkv(1, args.attn_heads, args.attn_heads, args.attn_seq, args.attn_seq, 128, seed=0, device=str(dev))
        mma = ["wait_k", "wait_s_empty", "issue_s", "wait_v", "wait_o_empty", "wait_p_full", "issue_pv", "other"]
        smx = ["wait_s_full", "unused", "max_and_rescale", "weights_chunk_1", "wait_p_empty", "store_reload_weights_chunk_0", "epilogue", "loop_top"]
        for causal in (True, False):
            for _ in range(2):
                rmm.rmm_reduced_attn(Q, Kk, V, causal, 0.5, 1.0)
            L.rmm_debug_attn_stamps(buf)
            rmm.rmm_reduced_attn(Q, Kk, V, causal, 0.5, 1.0)
            L.rmm_debug_attn_stamps(buf)
            v = list(buf)
            out[f"fused_attn_clocks_block0_causal{int(causal)}"] = {"mma_thread": dict(zip(mma, v[:8])), "softmax_warp": dict(zip(smx, v[8:]))}
    assert rmm.rmm_status_read() == 0
    print(json.dumps({"phase_stamps": out}))


def run_attention_only(args):
    import paper_2608_13426_b200 as rmm
    from paper_2608_13426_b200 import binding, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    res = attention_case(rmm, binding, synth, dev, args.attn_heads, args.attn_seq, reps=3)
    assert rmm.rmm_status_read() == 0
    print(json.dumps({"attention_prefill": res}))


def small_product_sweep(rmm, binding, synth, dev, peaks, rank, reps=40, n_sets=5, rhos=RHOS):
    """The 1B-class down projection (A 2048 x 8192, B 8192 x 2048): whole op per rho through rmm_product (one front-end
    launch + the product), its kernels, dense cuBLAS at the same shape and cuBLAS on operands gathered beforehand.
    Five (A, B, Y) sets (377 MB, above L2) are rotated."""
    sets = []
    for s_ in range(n_sets):
        A, B = synth.mlp_product(M1, K1, N1, seed=100 * rank + s_)
        sets.append((A.to(dev), B.to(dev), torch.empty(M1, N1, dtype=torch.bfloat16, device=dev)))
    for i in range(5):
        torch.matmul(sets[i % n_sets][0], sets[i % n_sets][1], out=sets[i % n_sets][2])
    dense_ms = time_region(lambda i: torch.matmul(sets[i % n_sets][0], sets[i % n_sets][1], out=sets[i % n_sets][2]), reps, 1)
    out = []
    for rho in rhos:
        kk = rmm.rmm_keep_count(rho, K1)
        idx_r = torch.empty(kk, dtype=torch.int32, device=dev)

        def step(i):
            A, B, Y = sets[i % n_sets]
            rmm.rmm_product(A, B, rho=rho, out=Y, idx=idx_r)

        for i in range(3):
            step(i)
        whole = time_region(step, reps, 1)
        kt = binding.KernelTimer(4 * reps)
        with kt:
            for i in range(reps):
                step(i)
        parts = {}
        for name, x in kt.times_ms():
            parts.setdefault(name, []).append(1e3 * x)
        parts = {name: sum(v) / reps for name, v in parts.items()}      # us per step, launch gaps included
        g = parts.get("reduced_gemm_tc_kernel", float("nan")) * 1e-3
        front = sum(v for name, v in parts.items() if name != "reduced_gemm_tc_kernel") * 1e-3
        pre = [(a_[:, idx_r.long()].contiguous(), b_[idx_r.long()].contiguous(), y_) for a_, b_, y_ in sets]
        for i in range(3):
            torch.matmul(pre[i % n_sets][0], pre[i % n_sets][1], out=pre[i % n_sets][2])
        ideal = time_region(lambda i: torch.matmul(pre[i % n_sets][0], pre[i % n_sets][1], out=pre[i % n_sets][2]), reps, 1)
        del pre
        fl = retained_flops(rho, M1, K1, N1)
        out.append({"rho": rho, "k": kk, "shape": [M1, K1, N1], "whole_op_ms": whole, "whole_op_tflops": fl / whole / 1e9,
                    "kernels_us_event_bracketed": parts,
                    "gemm_kernel_ms": g, "gemm_kernel_tflops": fl / g / 1e9,
                    "gemm_frac_of_burst_peak": fl / g / 1e9 / peaks["bf16_burst"],
                    "gemm_frac_of_sustained_peak": fl / g / 1e9 / peaks["bf16_sustained"],
                    "gemm_frac_of_nominal_peak": fl / g / 1e9 / NOMINAL_BF16_TFLOPS,
                    "front_end_ms": front, "front_end_gbs": M1 * K1 * 2 / front / 1e6 if front > 0 else None,
                    "front_end_frac_of_hbm": M1 * K1 * 2 / front / 1e6 / peaks["hbm_gbs"] if front > 0 else None,
                    "cublas_on_pregathered_ms": ideal, "dense_cublas_ms": dense_ms, "speedup_vs_dense_cublas": dense_ms / whole})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the CPU oracle timing (quick runs, profiling)")
    ap.add_argument("--no-sweep", action="store_true", help="skip everything but the headline step (quick runs, profiling)")
    ap.add_argument("--rows", type=int, default=M, help="rows of the headline product (smaller: profiler captures)")
    ap.add_argument("--attention-only", action="store_true",
                    help="run only the reduced-attention case (a few launches: for profiler captures) and print its own JSON line")
    ap.add_argument("--mlp-1b-only", action="store_true",
                    help="run only the 1B-class product at rho = 0.5 (for profiler captures) and print its own JSON line")
    ap.add_argument("--phase-stamps", action="store_true",
                    help="print per-phase timelines; needs a library built with -DRMM_GEMM_STAMPS -DRMM_FRONT_STAMPS -DRMM_ATTN_STAMPS")
    ap.add_argument("--attn-heads", type=int, default=32)
    ap.add_argument("--attn-seq", type=int, default=4096)
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.attention_only:
        return run_attention_only(args)
    if args.mlp_1b_only:
        return run_mlp_1b_only(args)
    if args.phase_stamps:
        return run_phase_stamps(args)
    if args.warmup < 3:
        args.warmup = 3

    import paper_2608_13426_b200 as rmm
    from paper_2608_13426_b200 import binding, synth

    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local if world > 1 else 0)
    peaks = measured_peaks()
    m = args.rows

    # ---- inputs, resident in HBM before the timed region: A 1.88 GB, B 470 MB, Y 537 MB (far above the 126 MB L2)
    A = synth.heavy_tailed_activations(m, K, seed=100 * rank, device=str(dev))
    B = synth.weight(K, N, seed=100 * rank + 1, device=str(dev))
    Y = torch.empty(m, N, dtype=torch.bfloat16, device=dev)
    k = rmm.rmm_keep_count(RHO, K)
    idx_buf = torch.empty(k, dtype=torch.int32, device=dev)
    resident_bytes = (m * K + K * N + m * N) * 2

    def step(i, rho=RHO, idx=idx_buf):
        rmm.rmm_product(A, B, rho=rho, out=Y, idx=idx)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert rmm.rmm_status_read() == 0

    # ---- timed region: exactly K steps; every GEMM launch is bracketed by events on the same stream (a step lasts
    # milliseconds, so the event records cost nothing measurable)
    sampler = ClockSampler(local if world > 1 else 0)
    timer = binding.KernelTimer(min(args.steps, 4096), "reduced_gemm_tc_kernel")
    launches0 = rmm.rmm_launch_count()
    sampler.start()
    with timer:
        ms_step = time_region(step, args.steps, world)
    clocks = sampler.stop()
    launches = rmm.rmm_launch_count() - launches0
    gemm_ms = [t for _, t in timer.times_ms()]
    gemm_ms_avg = sum(gemm_ms) / len(gemm_ms)
    assert rmm.rmm_status_read() == 0
    flops_step = retained_flops(RHO, m, K, N)
    value = world * flops_step / (ms_step * 1e-3) / 1e12

    # ---- roofline of the dominant kernel (the tensor-core GEMM): retained FLOPs of one launch / its mean duration
    achieved = flops_step / (gemm_ms_avg * 1e-3) / 1e12
    roofline = gemm_roofline(achieved, gemm_ms_avg, peaks, clocks, GEMM_DRAM_TRAFFIC_BYTES if m == M else None)

    # ---- per-kernel breakdown of one step (a separate, untimed pass with every launch bracketed by events)
    breakdown = {}
    if rank == 0:
        nb = 5
        kt = binding.KernelTimer(nb * 8)
        with kt:
            for i in range(nb):
                step(i)
        for name, t in kt.times_ms():
            breakdown.setdefault(name, []).append(t)
        breakdown = {name: {"launches_per_step": len(v) / nb, "mean_ms": sum(v) / len(v)} for name, v in breakdown.items()}
        sel_ms = sum(v["mean_ms"] * v["launches_per_step"] for name, v in breakdown.items() if name in ("score_tma_kernel", "select_kernel", "score_select_kernel"))
        if sel_ms > 0:
            gbs = m * K * 2 / sel_ms / 1e6
            breakdown["selection_pass"] = {"ms": sel_ms, "gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                                           "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBS}

    # ---- per-rho sweep on the headline product: whole op beside dense cuBLAS at the same shape
    per_rho = []
    if not args.no_sweep and rank == 0 and world == 1:  # (replicas: the headline only)
        res, dense_ms = interleaved_rho_sweep(rmm, binding, A, B, Y, RHOS)
        for rho in RHOS:
            whole, g = res[rho]
            fl = retained_flops(rho, m, K, N)
            per_rho.append({"rho": rho, "k": rmm.rmm_keep_count(rho, K), "whole_op_ms": whole, "whole_op_tflops": fl / whole / 1e9,
                            "gemm_kernel_ms": g, "gemm_kernel_tflops": fl / g / 1e9,
                            "gemm_frac_of_sustained_peak": fl / g / 1e9 / peaks["bf16_sustained"],
                            "gemm_frac_of_burst_peak": fl / g / 1e9 / peaks["bf16_burst"],
                            "gemm_frac_of_nominal_peak": fl / g / 1e9 / NOMINAL_BF16_TFLOPS,
                            "dense_cublas_ms": dense_ms, "dense_cublas_tflops": 2.0 * m * K * N / dense_ms / 1e9,
                            "speedup_vs_dense_cublas": dense_ms / whole, "timing": "variants interleaved call by call"})

    # ---- CPU oracle on a bounded sample of the same workload (rank 0, one GPU only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_oracle_sample(A[:1024].cpu(), B.cpu(), RHO, m)

    # ---- end to end: host buffers in, host buffer out, through the C-ABI host entry point (copies inside the timed region)
    Ah = torch.empty(m, K, dtype=torch.bfloat16).pin_memory()
    Bh = torch.empty(K, N, dtype=torch.bfloat16).pin_memory()
    Ah.copy_(A)
    Bh.copy_(B)
    Yh = torch.empty(m, N, dtype=torch.bfloat16).pin_memory()
    ih = torch.empty(K, dtype=torch.int32).pin_memory()
    del A, B, Y
    torch.cuda.empty_cache()

    def step_e2e(i):
        rmm.rmm_product_host(Ah, Bh, RHO, Yh, ih)
        torch.cuda.current_stream().synchronize()      # the caller reads Y_host after every step

    for i in range(2):
        step_e2e(i)
    e2e_steps = max(3, min(args.steps, 5))
    ms_e2e = time_region(step_e2e, e2e_steps, world)
    e2e = {"value": world * flops_step / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e, "steps": e2e_steps,
           "h2d_bytes_per_step": (m * K + K * N) * 2, "d2h_bytes_per_step": m * N * 2 + k * 4}
    del Ah, Bh, Yh
    binding._ws_cache.clear()
    torch.cuda.empty_cache()

    extras = {}
    if not args.no_sweep and rank == 0 and world == 1:  # (replicas: the headline only)
        # ---- the 1B-class product (where launch and selection latencies matter most)
        extras["mlp_1b"] = small_product_sweep(rmm, binding, synth, dev, peaks, rank)

        # ---- the selection pass on a 70B-class activation (32768 tokens x 8192 hidden, 537 MB): bandwidth-bound
        Ml, Kl = 32768, 8192
        big = [synth.heavy_tailed_activations(Ml, Kl, seed=50 + i, device=str(dev)) for i in range(2)]
        idx_l = torch.empty(rmm.rmm_keep_count(RHO, Kl), dtype=torch.int32, device=dev)
        for i in range(3):
            rmm.rmm_score_select(big[i % 2], rho=RHO, idx=idx_l)
        t = time_region(lambda i: rmm.rmm_score_select(big[i % 2], rho=RHO, idx=idx_l), 20, 1)
        gbs = Ml * Kl * 2 / t / 1e6
        extras["selection_pass_large"] = {"shape": [Ml, Kl], "ms": t, "gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                                          "frac_of_nominal_hbm": gbs / NOMINAL_HBM_GBS,
                                          "note": "fused score + top-k select, two alternating 537 MB inputs (above L2)"}
        del big

        # ---- decode step (one activation row) on a 70B-class gate/up projection: the gathered GEMV reads only the kept rows
        Kd, Nd = 8192, 28672
        Ws = [synth.weight(Kd, Nd, seed=70 + i, device=str(dev)) for i in range(3)]     # 3 x 470 MB, rotated
        x = synth.heavy_tailed_activations(1, Kd, seed=73, device=str(dev))
        yd = torch.empty(1, Nd, dtype=torch.bfloat16, device=dev)
        decode = []
        for i in range(3):
            torch.matmul(x, Ws[i], out=yd)
        dense = time_region(lambda i: torch.matmul(x, Ws[i % 3], out=yd), 30, 1)
        for rho in (0.25, 0.5, 1.0):
            idx_d, _, _, _ = rmm.rmm_score_select(x, rho=rho)
            for i in range(3):
                rmm.rmm_reduced_gemm(x, Ws[i % 3], idx_d, out=yd)
            t = time_region(lambda i: rmm.rmm_reduced_gemm(x, Ws[i % 3], idx_d, out=yd), 30, 1)
            gbs = idx_d.numel() * Nd * 2 / t / 1e6
            decode.append({"rho": rho, "shape": [1, Kd, Nd], "reduced_gemv_ms": t, "kept_rows_gbs": gbs,
                           "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "dense_cublas_ms": dense, "speedup_vs_dense": dense / t})
        for Mb in (4, 16, 64, 128):
            xb = synth.heavy_tailed_activations(Mb, Kd, seed=74, device=str(dev))
            yb = torch.empty(Mb, Nd, dtype=torch.bfloat16, device=dev)
            idx_b, _, _, _ = rmm.rmm_score_select(xb, rho=0.5)
            for i in range(3):
                rmm.rmm_reduced_gemm(xb, Ws[i % 3], idx_b, out=yb)
                torch.matmul(xb, Ws[i % 3], out=yb)
            t = time_region(lambda i: rmm.rmm_reduced_gemm(xb, Ws[i % 3], idx_b, out=yb), 30, 1)
            dn = time_region(lambda i: torch.matmul(xb, Ws[i % 3], out=yb), 30, 1)
            gbs = idx_b.numel() * Nd * 2 / t / 1e6
            decode.append({"rho": 0.5, "shape": [Mb, Kd, Nd], "reduced_product_ms": t, "kept_rows_gbs": gbs,
                           "frac_of_hbm_peak": gbs / peaks["hbm_gbs"], "dense_cublas_ms": dn, "speedup_vs_dense": dn / t})
        del Ws
        extras["decode_step"] = decode

        # ---- reduced attention on a 7B-class prefill, the paper's kernel-latency setting, the attention products as GEMMs
        extras["attention_prefill"] = attention_case(rmm, binding, synth, dev, 32, 4096)
        extras["attention_wide_heads"] = attention_case(rmm, binding, synth, dev, 16, 4096, head_dim=256, reps=5,
                                                        ratios=((0.5, 1.0), (0.25, 1.0), (0.5, 0.5), (0.75, 1.0)))
        extras["attention_paper_setting"] = paper_table5_case(rmm, synth, dev)
        extras["attention_products_in_memory"] = gemm_framed_attention(rmm, synth, dev, peaks)

        # ---- 8-bit operands beside bf16
        extras["low_bit_operands"] = low_bit_sweep(rmm, binding, synth, dev, peaks)

        # ---- the other 70B-class products and the attention of one layer
        extras["layer_sweep_70b"] = layer_sweep_70b(rmm, binding, synth, dev, peaks)

        # ---- up projection -> reduced down projection, the index set taken from the up projection's epilogue energies
        extras["mlp_block_70b"] = chained_mlp_70b(rmm, synth, dev)

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "rho": RHO, "k": k, "M": m, "K": K, "N": N, "parallelism": f"replicas x{world}",
                       "l2_policy": f"inputs larger than L2: {resident_bytes / 1e9:.2f} GB of operands resident per GPU"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "kernel_breakdown": breakdown, "per_rho": per_rho, "peaks": peaks,
        }
        out.update(extras)
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
