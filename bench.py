"""Benchmark of the PRQuant hot path on B200: activation quantisation + compensated MXFP4 GEMM.

One "step" = one pass of the whole online path (prq_quantize_act then prq_linear) over one batch of
M tokens of a Qwen3-4B-shaped down_proj (N = 2560, K = 9728, tail k = 256).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--full]

`value` is executed TFLOP/s (2 M N (K + k) per step) with inputs resident in HBM; `e2e` is the same
through prq_forward_host with pinned host buffers (H2D of x and D2H of y inside the timed region).
With N > 1 every rank runs an independent replica on its own GPU (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "PRQuant W4A4 GEMM µs & TFLOP/s, Qwen3-4B down_proj; % of FP4/HBM roofline"
N_OUT, K_IN, K_TAIL, M_TOK = 2560, 9728, 256, 2048
FP4_OVER_BF16 = 4.0  # nominal dense tensor ratio (9 vs 2.25 PFLOP/s)
# DRAM bytes of one prefill GEMM launch at this workload from the ncu capture summarised in
# profiles/prefill_M2048.txt (dram__bytes_read.sum + dram__bytes_write.sum; the outputs were still in L2).
NCU_PREFILL_DRAM_BYTES = 24.37e6 + 0.63e6


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def flops(M, k):
    return 2.0 * M * N_OUT * (K_IN + k)


def gemm_bytes(M, k, out_bytes=4):
    """Algorithmic HBM bytes of one GEMM call: weights and activations read once, output written once."""
    return 0.53125 * N_OUT * (K_IN + k) + 0.53125 * M * K_IN + M * N_OUT * out_bytes


def quant_bytes(M):
    return 2.53125 * M * K_IN


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.stop = [], set(), False
        self.max_mhz = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.t = threading.Thread(target=self.run, daemon=True)

    def run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self.stop:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv:
            self.t.start()
        return self

    def __exit__(self, *a):
        self.stop = True
        if self.nv:
            self.t.join(timeout=1)

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def oracle_step(orc, x_rows, prep):
    """The oracle's statement of one step on a sample of rows: quantise, expose the tail, FP64 product."""
    y, _, _ = orc.linear(x_rows, prep, identity=True)
    return y


def run_reference(args, rank, world):
    """--impl reference: the CPU oracle as it stands, timed on the host cores on a bounded row sample."""
    if rank != 0:
        return
    from oracle import prq_oracle as orc
    from paper_2609_22106_b200 import synth

    orc.build()
    rows = 16
    L = synth.layer(1, N_OUT, K_IN, rows, T_cal=64)
    prep = orc.prepare(L["W"], orc.channel_amax(L["zcal"]), 0.5, K_TAIL)
    for _ in range(max(args.warmup, 1)):
        oracle_step(orc, L["x"], prep)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(orc, L["x"], prep)
    dt = (time.perf_counter() - t0) / args.steps
    val = flops(rows, K_TAIL) / dt / 1e12
    sample = f"{rows} of {M_TOK} token rows per step (quantise + tail + FP64 product over K+k={K_IN + K_TAIL})"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"qwen3-4b down_proj N={N_OUT} K={K_IN} k_tail={K_TAIL} M={M_TOK}", "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--full", action="store_true", help="also time every (M, k) of the down_proj config")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch

    from paper_2609_22106_b200 import binding as prq
    from paper_2609_22106_b200 import build, synth

    build.build()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    pk = peaks()
    fp4_peak = pk["bf16_tflops"] * FP4_OVER_BF16

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs (seeded, synthetic, Qwen3-4B down_proj shape, heavy-tailed activations) ----
    L = synth.layer(1, N_OUT, K_IN, M_TOK, T_cal=512)
    amax = np.abs(synth.bf16_to_f32(L["zcal"])).max(axis=0)
    ks = (K_TAIL, 0, 128) if args.full else (K_TAIL, 0)
    base = {k: prq.prepare_weights(L["W"], amax, 0.5, k) for k in ks}
    x_src = torch.from_numpy(L["x"].view(np.int16)).to(dev).view(torch.bfloat16)
    W_bf16 = torch.from_numpy(L["W"].view(np.int16)).to(dev).view(torch.bfloat16)
    L2_BYTES = 126e6
    clones = {k: [base[k]] for k in ks}

    def weight_copies(k, n):
        """n independent device copies of the prepared weights (rotation targets)."""
        while len(clones[k]) < n:
            clones[k].append(base[k].clone())
        return clones[k][:n]

    def operand_sets(M, k, y_dtype):
        """Enough independent (weights, x, codes, scales, y, workspace) sets that one pass over all of them
        touches more than twice the L2: every launch then finds its operands in HBM, without any flush."""
        per_set = 2.0 * M * K_IN + 0.53125 * M * K_IN + 0.53125 * N_OUT * (K_IN + k) + 4.0 * M * N_OUT
        R = int(min(24, max(2, np.ceil(2.2 * L2_BYTES / per_set))))
        sets = []
        for w in weight_copies(k, R):
            x = x_src[:M].clone()
            codes = torch.empty(prq.act_bytes(M, K_IN, k, 1, prq.BUF_CODES), dtype=torch.uint8, device=dev)
            sf = torch.empty(prq.act_bytes(M, K_IN, k, 1, prq.BUF_SCALES_SF), dtype=torch.uint8, device=dev)
            y = torch.empty((M, N_OUT), dtype=torch.float32 if y_dtype == prq.F32 else torch.bfloat16, device=dev)
            sets.append(dict(w=w, x=x, codes=codes, sf=sf, y=y, ws=prq.new_workspace(w, M, dev)))
        return sets

    side = torch.cuda.Stream(device=dev)

    def capture(fns):
        for f in fns:
            f()  # first calls configure the kernels; must precede capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for f in fns:
                f()
        return g

    def run_timed(fns, n, warm):
        """Exactly n calls, round-robin over `fns`, between one pair of events; returns seconds.  The calls
        are replayed from two CUDA graphs (one whole rotation, one remainder) so that the host-side cost
        of a call (ctypes, tensor-map encoding) cannot starve the GPU inside the timed region."""
        R = len(fns)
        g_full = capture(fns)
        g_rem = capture(fns[: n % R]) if n % R else None
        for _ in range(max(1, warm // R)):
            g_full.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n // R):
            g_full.replay()
        if g_rem is not None:
            g_rem.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e-3

    def build_graphs(M, k, y_dtype=prq.F32):
        sets = operand_sets(M, k, y_dtype)
        q = lambda s: (lambda: prq.quantize_act(s["w"], s["x"], prq.ACT_IDENTITY, out=(s["codes"], None, s["sf"])))
        g = lambda s: (lambda: prq.linear(s["w"], s["codes"], s["sf"], M, y_dtype, workspace=s["ws"], out=s["y"]))
        step = [(lambda s=s: (q(s)(), g(s)())) for s in sets]
        return dict(step=step, quant=[q(s) for s in sets], gemm=[g(s) for s in sets], R=len(sets))

    def time_path(M, k, steps, warmup, y_dtype=prq.F32):
        gs = build_graphs(M, k, y_dtype)
        t_step = run_timed(gs["step"], steps, warmup)
        n_side = max(gs["R"], min(steps, 200))
        t_q = run_timed(gs["quant"], n_side, gs["R"])
        t_g = run_timed(gs["gemm"], n_side, gs["R"])
        return dict(step_us=t_step / steps * 1e6, quant_us=t_q / n_side * 1e6, gemm_us=t_g / n_side * 1e6,
                    step_total_s=t_step, rotation_sets=gs["R"], timed_launches=2 * steps)

    def time_bf16(M, steps):
        R = int(min(12, max(2, np.ceil(2.2 * L2_BYTES / (2.0 * N_OUT * K_IN + 2.0 * M * K_IN + 2.0 * M * N_OUT)))))
        Ws = [W_bf16.clone() for _ in range(R)]
        xs = [x_src[:M].clone() for _ in range(R)]
        ys = [torch.empty((M, N_OUT), dtype=torch.bfloat16, device=dev) for _ in range(R)]
        gs = [(lambda i=i: torch.matmul(xs[i], Ws[i].t(), out=ys[i])) for i in range(R)]
        n = max(R, min(steps, 200))
        return run_timed(gs, n, R) / n * 1e6

    # ---- main timed region: K steps at M = 2048, k = 256 ----
    w_main = base[K_TAIL]
    main_graphs = build_graphs(M_TOK, K_TAIL)
    barrier()
    with ClockSampler(physical_gpu_index(local_rank)) as clocks:
        total_s = run_timed(main_graphs["step"], args.steps, args.warmup)
        n_side = max(main_graphs["R"], min(args.steps, 400))
        gemm_s = run_timed(main_graphs["gemm"], n_side, main_graphs["R"])
        quant_s = run_timed(main_graphs["quant"], n_side, main_graphs["R"])
    barrier()
    main_t = dict(step_us=total_s / args.steps * 1e6, gemm_us=gemm_s / n_side * 1e6, quant_us=quant_s / n_side * 1e6,
                  rotation_sets=main_graphs["R"], timed_launches=2 * args.steps)
    launches = main_t["timed_launches"]  # K replays of a (quantise, GEMM) graph
    status = prq.last_device_status()
    if dist is not None:
        t = torch.tensor([total_s], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_s = float(t.item())
    ms_per_step = total_s / args.steps * 1e3
    value = world * flops(M_TOK, K_TAIL) / (ms_per_step * 1e-3) / 1e12

    # ---- end to end from host buffers (H2D of x, D2H of y inside the timed region) ----
    xh = torch.from_numpy(L["x"].view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    yh = torch.empty((M_TOK, N_OUT), dtype=torch.float32).pin_memory()
    scratch = torch.zeros(prq.forward_host_scratch_bytes(w_main, M_TOK), dtype=torch.uint8, device=dev)
    e2e_steps = min(args.steps, 50)
    for _ in range(3):
        prq.forward_host(w_main, xh, yh, prq.ACT_IDENTITY, scratch)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        prq.forward_host(w_main, xh, yh, prq.ACT_IDENTITY, scratch)
    e1.record()
    torch.cuda.synchronize()
    e2e_s = e0.elapsed_time(e1) * 1e-3
    if dist is not None:
        t = torch.tensor([e2e_s], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_val = world * flops(M_TOK, K_TAIL) * e2e_steps / e2e_s / 1e12

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- context rows: the same kernels at k = 0, BF16 matmul, the decode shapes ----
    side_steps = min(args.steps, 200)
    detail = {f"M{M_TOK}_k{K_TAIL}": dict(main_t)}
    shapes = [(M, k) for M in (1, 16, 128, M_TOK) for k in ks if (M, k) != (M_TOK, K_TAIL)]
    for M, k in shapes:
        detail[f"M{M}_k{k}"] = time_path(M, k, side_steps, 10)
    detail[f"M{M_TOK}_k{K_TAIL}_bf16out"] = time_path(M_TOK, K_TAIL, side_steps, 10, prq.BF16)
    for name, d in detail.items():
        M = int(name.split("_")[0][1:]); k = int(name.split("_")[1][1:])
        ob = 2 if name.endswith("bf16out") else 4
        d["gemm_tflops"] = flops(M, k) / d["gemm_us"] / 1e6
        d["gemm_gbs"] = gemm_bytes(M, k, ob) / d["gemm_us"] / 1e3
        d["quant_gbs"] = quant_bytes(M) / d["quant_us"] / 1e3
        t_hbm = gemm_bytes(M, k, ob) / pk["hbm_gbs"] / 1e3
        t_fp4 = flops(M, k) / fp4_peak / 1e6
        d["bound"] = "tensor" if t_fp4 > t_hbm else "hbm"
        d["gemm_roofline_frac"] = max(t_hbm, t_fp4) / d["gemm_us"]
        d["quant_roofline_frac"] = d["quant_gbs"] / pk["hbm_gbs"]
    bf16_us = {M: time_bf16(M, side_steps) for M in (1, 16, 128, M_TOK)}
    k0 = detail[f"M{M_TOK}_k0"]

    # ---- CPU baseline: the oracle on a bounded sample of the same workload ----
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import prq_oracle as orc

        orc.build()
        rows = M_TOK  # the whole step: about 10 s of host work on the machine's cores
        prep = orc.prepare(L["W"], amax, 0.5, K_TAIL)
        t0 = time.perf_counter()
        oracle_step(orc, L["x"][:rows], prep)
        dt = time.perf_counter() - t0
        cpu = {"value": flops(rows, K_TAIL) / dt / 1e12, "unit": "TFLOP/s", "cores": orc.num_threads(),
               "kind": "oracle", "sample": f"{rows} of {M_TOK} token rows, one pass (quantise + tail + FP64 product), {dt:.1f} s"}

    gemm_us = main_t["gemm_us"]
    achieved = flops(M_TOK, K_TAIL) / gemm_us / 1e6
    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "mxfp4 (e2m1 x e8m0), f32 accumulate", "data": "synthetic",
        "config": {"workload": f"qwen3-4b down_proj N={N_OUT} K={K_IN} k_tail={K_TAIL} M={M_TOK} (BASELINE configs[1]); "
                               "step = prq_quantize_act + prq_linear, fp32 output",
                   "l2": f"inputs larger than L2: steps rotate over {main_t['rotation_sets']} independent operand sets "
                         "(weights, activations, outputs), more than twice the 126 MB L2 per rotation; no flush",
                   "replicas": "independent per GPU, no collective"},
        "us": {"step": main_t["step_us"], "quant": main_t["quant_us"], "gemm": main_t["gemm_us"],
               "gemm_k0": k0["gemm_us"], "gemm_vs_k0": main_t["gemm_us"] / k0["gemm_us"],
               "bf16_matmul": bf16_us[M_TOK], "gemm_speedup_vs_bf16": bf16_us[M_TOK] / main_t["gemm_us"]},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": fp4_peak, "unit": "TFLOP/s",
                     "frac": achieved / fp4_peak, "frac_of_sustained": achieved / (pk["bf16_tflops_sustained"] * FP4_OVER_BF16),
                     "traffic": NCU_PREFILL_DRAM_BYTES, "algorithmic_bytes": gemm_bytes(M_TOK, K_TAIL),
                     "kernel": "prefill_kernel (stream-K, 128x224 tiles)", "launch_us": gemm_us,
                     "peak_source": f"4 x bf16 burst, of {pk['source']}"},
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_val, "unit": "TFLOP/s", "h2d_bytes_per_step": M_TOK * K_IN * 2, "d2h_bytes_per_step": M_TOK * N_OUT * 4},
        "gpu_launches": int(launches),
        "clocks": clocks.summary(),
        "device_status": status,
        "detail": detail,
        "bf16_matmul_us": bf16_us,
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
