"""Throughput of the MoE FFN layer (forward + backward) on B200, one process per GPU.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload qwen] [--impl ours|reference]

A step is one pass of the whole hot path (router, permutation, gate/up GEMM + SwiGLU, down GEMM, combine and
the full backward) over one batch of synthetic tokens.  Prints ONE JSON line (rank 0):
value = tokens/s of the whole job with inputs resident in HBM; e2e = the same through the host-buffer entry
point with host<->device copies inside the timed region; roofline = the dominant kernel against the
measured peak; cpu_baseline = the CPU oracle timed on a bounded sample on this machine's host cores.
With --impl reference the oracle itself is the timed arm.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2608_00916_b200 import synth  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram bytes per launch of the dominant kernel taken from the committed ncu capture (profiles/), by stage name;
# None where no capture has been taken for the workload.
NCU_TRAFFIC = {  # profiles/step_launch_list_and_dram_traffic_qwen.md, profiles/gemm_dram_traffic_skewed_and_coarse.md
    ("qwen", "gemm_gateup_swiglu"): 2.049e9, ("qwen", "gemm_down"): 1.148e9, ("qwen", "dgrad_down_swiglu_bwd"): 1.885e9,
    ("qwen", "wgrad_down"): 1.134e9, ("qwen", "dgrad_gateup"): 1.797e9, ("qwen", "wgrad_gateup"): 1.750e9,
    ("skewed", "gemm_gateup_swiglu"): 1.992e9, ("skewed", "gemm_down"): 1.138e9, ("skewed", "dgrad_down_swiglu_bwd"): 1.878e9,
    ("skewed", "wgrad_down"): 1.196e9, ("skewed", "dgrad_gateup"): 1.765e9, ("skewed", "wgrad_gateup"): 2.027e9,
}


OVERLAPPED_STAGES = ("router_bwd", "dW_r", "dx_router_term")


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        out = {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
        out["sm_max_mhz"] = float(d.get("sm_max_mhz", 1965.0))
        out["sustained_sm_mhz"] = float(d.get("clocks_under_load", {}).get("sm_mhz_median", 1297.0))
        return out
    return dict(FALLBACK_PEAKS) | {"source": "fallback", "sm_max_mhz": 1965.0, "sustained_sm_mhz": 1300.0}


def stage_work(shape: synth.MoEShape):
    """Algorithmic work per step of every stage: ("tensor", flops) or ("hbm", bytes).  R = T k routed rows."""
    T, d, E, k, f = shape.T, shape.d, shape.E, shape.k, shape.f
    R = T * k
    return {
        "router": ("hbm", 2 * T * d + 4 * T * E + 8 * R + 2 * d * E),
        "permute": ("hbm", 2 * T * d + 2 * R * d + 12 * R),
        "gemm_gateup_swiglu": ("tensor", 4 * R * d * f),
        "gemm_down": ("tensor", 2 * R * f * d),
        "combine": ("hbm", 2 * R * d + 2 * T * d + 8 * R),
        "combine_bwd": ("hbm", 2 * T * d + 2 * R * d + 4 * R),  # gather of dy rows (dg moved into the dgrad-down epilogue)
        "dgrad_down_swiglu_bwd": ("tensor", 2 * R * d * f),
        "wgrad_down": ("tensor", 2 * R * f * d),
        "dgrad_gateup": ("tensor", 4 * R * f * d),
        "wgrad_gateup": ("tensor", 4 * R * d * f),
        "router_bwd": ("hbm", 8 * T * E + 12 * R),
        "dW_r": ("hbm", 2 * T * d + 4 * T * E + 4 * d * E),
        "unpermute_bwd": ("hbm", 2 * R * d + 2 * T * d + 2 * T * d),
        "dx_router_term": ("hbm", 4 * T * E + 2 * T * d + 2 * d * E),
    }


class ClockSampler:
    """Samples the SM clock and the throttle reasons of one GPU every few milliseconds (NVML through pynvml; falls back
    to `nvidia-smi -lms 20`), each sample stamped with the host clock, so that summary(t0, t1) can keep only the samples
    that fall inside the timed region.  Read-only: no GPU setting is touched."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_s: float = 0.004):
        self.idx = gpu_index
        self.period = period_s
        self.samples = []  # (host time, sm MHz, max MHz, set of reasons)
        self.proc = None
        self.th = None
        self.stop_flag = False
        self.source = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.idx
            if vis:
                ent = vis.split(",")[self.idx].strip()
                phys = int(ent) if ent.isdigit() else self.idx
            h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            mx = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            bits = {"hw_slowdown": pynvml.nvmlClocksEventReasonHwSlowdown if hasattr(pynvml, "nvmlClocksEventReasonHwSlowdown") else 0x8,
                    "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

            def loop():
                while not self.stop_flag:
                    try:
                        mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                        try:
                            mask = int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                        except Exception:
                            mask = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                        self.samples.append((time.perf_counter(), mhz, mx, {n for n, b in bits.items() if mask & b}))
                    except Exception:
                        pass
                    time.sleep(self.period)
            self.th = threading.Thread(target=loop, daemon=True)
            self.th.start()
            self.source = "nvml"
            return
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
            self.source = "nvidia-smi"
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 9:
                continue
            try:
                sm, mx = float(p[1]), float(p[2])
            except ValueError:
                continue
            rs = {n for n, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9])
                  if v.lower().startswith("active")}
            self.samples.append((time.perf_counter(), sm, mx, rs))

    def stop(self):
        self.stop_flag = True
        if self.proc is not None:
            time.sleep(0.05)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                self.proc.kill()
        elif self.th is not None:
            self.th.join(timeout=1)

    def summary(self, t0: float, t1: float):
        """Median SM clock and the union of throttle reasons over the samples taken in [t0, t1] (host clock)."""
        if self.source is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock sampling unavailable"], "samples": 0}
        inside = [x for x in self.samples if t0 <= x[0] <= t1]
        note = None
        if not inside and self.samples:  # region shorter than one sampling period: nearest sample
            mid = 0.5 * (t0 + t1)
            inside = [min(self.samples, key=lambda x: abs(x[0] - mid))]
            note = "region shorter than the sampling period: nearest sample"
        reasons = set()
        for x in inside:
            reasons |= x[3]
        out = {"sm_mhz": float(np.median([x[1] for x in inside])) if inside else None,
               "sm_max_mhz": max(x[2] for x in inside) if inside else None, "reasons": sorted(reasons),
               "samples": len(inside), "source": self.source}
        if note:
            out["note"] = note
        return out


def choose_peak(peaks: dict, sm_mhz, sm_max_mhz):
    """Which measured bf16 peak describes the regime the timed region ran in.  The sustained figure was measured with
    the SM clock settled under the power cap (about 1300 MHz on this part), the burst figure near the maximum clock;
    the timed region's own median clock decides, halfway between the two being the dividing line."""
    sustained_mhz = float(peaks.get("sustained_sm_mhz", 1297.0))
    top = float(sm_max_mhz or peaks.get("sm_max_mhz", 1965.0))
    if sm_mhz is None:
        return "sustained", peaks["bf16_tflops_sustained"]
    if sm_mhz >= 0.5 * (sustained_mhz + top):
        return "burst", peaks["bf16_tflops"]
    return "sustained", peaks["bf16_tflops_sustained"]


def oracle_sample_tokens_per_s(inp, shape, sample_T, repeats=1):
    """Times the CPU oracle (float32 mode, as it stands) on the first sample_T tokens of the workload."""
    from oracle import moe_oracle as orc
    sl = slice(0, sample_T)
    t0 = time.perf_counter()
    for _ in range(repeats):
        fw = orc.forward(inp["x"][sl], inp["W_r"], inp["W_gate"], inp["W_up"], inp["W_down"], shape.k,
                         b_r=inp.get("b_r"), dtype=np.float32)
        orc.backward(fw, inp["dy"][sl], inp["d_aux"], inp["x"][sl], inp["W_r"], inp["W_gate"], inp["W_up"],
                     inp["W_down"], dtype=np.float32)
    dt = (time.perf_counter() - t0) / repeats
    return sample_T / dt, dt


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def workload_config(workload, mode, shape, world, parallelism_note="no data-path collective"):
    """The `config` object of the JSON line: what identifies the workload.  Both arms print the same object for the same
    command-line arguments; what differs between runs (conditioning steps, redrawn tokens, the reference arm's sample)
    sits beside it."""
    w_gb = 3 * shape.E * shape.d * shape.f * 2 / 1e9
    l2_note = (f"inputs larger than L2 ({w_gb:.2f} GB of expert weights streamed per pass); no explicit flush"
               if w_gb > 0.2 else f"working set ({w_gb * 1e3:.0f} MB of weights) fits in L2: L2-warm, launch-bound numbers")
    return {"workload": workload, "mode": mode, "T_per_gpu": shape.T, "d": shape.d, "E": shape.E, "top_k": shape.k,
            "f": shape.f,
            "parallelism": f"dp{world} over tokens, experts replicated (EP=1), " + parallelism_note,
            "l2": l2_note}


def routing_report(counts, meta):
    """The realised per-expert load of the last timed step (the GPU's own counts) and what the generator did to get it."""
    c = np.asarray(counts, dtype=np.int64)
    rows = int(c.sum())
    padded = int(((c + 127) // 128 * 128).sum())
    return {"rows_per_expert": {"min": int(c.min()), "max": int(c.max()), "mean": float(c.mean())},
            "empty_experts": int((c == 0).sum()), "largest_five": sorted((int(v) for v in c), reverse=True)[:5],
            "padding_rows_fraction": (padded - rows) / rows if rows else 0.0,
            "zipf_bias_alpha": meta.get("alpha"), "redrawn_tokens": meta.get("redrawn")}


def run_reference(args, shape, inp, workload):
    """--impl reference: the oracle is the timed arm (bounded sample per step)."""
    sample_T = min(shape.T, 2048)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_tokens_per_s(inp, shape, sample_T)
    times = []
    for _ in range(args.steps):
        _, dt = oracle_sample_tokens_per_s(inp, shape, sample_T)
        times.append(dt)
    ms = 1e3 * float(np.mean(times))
    val = sample_T / (ms / 1e3)
    cores = host_cores()
    line = {"impl": "reference", "metric": "moe_layer_fwd_bwd_tokens_per_s", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(workload, "train", shape, args.gpus),
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": f"each step: the first {sample_T} of the batch's {shape.T} tokens, all {shape.E} "
                                       f"experts' weights, fp32 numpy, forward + backward"},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="qwen", choices=list(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ep-world", type=int, default=4, help="--mode ep: ranks of the expert-parallel group")
    ap.add_argument("--mode", default="train", choices=["train", "inference", "accumulate", "lora", "library-gemm", "ep"],
                    help="train: forward + backward (the headline metric); inference: forward-only entry point; "
                         "accumulate: forward + backward that adds weight gradients into fp32 buffers; "
                         "lora: forward + backward of the expert-LoRA variant (rank 16, frozen expert weights); "
                         "ep: the expert-parallel path with all ranks of the group run as a local group on ONE GPU (same "
                         "kernels as a multi-GPU group, phases enqueued rank after rank; the batch is split evenly over the "
                         "ranks, so the work equals one train step and the difference is the cost of the EP path itself); "
                         "library-gemm: calibration only - the library's batched bf16 GEMM (torch.bmm) at the three "
                         "row-GEMM shapes of the workload with uniform rows per expert, in the same steady state")
    ap.add_argument("--condition-seconds", type=float, default=2.0,
                    help="untimed back-to-back steps before the timed region, so that the timed steps run in the "
                         "power-capped steady state the sustained peak describes (0 disables)")
    ap.add_argument("--micro-batches", type=int, default=4,
                    help="accumulate mode: steps per accumulation window (gradients are summed over the ranks and the "
                         "buffers zeroed once per window)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay of the step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2608_00916_b200 import dist as pdist
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # started by hand as `python bench.py --gpus N`: become the launcher of N ranks (one process per GPU)
        raise SystemExit(pdist.launch_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    shape, seed, x_std, skew = synth.CONFIGS[args.workload]

    if args.impl == "reference":
        if rank != 0:
            return
        inp = synth.make_inputs(shape, seed, x_std=x_std, skew=skew)
        run_reference(args, shape, inp, args.workload)
        return

    import torch
    from paper_2608_00916_b200.binding import MoELayer, STAGE_NAMES, kernel_launches

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the CUDA path has no CPU fallback)")
    if world > torch.cuda.device_count():
        raise SystemExit(f"bench.py: {world} ranks but only {torch.cuda.device_count()} visible GPUs")
    torch.cuda.set_device(local_rank)
    pdist.init(world, rank, backend="nccl")

    # every rank draws its own token batch (data parallel over tokens, weights replicated: same seed for weights);
    # the batch of rank r > 0 is guarded against the SHARED router weight and bias
    inp = synth.make_inputs(shape, seed, x_std=x_std, skew=skew)
    if rank > 0:
        shard = synth.make_tokens(shape, pdist.shard_seed(seed, rank), inp["W_r"], inp["b_r"], x_std=x_std)
        inp["x"], inp["dy"] = shard["x"], shard["dy"]
        inp["meta"]["redrawn"] = shard["redrawn"]

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    T = shape.T
    layer = MoELayer(shape.d, shape.E, shape.f, shape.k)
    tens = {n: dev(inp[n]) for n in ("x", "W_r", "W_gate", "W_up", "W_down", "dy")}
    b_r = None if inp.get("b_r") is None else torch.from_numpy(inp["b_r"]).cuda()
    grads = {"dx": torch.empty_like(tens["x"]), "dW_r": torch.empty(shape.d, shape.E, dtype=torch.float32, device="cuda"),
             "dW_gate": torch.empty_like(tens["W_gate"]), "dW_up": torch.empty_like(tens["W_up"]),
             "dW_down": torch.empty_like(tens["W_down"])}

    if args.mode == "ep":
        from paper_2608_00916_b200 import ep as pep
        W = args.ep_world
        assert shape.E % W == 0 and T % W == 0
        per = T // W
        xs = [tens["x"][r * per:(r + 1) * per].contiguous() for r in range(W)]
        dys = [tens["dy"][r * per:(r + 1) * per].contiguous() for r in range(W)]
        grp = pep.LocalGroup(shape.d, shape.E, shape.f, shape.k, W, pep.rows_cap_bound([per] * W, shape.k, shape.E, W))

        def estep():
            grp.forward(xs, tens["W_r"], tens["W_gate"], tens["W_up"], tens["W_down"], b_r=b_r)
            grp.backward(dys, inp["d_aux"])
        for _ in range(args.warmup):
            estep()
        grp.poll()
        t_c = time.perf_counter()
        while time.perf_counter() - t_c < args.condition_seconds:
            for _ in range(5):
                estep()
            torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = kernel_launches()
        f0.record()
        for _ in range(args.steps):
            estep()
        f1.record()
        torch.cuda.synchronize()
        grp.poll()
        ms = f0.elapsed_time(f1) / args.steps
        print(json.dumps({"metric": "moe_layer_ep_local_group_fwd_bwd_tokens_per_s", "value": T / (ms / 1e3),
                          "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "none", "vs_baseline": None, "dtype": "bf16",
                          "data": "synthetic",
                          "config": {"workload": args.workload, "mode": "ep", "ep_world": W, "tokens_per_rank": per,
                                     "experts_per_rank": shape.E // W, "d": shape.d, "E": shape.E, "top_k": shape.k,
                                     "f": shape.f,
                                     "note": "all ranks of the group on one GPU, phases enqueued rank after rank; not a "
                                             "multi-GPU measurement"},
                          "gpu_launches": kernel_launches() - launches0}))
        pdist.finish()
        return

    if args.mode == "library-gemm":
        # What a plain library GEMM reaches at the expert shapes under the same power-capped steady state: no ragged
        # rows, no padding, no fused epilogue, one output.  Context for the roofline fractions, not a product path.
        rows = max(1, (T * shape.k) // shape.E)
        out = {}
        for name, (M, K, N) in {"gate_up (hg | hu)": (rows, shape.d, 2 * shape.f), "down": (rows, shape.f, shape.d),
                                "dgrad_down": (rows, shape.d, shape.f)}.items():
            a = torch.randn(shape.E, M, K, device="cuda", dtype=torch.bfloat16)
            b = torch.randn(shape.E, K, N, device="cuda", dtype=torch.bfloat16) * 0.02
            c = torch.empty(shape.E, M, N, device="cuda", dtype=torch.bfloat16)
            t_c = time.perf_counter()
            while time.perf_counter() - t_c < max(args.condition_seconds, 0.2):
                for _ in range(20):
                    torch.bmm(a, b, out=c)
                torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record()
            for _ in range(args.steps):
                torch.bmm(a, b, out=c)
            g1.record()
            torch.cuda.synchronize()
            ms = g0.elapsed_time(g1) / args.steps
            out[name] = {"E_M_K_N": [shape.E, M, K, N], "us": 1e3 * ms, "TFLOP/s": 2 * shape.E * M * K * N / (ms * 1e-3) / 1e12}
            del a, b, c
        if rank == 0:
            print(json.dumps({"metric": "library_batched_gemm_tflops", "unit": "TFLOP/s", "dtype": "bf16", "data": "synthetic",
                              "config": {"workload": args.workload, "mode": "library-gemm", "rows_per_expert": rows},
                              "shapes": out, "steps": args.steps, "n_gpus": world,
                              "note": "torch.bmm (cuBLAS) after the same untimed conditioning; calibration, not a product path"}))
        pdist.finish()
        return

    if args.mode == "lora":
        # expert-LoRA training step (a "next" row beyond the full fine-tuning step): own metric, device-resident timing
        rank, scale = 16, 2.0
        lo = synth.make_lora(shape, seed, rank=rank)
        dlo = {n: dev(lo[n]) for n in ("A1", "B1_gate", "B1_up", "A2", "B2")}

        def lstep():
            layer.lora_forward(tens["x"], tens["W_r"], tens["W_gate"], tens["W_up"], tens["W_down"], dlo, scale, b_r=b_r)
            layer.lora_backward(tens["dy"], inp["d_aux"])
        for _ in range(args.warmup):
            lstep()
        layer.poll()
        layer.set_profiling(True)
        pdist.barrier()
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        launches0 = kernel_launches()
        for _ in range(args.steps):
            lstep()
        f1.record()
        torch.cuda.synchronize()
        pdist.barrier()
        stage_ms, n = layer.stage_times()
        ms = pdist.max_over_ranks(f0.elapsed_time(f1)) / args.steps
        if int(os.environ.get("RANK", "0")) == 0:
            Rr = T * shape.k
            fl = 12 * Rr * shape.d * shape.f  # base forward + dgrad GEMMs; the low-rank terms add < 3 %
            print(json.dumps({"metric": "moe_layer_lora_fwd_bwd_tokens_per_s", "value": world * T / (ms / 1e3),
                              "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                              "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                              "dtype": "bf16", "data": "synthetic",
                              "config": {"workload": args.workload, "mode": "lora", "rank": rank, "T_per_gpu": T,
                                         "d": shape.d, "E": shape.E, "top_k": shape.k, "f": shape.f},
                              "base_gemm_useful_tflops_over_whole_step": fl / (ms * 1e-3) / 1e12,
                              "stages_ms": {STAGE_NAMES[i]: stage_ms[i] / max(n, 1) for i in range(len(STAGE_NAMES))},
                              "gpu_launches": kernel_launches() - launches0}))
        pdist.finish()
        return

    if args.mode == "inference":
        # forward-only scoring pass (a "next" row beyond the training step): own metric, device-resident timing only
        def fstep():
            layer.forward(tens["x"], tens["W_r"], tens["W_gate"], tens["W_up"], tens["W_down"], b_r=b_r, want_perm=False,
                          inference=True)
        for _ in range(args.warmup):
            fstep()
        layer.poll()
        pdist.barrier()
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        launches0 = kernel_launches()
        for _ in range(args.steps):
            fstep()
        f1.record()
        torch.cuda.synchronize()
        pdist.barrier()
        ms = pdist.max_over_ranks(f0.elapsed_time(f1)) / args.steps
        if rank == 0:
            fl = 6 * T * shape.k * shape.d * shape.f
            print(json.dumps({"metric": "moe_layer_fwd_tokens_per_s", "value": world * T / (ms / 1e3), "unit": "tokens/s",
                              "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                              "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                              "data": "synthetic", "config": {"workload": args.workload, "mode": "inference",
                                                              "T_per_gpu": T, "d": shape.d, "E": shape.E,
                                                              "top_k": shape.k, "f": shape.f},
                              "grouped_gemm_useful_tflops_over_whole_pass": fl / (ms * 1e-3) / 1e12,
                              "gpu_launches": kernel_launches() - launches0}))
        pdist.finish()
        return

    acc = None
    if args.mode == "accumulate":
        acc = {"dW_r": torch.zeros(shape.d, shape.E, device="cuda"),
               "dW_gate": torch.zeros(shape.E, shape.d, shape.f, device="cuda"),
               "dW_up": torch.zeros(shape.E, shape.d, shape.f, device="cuda"),
               "dW_down": torch.zeros(shape.E, shape.f, shape.d, device="cuda")}

    reducer = pdist.GradAllReducer() if (acc is not None and world > 1) else None
    window = max(1, args.micro_batches)
    step_no = [0]

    def step():
        layer.forward(tens["x"], tens["W_r"], tens["W_gate"], tens["W_up"], tens["W_down"], b_r=b_r, want_perm=False)
        if acc is not None:
            # an accumulation window of `window` micro-batches: the buffers start at zero, every step adds its weight
            # gradients, the last step of the window is followed by the sum over the ranks (which then overlaps the next
            # step's forward); the optimizer would consume the buffers where they are zeroed here
            if step_no[0] % window == 0:
                if reducer is not None:
                    reducer.wait()
                for t in acc.values():
                    t.zero_()
            last = (step_no[0] + 1) % window == 0
            # the window's last micro-batch runs its weight gradients in ranges of experts and signals each range, so
            # that the sum over the ranks of a finished range overlaps the rest of this backward pass
            layer.backward_accumulate(tens["dy"], inp["d_aux"], acc,
                                      group_events=reducer.events() if (reducer is not None and last) else None)
            step_no[0] += 1
            if reducer is not None and last:
                reducer.start_grouped(acc)
        else:
            layer.backward(tens["dy"], inp["d_aux"], grads=grads)

    for _ in range(args.warmup):
        step()
    layer.poll()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    # A short look at the burst regime first (informative only, reported under "burst"): min(steps, 20) steps right after
    # the warm-up, before the power cap has pulled the clocks down.  The headline below is the steady state.
    burst = None
    if args.condition_seconds > 0:
        nb = max(3, min(args.steps, 20))
        layer.set_profiling(True)
        torch.cuda.synchronize()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        tb0 = time.perf_counter()
        b0.record()
        for _ in range(nb):
            step()
        b1.record()
        torch.cuda.synchronize()
        tb1 = time.perf_counter()
        bst, bn = layer.stage_times()
        layer.set_profiling(False)
        burst = {"steps": nb, "ms_per_step": b0.elapsed_time(b1) / nb,
                 "stages_ms": {STAGE_NAMES[i]: bst[i] / max(bn, 1) for i in range(len(STAGE_NAMES))},
                 "window": (tb0, tb1)}
    # untimed conditioning: the same step back to back until the power state has settled
    cond_steps = 0
    if args.condition_seconds > 0:
        t_c = time.perf_counter()
        while time.perf_counter() - t_c < args.condition_seconds:
            for _ in range(10):
                step()
            torch.cuda.synchronize()
            cond_steps += 10
    layer.poll()
    layer.set_profiling(True)
    pdist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = kernel_launches()
    t_host0 = time.perf_counter()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    t_host1 = time.perf_counter()
    launches = kernel_launches() - launches0
    # per-stage CUDA events were recorded on the stream inside the calls, one set per step
    stage_ms, prof_steps = layer.stage_times()
    pdist.barrier()
    clocks = None
    if rank == 0:
        clocks = sampler.summary(t_host0, t_host1)
        if burst is not None:
            w0, w1 = burst.pop("window")
            burst["sm_mhz"] = sampler.summary(w0, w1).get("sm_mhz")
            burst["tokens_per_s"] = world * T / (burst["ms_per_step"] / 1e3)
            burst["note"] = ("first steps after the warm-up, before the power cap settles the clock; not the headline "
                             "(the headline value is the conditioned steady state)")
    layer.poll()
    layer.set_profiling(False)
    ms_step = pdist.max_over_ranks(ev0.elapsed_time(ev1)) / args.steps
    value = pdist.job_throughput(T, ms_step)  # tokens of all ranks over the slowest rank's time

    # ---- the same step replayed from a CUDA graph (informative: what a training loop that captures its step gets; the
    # library's calls are legal inside a stream capture, second stream included).  Only the plain training step.
    graph = None
    if args.mode == "train" and acc is None and not args.no_graph:
        try:
            cap = torch.cuda.Stream()
            cap.wait_stream(torch.cuda.current_stream())
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(cap):
                step()
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=cap):
                    step()
            torch.cuda.synchronize()
            for _ in range(max(3, args.warmup)):
                g.replay()
            t_c = time.perf_counter()  # the capture paused the GPU: settle the power state again, as for the headline
            while time.perf_counter() - t_c < args.condition_seconds:
                for _ in range(10):
                    g.replay()
                torch.cuda.synchronize()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()  # no collective in this block: a rank that fails here must not strand the others
            g0.record()
            for _ in range(args.steps):
                g.replay()
            g1.record()
            torch.cuda.synchronize()
            layer.poll()
            gms = g0.elapsed_time(g1) / args.steps
            graph = {"ms_per_step": gms, "tokens_per_s_this_rank": T / (gms / 1e3), "steps": args.steps,
                     "note": "this rank's timed step captured once and replayed after the same conditioning (no per-stage "
                             "events, one launch per step); informative, the headline is the eager step"}
            del g
        except Exception as exc:  # the informative block must never cost the benchmark line
            graph = {"unavailable": f"{type(exc).__name__}: {exc}"[:200]}
            torch.cuda.synchronize()

    # ---- end to end through the host-buffer entry point (weights resident, activations cross PCIe each step)
    e2e = None
    if not args.no_e2e:
        host = {n: torch.from_numpy(inp[n].view(np.int16)).pin_memory() for n in ("x", "dy", "W_r", "W_gate", "W_up", "W_down")}
        host["y"] = torch.empty(T, shape.d, dtype=torch.int16).pin_memory()
        host["dx"] = torch.empty(T, shape.d, dtype=torch.int16).pin_memory()
        host["aux"] = torch.empty(1, dtype=torch.float32).pin_memory()
        host["dW_r"] = torch.empty(shape.d, shape.E, dtype=torch.float32).pin_memory()
        for n in ("dW_gate", "dW_up", "dW_down"):
            host[n] = torch.empty(inp["W_gate"].size if n != "dW_down" else inp["W_down"].size, dtype=torch.int16).pin_memory()
        dev_buf = torch.empty(layer.e2e_device_bytes(T), dtype=torch.uint8, device="cuda")
        layer.step_host(T, dev_buf, host, inp["d_aux"], copy_weights=True)  # uploads the weights once (untimed)
        # timed: the pipelined host step (two slots in flight, as a training loop that prefetches its next batch
        # would call it); every step still uploads its x, dy and downloads its y, dx, aux inside the timed region
        slots = [dict(host, y=torch.empty(T, shape.d, dtype=torch.int16).pin_memory(),
                      dx=torch.empty(T, shape.d, dtype=torch.int16).pin_memory(),
                      aux=torch.empty(1, dtype=torch.float32).pin_memory()) for _ in range(2)]

        def run_pipelined(n):
            layer.step_host_begin(0, T, dev_buf, slots[0], inp["d_aux"])
            for i in range(1, n):
                layer.step_host_begin(i % 2, T, dev_buf, slots[i % 2], inp["d_aux"])
                layer.step_host_end((i - 1) % 2)
            layer.step_host_end((n - 1) % 2)
        run_pipelined(3)
        # the same untimed conditioning as for the device-resident number (setting up the pinned buffers above took
        # long enough for the power state to relax)
        t_c = time.perf_counter()
        while time.perf_counter() - t_c < args.condition_seconds:
            run_pipelined(20)
        pdist.barrier()
        torch.cuda.synchronize()
        # as many steps as the device-resident region: the pipeline's fill (the first step's inputs) and drain (the last
        # step's results) are inside the timed region and weigh 1/n of it
        n_e2e = max(4, args.steps)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_e0 = time.perf_counter()
        p0.record()
        run_pipelined(n_e2e)  # returns after the last step's results have reached the host buffers
        p1.record()
        torch.cuda.synchronize()
        t_e1 = time.perf_counter()
        pdist.barrier()
        e2e_ms = pdist.max_over_ranks(p0.elapsed_time(p1)) / n_e2e
        layer.poll()
        # the blocking single-call form for comparison
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            layer.step_host(T, dev_buf, host, inp["d_aux"], copy_weights=False)
        e1.record()
        torch.cuda.synchronize()
        blocking_ms = e0.elapsed_time(e1) / 3
        td = 2 * T * shape.d
        e2e = {"value": world * T / (e2e_ms / 1e3), "unit": "tokens/s", "h2d_bytes_per_step": 2 * td,
               "d2h_bytes_per_step": 2 * td + 4, "steps": n_e2e, "ms_per_step": e2e_ms,
               "ms_per_step_blocking_call": blocking_ms,
               "sm_mhz": sampler.summary(t_e0, t_e1).get("sm_mhz") if rank == 0 else None,
               "note": "moe_step_host_begin/end with two slots in flight: x, dy in and y, dx, aux out every step; the closing "
                       "CUDA event is recorded after the last step's results reached the host; weights and weight "
                       "gradients stay on the device"}
        del dev_buf
    if rank == 0:
        sampler.stop()

    if rank != 0:
        pdist.finish()
        return

    peaks = load_peaks()
    work = stage_work(shape)
    regime, tensor_peak = choose_peak(peaks, clocks.get("sm_mhz"), clocks.get("sm_max_mhz"))
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    mhz = clocks.get("sm_mhz")
    stages = {}
    gemm_flops = gemm_ms = 0.0
    for i, name in enumerate(STAGE_NAMES):
        ms = stage_ms[i] / max(prof_steps, 1)
        kind, amount = work[name]
        if kind == "tensor":
            ach = amount / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
            stages[name] = {"ms": ms, "TFLOP/s": ach, "frac_of_sustained": ach / peaks["bf16_tflops_sustained"],
                            "frac_of_burst": ach / peaks["bf16_tflops"]}
            if mhz and ms > 0:
                stages[name]["flop_per_clk_per_sm"] = amount / (ms * 1e-3 * mhz * 1e6 * sm_count)
            gemm_flops += amount
            gemm_ms += ms
        else:
            ach = amount / (ms * 1e-3) / 1e9 if ms > 0 else 0.0
            stages[name] = {"ms": ms, "GB/s": ach, "frac_of_hbm": ach / peaks["hbm_gbs"]}
    # the router's gradient chain runs on the context's second stream beside the weight-gradient and dgrad GEMMs: its
    # event-to-event times include waiting for free SMs, so they say nothing about the kernels and cannot dominate
    for name in OVERLAPPED_STAGES:
        stages[name]["overlapped"] = "second stream, beside the expert GEMMs; time includes waiting for SMs"
    dom = max((n for n in STAGE_NAMES if n not in OVERLAPPED_STAGES), key=lambda n: stages[n]["ms"])
    kind, amount = work[dom]
    if kind == "tensor":
        roof = {"bound": "tensor", "kernel": dom, "achieved": stages[dom]["TFLOP/s"], "peak": tensor_peak,
                "unit": "TFLOP/s", "frac": stages[dom]["TFLOP/s"] / tensor_peak,
                "peak_source": f"{peaks['source']} bf16 {regime} (median SM clock of the timed region "
                               f"{mhz} MHz; sustained peak measured at {peaks['sustained_sm_mhz']:.0f} MHz, burst near "
                               f"{peaks['sm_max_mhz']:.0f} MHz)",
                "frac_of_burst": stages[dom]["frac_of_burst"], "frac_of_sustained": stages[dom]["frac_of_sustained"],
                # the sustained peak rescaled to the clock this region ran at (that peak was measured at
                # sustained_sm_mhz; a box that settles at a lower clock under the same cap has a lower ceiling)
                "frac_of_sustained_at_this_clock": (stages[dom]["TFLOP/s"] / (peaks["bf16_tflops_sustained"] * mhz /
                                                                             peaks["sustained_sm_mhz"])) if mhz else None,
                "flop_per_clk_per_sm": stages[dom].get("flop_per_clk_per_sm"),
                "traffic": NCU_TRAFFIC.get((args.workload, dom))}
    else:
        roof = {"bound": "hbm", "kernel": dom, "achieved": stages[dom]["GB/s"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": stages[dom]["GB/s"] / peaks["hbm_gbs"], "peak_source": peaks["source"] + " copy bandwidth",
                "traffic": NCU_TRAFFIC.get((args.workload, dom))}
    gemm_tflops = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0

    cpu = None
    if not args.no_cpu_baseline and world == 1:  # the oracle is timed beside the one-GPU run only
        sample_T = min(T, 16384)
        v, dt = oracle_sample_tokens_per_s(inp, shape, sample_T)
        cpu = {"value": v, "unit": "tokens/s", "cores": host_cores(), "kind": "oracle", "seconds": dt,
               "sample": f"first {sample_T} tokens of the batch through the fp32 numpy oracle, forward + backward, "
                         f"all {shape.E} experts' weights"}

    line = {"metric": "moe_layer_fwd_bwd_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(args.workload, args.mode, shape, world,
                                      "weight gradients all-reduced once per accumulation window, range by range of "
                                      "experts while the backward pass still runs" if reducer is not None
                                      else "no data-path collective"),
            "conditioning": f"{cond_steps} untimed steps (>= {args.condition_seconds} s) before the timed region",
            "routing": routing_report(layer.buffer("counts", torch.int32).cpu().numpy(), inp["meta"]),
            "grouped_gemm_tflops": gemm_tflops,
            "grouped_gemm_frac_of_sustained_bf16": gemm_tflops / peaks["bf16_tflops_sustained"],
            "grouped_gemm_frac_of_burst_bf16": gemm_tflops / peaks["bf16_tflops"],
            "grouped_gemm_frac_of_regime_peak": gemm_tflops / tensor_peak, "regime": regime,
            "roofline": roof, "stages": stages, "burst": burst, "graph_replay": graph, "cpu_baseline": cpu, "e2e": e2e,
            "clocks": clocks,
            "gpu_launches": launches}
    print(json.dumps(line))
    pdist.finish()


if __name__ == "__main__":
    main()
