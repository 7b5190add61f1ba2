#!/usr/bin/env python
"""Benchmark of the bidirectional Mamba-2 mixer layer (the hot path of one denoising step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" = one dm_bimamba_forward call (in_proj, fused conv+scan+gate of both directions, out_proj and
the sum of directions) over one batch of synthetic activations.  Metric: denoised tokens/s per
bidirectional Mamba layer.  N > 1 runs N independent replicas (one process per GPU, no data-path
collective); the value is the tokens all ranks processed divided by the slowest rank's device time.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_15927_b200 import inputs as I  # noqa: E402

METRIC = "denoised tokens/s per bidirectional Mamba layer"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused scan kernel, from the ncu captures
# summarised under profiles/ (None = not captured for that workload).
NCU_SCAN_TRAFFIC_BYTES = {}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def scan_bytes_per_token(s: I.MixerShape, es: int, gated_norm: bool = True) -> int:
    """Algorithmic HBM bytes of the fused conv+scan+gate launch per token, both directions: it reads each
    direction's in_proj row (z, x, B, C, dt) once and writes the gated output once (plus, with the gated
    norm, one fp32 sum of squares per head)."""
    return 2 * ((s.d_in_proj + s.d_inner) * es + (4 * s.n_heads if gated_norm else 0))


def gemm_flops_per_token(s: I.MixerShape):
    return 2 * 2 * s.d_model * s.d_in_proj, 2 * 2 * s.d_inner * s.d_model


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only queries) from a thread while the timed
    region runs."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, gpu_index: int, period_s: float = 0.005):
        import threading
        self.sm, self.power, self.bits, self.err = [], [], 0, None
        self.max_sm = None
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = None
            try:                                     # the CUDA device's own UUID names the NVML device unambiguously
                import torch
                self.h = pynvml.nvmlDeviceGetHandleByUUID("GPU-" + str(torch.cuda.get_device_properties(gpu_index).uuid))
            except Exception:
                self.h = None
            if self.h is None:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
                ids = [v.strip() for v in vis.split(",") if v.strip()]
                phys = int(ids[gpu_index]) if len(ids) > gpu_index and ids[gpu_index].isdigit() else gpu_index
                self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                       # no NVML: report that, never guess
            self.err = f"nvml unavailable: {e}"
            self.t = None
            return
        self.period = period_s
        self.t = threading.Thread(target=self._run, daemon=True)
        self.t.start()

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                self.bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception as e:
                self.err = str(e)
                return
            self._stop.wait(self.period)

    def stop(self) -> dict:
        if self.t is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.err or "no sampler"]}
        self._stop.set()
        self.t.join(timeout=2)
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": [self.err or "no samples"]}
        return {"sm_mhz": float(np.median(self.sm)), "sm_max_mhz": self.max_sm, "power_w_max": float(max(self.power)),
                "samples": len(self.sm), "reasons": sorted(n for n, b in self.REASONS if self.bits & b)}


def oracle_sample_seconds(shape: I.MixerShape, dtype: str, sample_len: int, seed: int = 0):
    """Time the fp64 oracle, as it stands, on batch row 0 truncated to sample_len tokens of the workload."""
    from oracle import bimamba_oracle as O
    s = I.MixerShape(1, sample_len, shape.d_model, shape.expand, shape.d_state, shape.d_conv, shape.n_heads, shape.n_groups)
    wf, wr = I.make_mixer_weights(s, seed, dtype)
    x = I.make_activations(s, seed, dtype)
    t0 = time.perf_counter()
    O.bimamba_forward(x, wf, wr, expand=s.expand, d_state=s.d_state, n_heads=s.n_heads, n_groups=s.n_groups)
    return time.perf_counter() - t0


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return int(max(n)) if n else 1
    except Exception:
        return 1


def run_reference(args, shape, dtype, rank):
    """The reference arm: the CPU oracle on the host cores, each step a bounded sample of the workload."""
    if rank != 0:
        return
    sample = min(shape.seqlen, args.ref_tokens)
    for _ in range(args.warmup):
        oracle_sample_seconds(shape, dtype, sample)
    t = [oracle_sample_seconds(shape, dtype, sample) for _ in range(args.steps)]
    sec = float(np.sum(t))
    value = sample * args.steps / sec
    desc = f"batch row 0, first {sample} tokens of {args.workload} per step (full widths, both directions)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg1", choices=sorted(I.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=128, help="tokens per step of the reference arm's sample")
    ap.add_argument("--cpu-baseline-tokens", type=int, default=2048)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = max(args.warmup, 1) if args.impl == "reference" else 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    shape, dtype = I.CONFIGS[args.workload]

    if args.impl == "reference":
        run_reference(args, shape, dtype, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2511_15927_b200 import build
    if rank == 0 or world == 1:
        build.build()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2511_15927_b200 import binding as dm
    torch.cuda.set_device(local_rank)
    from paper_2511_15927_b200 import torch_io as G

    es = 2 if dtype == I.BF16 else 4
    T = shape.batch * shape.seqlen
    cfg = G.cfg_of(shape, dtype)
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    dwf, dwr = G.dev_dir_weights(wf, dtype), G.dev_dir_weights(wr, dtype)
    cw = (dm.make_dir_weights(dwf), dm.make_dir_weights(dwr))
    n_rot = 4                                                   # rotate inputs so that no step finds its x in L2
    x_host = I.make_activations(shape, 0, dtype)
    xs = [G.dev(np.roll(x_host, i, axis=1), dtype) for i in range(n_rot)]
    y = torch.empty_like(xs[0])
    nb = dm.dm_bimamba_workspace_bytes(cfg)
    act_bytes = (T * shape.d_model * es + 255) // 256 * 256
    ws = G.workspace(nb + 2 * act_bytes)
    stream = torch.cuda.current_stream().cuda_stream

    def step(i):
        dm.dm_bimamba_forward(cfg, cw, xs[i % n_rot].data_ptr(), y.data_ptr(), ws.data_ptr(), nb, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    dm.dm_check(stream)
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    dm.dm_profile_enable(True)
    dm.dm_profile_read()
    launches0 = dm.dm_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    launches = dm.dm_kernel_launch_count() - launches0
    stage_ms, stage_n = dm.dm_profile_read()
    dm.dm_profile_enable(False)
    clocks = sampler.stop() if sampler else None
    dm.dm_check(stream)
    if world > 1:
        t = torch.tensor([ms_total], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / args.steps
    value = world * T * args.steps / (ms_total * 1e-3)

    # ---- end to end through the host entry point: pinned host x in, y out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        xh = torch.from_numpy(x_host).to(G.tdtype(dtype)).pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        for _ in range(2):
            dm.dm_bimamba_forward_host(cfg, cw, xh.data_ptr(), yh.data_ptr(), ws.data_ptr(), nb + 2 * act_bytes, stream)
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            dm.dm_bimamba_forward_host(cfg, cw, xh.data_ptr(), yh.data_ptr(), ws.data_ptr(), nb + 2 * act_bytes, stream)
        torch.cuda.synchronize()
        sec = time.perf_counter() - t0
        if world > 1:
            t = torch.tensor([sec], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            sec = float(t.item())
        e2e = {"value": world * T * args.steps / sec, "unit": UNIT, "h2d_bytes_per_step": T * shape.d_model * es,
               "d2h_bytes_per_step": T * shape.d_model * es}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    scan_ms = stage_ms[dm.DM_STAGE_SCAN] / max(stage_n[dm.DM_STAGE_SCAN], 1)
    inp_ms = stage_ms[dm.DM_STAGE_IN_PROJ] / args.steps
    outp_ms = stage_ms[dm.DM_STAGE_OUT_PROJ] / args.steps
    scan_bytes = scan_bytes_per_token(shape, es) * T
    f_in, f_out = gemm_flops_per_token(shape)
    scan_gbs = scan_bytes / (scan_ms * 1e-3) / 1e9
    in_tf = f_in * T / (inp_ms * 1e-3) / 1e12
    out_tf = f_out * T / (outp_ms * 1e-3) / 1e12
    tensor_peak = peaks["bf16_tflops_sustained"]
    kernels = {
        "in_proj": {"ms": inp_ms, "tflops": in_tf, "frac_of_%s_tensor_peak" % peaks["source"]: in_tf / tensor_peak if dtype == I.BF16 else None},
        "scan": {"ms": scan_ms, "gbs": scan_gbs, "frac_of_%s_hbm_peak" % peaks["source"]: scan_gbs / peaks["hbm_gbs"],
                 "frac_of_nominal_8tbs": scan_gbs / 8000.0, "algorithmic_bytes": scan_bytes},
        "out_proj": {"ms": outp_ms, "tflops": out_tf, "frac_of_%s_tensor_peak" % peaks["source"]: out_tf / tensor_peak if dtype == I.BF16 else None},
    }
    dominant = max(("in_proj", inp_ms), ("scan", scan_ms), ("out_proj", outp_ms), key=lambda kv: kv[1])[0]
    if dominant == "scan" or dtype != I.BF16:
        roofline = {"kernel": "fused conv+scan+gate", "bound": "hbm", "achieved": scan_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": scan_gbs / peaks["hbm_gbs"], "traffic": NCU_SCAN_TRAFFIC_BYTES.get(args.workload),
                    "peak_source": peaks["source"] + " (sustained copy)"}
    else:
        tf = in_tf if dominant == "in_proj" else out_tf
        roofline = {"kernel": dominant + " GEMM", "bound": "tensor", "achieved": tf, "peak": tensor_peak, "unit": "TFLOP/s",
                    "frac": tf / tensor_peak, "traffic": None, "peak_source": peaks["source"] + " (sustained bf16)"}

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        n_tok = min(shape.seqlen, args.cpu_baseline_tokens)
        sec = oracle_sample_seconds(shape, dtype, n_tok)
        cpu_baseline = {"value": n_tok / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                        "sample": f"batch row 0, first {n_tok} tokens of {args.workload} (full widths, both directions), {sec:.1f} s"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if dtype == I.BF16 else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "batch": shape.batch, "seq_len": shape.seqlen, "d_model": shape.d_model,
                       "expand": shape.expand, "d_state": shape.d_state, "d_conv": shape.d_conv, "heads": shape.n_heads,
                       "headdim": shape.headdim, "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "l2": f"inputs rotate over {n_rot} buffers; per-step working set "
                             f"{(2 * T * (shape.d_in_proj + shape.d_inner) * es) >> 20} MiB exceeds the 126 MB L2"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "kernels": kernels,
            "cpu_baseline": cpu_baseline}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
