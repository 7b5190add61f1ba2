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
# dram__bytes_read.sum + dram__bytes_write.sum per launch come from the ncu summaries committed under profiles/ (captured on
# cfg3_8k = 8192 tokens; the traffic of both kernels grows in proportion to the token count, so other single-layer bf16
# workloads of the same widths scale it by their tokens; None = no capture applies).
NCU_PROFILES = {"scan": "ssd_scan_cfg3_8k.txt", "in_proj": "gemm_tc_cfg3_8k.txt"}
NCU_TOKENS = 8192
NCU_WIDTHS = (2048, 128, 64)                                             # d_model, d_state, heads the captures were taken at


def profile_traffic(kind):
    """Bytes per launch (DRAM read + write) of the first captured launch in the kernel's profile summary, or None."""
    import re
    path = os.path.join(ROOT, "profiles", NCU_PROFILES.get(kind, ""))
    if not os.path.isfile(path):
        return None
    rd = wr = None
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    with open(path) as f:
        for line in f:
            m = re.match(r"\s*dram__bytes_(read|write)\.sum\s+(\w+)\s+([0-9.eE+-]+)", line)
            if m and m.group(2) in scale:
                v = float(m.group(3)) * scale[m.group(2)]
                if m.group(1) == "read" and rd is None:
                    rd = v
                elif m.group(1) == "write" and wr is None:
                    wr = v
    return rd + wr if rd is not None and wr is not None else None


def ncu_traffic(kind, shape, dtype, tokens):
    if dtype != I.BF16 or (shape.d_model, shape.d_state, shape.n_heads) != NCU_WIDTHS:
        return None
    per_launch = profile_traffic(kind)
    return per_launch / NCU_TOKENS * tokens if per_launch else None


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


def oracle_stack_sample_seconds(spec, n_tok: int, n_layers: int = 2, seed: int = 0):
    """Time the fp64 oracle, as it stands, on a bounded sample of a stack workload: batch row 0, the first n_tok tokens, the
    first n_layers layers at full widths plus the output head.  The metric is per layer, so fewer layers do not change what
    is measured.  Returns (seconds, layers run)."""
    from oracle import bimamba_oracle as O
    sh = spec["shape"]
    s1 = I.MixerShape(1, n_tok, sh.d_model, sh.expand, sh.d_state, sh.d_conv, sh.n_heads, sh.n_groups)
    sw = I.make_stack_weights(s1, n_layers, spec["vocab"], seed=seed, dtype=I.BF16)
    tok = I.make_tokens(1, n_tok, 50257, 50257, seed=seed)
    kw = dict(expand=sh.expand, d_state=sh.d_state, n_heads=sh.n_heads, n_groups=sh.n_groups)
    cond = spec.get("cond")
    if cond:
        I.add_block_weights(sw, s1, cond["d_ff"], cond["d_cond"], seed=seed, dtype=I.BF16)
        tau = I.make_timestep_embedding(1, cond["d_cond"], seed=seed)
    t0 = time.perf_counter()
    if cond:
        O.denoise_step_cond(tok, tau, sw, **kw)
    else:
        O.denoise_step(tok, sw, **kw)
    return time.perf_counter() - t0, n_layers


def host_cores() -> int:
    return int(os.cpu_count() or 1)


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
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "threads_used": blas_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_reference_stack(args):
    """The reference arm on a stack workload: the CPU oracle on a bounded sample (see oracle_stack_sample_seconds)."""
    spec = STACKS[args.workload]
    if spec.get("hybrid"):
        print(json.dumps({"impl": "reference", "unavailable": "the oracle sample covers the Mamba stacks; the hybrid's attention layers are not sampled"}), flush=True)
        return
    n_tok = min(spec["shape"].seqlen, args.ref_tokens)
    for _ in range(min(args.warmup, 1)):
        oracle_stack_sample_seconds(spec, n_tok)
    secs, nl = [], 2
    for _ in range(args.steps):
        sec, nl = oracle_stack_sample_seconds(spec, n_tok)
        secs.append(sec)
    sec = float(np.sum(secs))
    value = n_tok * nl * args.steps / sec
    desc = f"batch row 0, first {n_tok} tokens, first {nl} layers + output head of {args.workload} per step (full widths)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": args.workload, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "threads_used": blas_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# Stack workloads (dm_denoise_step): shape of one step's token tensor, layers, vocabulary; "prefix" marks block decoding.
STACKS = {
    "cfg2_stack": dict(shape=I.MixerShape(4, 4096, 1024, 2, 16, 4, 32), layers=24, vocab=50304),
    "cfg2_stack_n128": dict(shape=I.MixerShape(4, 4096, 1024, 2, 128, 4, 32), layers=24, vocab=50304),
    "cfg4_decode": dict(shape=I.MixerShape(16, 32, 2048, 2, 128, 4, 64), layers=24, vocab=50304, prefix=2048),
    # the same stack with the timestep-conditioned block of App. A.1 in every layer (AdaLN, mixer, AdaLN, MLP with d_ff = 2 d)
    # one reverse step of the masked diffusion (Sec. 2, Eq. 3) on the cfg 2 stack, mid-generation: half of the positions
    # masked, p = 16 of them drawn per sequence and step (K = L / p steps per generation, Sec. 4.3)
    "cfg2_sample": dict(shape=I.MixerShape(4, 4096, 1024, 2, 16, 4, 32), layers=24, vocab=50304, sample=dict(p=16)),
    # the hybrid of Sec. 3.3 on the cfg 2 stack: attention mixer in layers 0, 5, 10, 15, 20 (16 heads of 64), Mamba elsewhere
    "cfg2_stack_hybrid": dict(shape=I.MixerShape(4, 4096, 1024, 2, 16, 4, 32), layers=24, vocab=50304, hybrid=dict(period=5, heads=16)),
    # the paper's 1.3B DiffuMamba (App. A.1: d = 1920, 24 timestep-conditioned blocks, 120 heads of 32, d_state 128, d_ff = 2 d) at its
    # B = 8, L = 1024 throughput point (App. D): one reverse step with p = 16 tokens drawn per sequence, K = L / 16 steps per generation
    "paper_b8_1k_sample": dict(shape=I.MixerShape(8, 1024, 1920, 2, 128, 4, 120), layers=24, vocab=50304,
                               cond=dict(d_ff=3840, d_cond=128), sample=dict(p=16)),
    # the paper's 1.3B hybrid (Sec. 3.3, App. A.3: the same blocks with an attention mixer of 24 heads x 80 channels in every fifth layer)
    "paper_b8_1k_hybrid": dict(shape=I.MixerShape(8, 1024, 1920, 2, 128, 4, 120), layers=24, vocab=50304,
                               cond=dict(d_ff=3840, d_cond=128), hybrid=dict(period=5, heads=24)),
    "cfg2_stack_cond": dict(shape=I.MixerShape(4, 4096, 1024, 2, 16, 4, 32), layers=24, vocab=50304, cond=dict(d_ff=2048, d_cond=128)),
    # block-autoregressive decoding as stated: a 2048-token prefix committed once, then 64 blocks of 32 tokens, each with 8 denoising
    # passes that read the carried state and one commit pass that writes the next block's state (ping-pong); step = one block
    "cfg4_loop": dict(shape=I.MixerShape(16, 32, 2048, 2, 128, 4, 64), layers=24, vocab=50304, prefix=2048, loop=dict(blocks=64, passes=8)),
    # whole generations with dm_generate: K = L / p reverse steps of Eq. 3 plus the clean-up pass, from an all-mask start; step = one generation
    "paper_b8_1k_generate": dict(shape=I.MixerShape(8, 1024, 1920, 2, 128, 4, 120), layers=24, vocab=50304,
                                 cond=dict(d_ff=3840, d_cond=128), generate=dict(p=16)),
    "cfg2_generate_1k": dict(shape=I.MixerShape(4, 1024, 1024, 2, 16, 4, 32), layers=24, vocab=50304, generate=dict(p=16)),
}


def device_stack_weights(torch, shape, layers, vocab, seed=0, cond=None, hybrid=None):
    """Random-init bf16 weights of a stack, drawn on the device with the distributions of inputs.py (the host
    generator would take minutes at these sizes).  Returns the dict layout make_stack_weights() of the binding takes."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    s, bf = shape, torch.bfloat16
    k = s.d_conv

    def normal(*sz):
        return (0.02 * torch.randn(*sz, generator=g, device="cuda", dtype=torch.float32)).to(bf)

    def uniform(lo, hi, *sz):
        return lo + (hi - lo) * torch.rand(*sz, generator=g, device="cuda", dtype=torch.float32)

    def direction():
        dt = torch.exp(uniform(float(np.log(1e-3)), float(np.log(1e-1)), s.n_heads))
        return {"w_in": normal(s.d_in_proj, s.d_model), "conv_w": uniform(-k ** -0.5, k ** -0.5, s.conv_ch, k).to(bf),
                "conv_b": uniform(-k ** -0.5, k ** -0.5, s.conv_ch).to(bf), "A_log": torch.log(uniform(1.0, 16.0, s.n_heads)),
                "dt_bias": dt + torch.log(-torch.expm1(-dt)), "D": torch.ones(s.n_heads, device="cuda"),
                "norm_w": torch.ones(s.d_inner, device="cuda", dtype=bf), "w_out": normal(s.d_model, s.d_inner)}

    def block():
        d, d_ff, d_c = s.d_model, cond["d_ff"], cond["d_cond"]
        base = torch.tensor([0.0, 1.0, 1.0], device="cuda").repeat_interleave(d).repeat(2)      # shift 0, scale 1, gate 1
        return {"w_cond": normal(6 * d, d_c), "b_cond": base + 0.1 * torch.randn(6 * d, generator=g, device="cuda"),
                "w_up": normal(d_ff, d), "b_up": 0.02 * torch.randn(d_ff, generator=g, device="cuda"),
                "w_down": normal(d, d_ff), "b_down": 0.02 * torch.randn(d, generator=g, device="cuda")}

    out = {"embed": normal(vocab, s.d_model), "w_vocab": normal(vocab, s.d_model),
           "final_norm_w": torch.ones(s.d_model, device="cuda", dtype=bf),
           "layers": [{"norm_w": torch.ones(s.d_model, device="cuda", dtype=bf), "fwd": direction(), "rev": direction()}
                      for _ in range(layers)]}
    if cond:
        out["blocks"] = [block() for _ in range(layers)]
    if hybrid:
        d = s.d_model
        out["attn"] = [({"w_qkv": (torch.randn(3 * d, d, generator=g, device="cuda") / d ** 0.5).to(bf),
                         "w_o": (0.5 * torch.randn(d, d, generator=g, device="cuda") / d ** 0.5).to(bf)} if i % hybrid["period"] == 0 else None)
                       for i in range(layers)]
    return out


def run_stack(args, rank, local_rank, world):
    """One step = one dm_denoise_step (embedding, 24 x (RMSNorm, mixer, residual), final norm, vocabulary projection,
    arg-max); cfg2_stack_cond: one dm_denoise_step_cond (24 x the timestep-conditioned block instead).  cfg4_decode: the step covers the 32-token active block of every sequence, starting from the carried
    state of a committed 2048-token prefix; the same stack's full re-encode of prefix + block is timed beside it."""
    import torch
    from paper_2511_15927_b200 import build
    if rank == 0 or world == 1:
        build.build()
    from paper_2511_15927_b200 import dist_util as D
    D.init("nccl", local_rank)
    from paper_2511_15927_b200 import binding as dm
    torch.cuda.set_device(local_rank)
    from paper_2511_15927_b200 import torch_io as G
    spec = STACKS[args.workload]
    shape, layers, vocab, prefix = spec["shape"], spec["layers"], spec["vocab"], spec.get("prefix")
    B, Lb = shape.batch, shape.seqlen
    cond = spec.get("cond")
    hyb = spec.get("hybrid")
    w = device_stack_weights(torch, shape, layers, vocab, cond=cond, hybrid=hyb)
    csw, keep = dm.make_stack_weights(w)
    stream = torch.cuda.current_stream().cuda_stream
    stream_box = [stream]                      # the stream the library is given (the capture stream while a graph is recorded)
    if cond:
        blk = dm.dm_block_cfg(cond["d_ff"], cond["d_cond"], 1e-5)
        cbw = dm.make_block_weights(w["blocks"])
        tau = torch.from_numpy(I.make_timestep_embedding(B, cond["d_cond"], seed=0)).cuda()

    smp = spec.get("sample")
    if smp:
        masked_per_row = Lb // 2
        scfg_s = dm.dm_sample_cfg(50257, 50258, 1.0 - smp["p"] / masked_per_row)
        gen = torch.Generator(device="cuda").manual_seed(1)
        u_keep = torch.rand(B, Lb, generator=gen, device="cuda")
        u_cat = torch.rand(B, Lb, generator=gen, device="cuda")

    if hyb:
        hcfg = dm.dm_hybrid_cfg(hyb["period"], hyb["heads"])
        caw = dm.make_attn_weights(w["attn"])

    def ws_bytes(cfg):
        if hyb:
            return dm.dm_denoise_hybrid_workspace_bytes(cfg, blk if cond else None)
        if smp:
            return dm.dm_denoise_sample_workspace_bytes(cfg, blk if cond else None)
        return dm.dm_denoise_cond_workspace_bytes(cfg, blk) if cond else dm.dm_denoise_workspace_bytes(cfg)

    def denoise(cfg, tok_ptr, amax_ptr, st):
        if hyb:
            dm.dm_denoise_step_hybrid(cfg, blk if cond else None, hcfg, csw, cbw if cond else None, caw, tok_ptr, tau.data_ptr() if cond else 0,
                                      0, amax_ptr, ws.data_ptr(), ws.numel(), stream_box[0])
        elif smp:
            dm.dm_denoise_sample_step(cfg, blk if cond else None, csw, cbw if cond else None, tok_ptr, tau.data_ptr() if cond else 0, scfg_s,
                                      u_keep.data_ptr(), u_cat.data_ptr(), amax_ptr, st, ws.data_ptr(), ws.numel(), stream_box[0])
        elif cond:
            dm.dm_denoise_step_cond(cfg, blk, csw, cbw, tok_ptr, tau.data_ptr(), 0, amax_ptr, st, ws.data_ptr(), ws.numel(), stream_box[0])
        else:
            dm.dm_denoise_step(cfg, csw, tok_ptr, 0, amax_ptr, st, ws.data_ptr(), ws.numel(), stream_box[0])

    def stack_cfg(L):
        sh = I.MixerShape(B, L, shape.d_model, shape.expand, shape.d_state, shape.d_conv, shape.n_heads)
        return dm.dm_stack_cfg(G.cfg_of(sh, I.BF16), layers, vocab, 1e-5)

    def tokens(L, n):
        if smp:                                   # mid-generation: every other position is [MASK]
            out = []
            for i in range(n):
                t = I.make_tokens(B, L, 50257, 50257, seed=i)
                t[:, (i % 2)::2] = 50257
                t[:, (1 - i % 2)::2] = np.where(t[:, (1 - i % 2)::2] == 50257, 11, t[:, (1 - i % 2)::2])
                out.append(torch.from_numpy(t).cuda())
            return out
        return [torch.from_numpy(I.make_tokens(B, L, 50257, 50257, seed=i)).cuda() for i in range(n)]

    scfg = stack_cfg(Lb)
    nb = ws_bytes(scfg)
    states = None
    extra = {}
    if prefix:
        # commit the prefix once (block step over the prefix, NULL state in), then time steps over the active block
        pcfg = stack_cfg(prefix)
        nbp = ws_bytes(pcfg)
        ws = G.workspace(max(nb, nbp, ws_bytes(stack_cfg(prefix + Lb))))
        st_bufs = [(torch.empty((B, shape.n_heads, shape.headdim, shape.d_state), device="cuda"),
                    torch.empty((B, shape.d_conv - 1, shape.conv_ch), device="cuda", dtype=torch.bfloat16)) for _ in range(layers)]
        pst = (dm.dm_layer_state * layers)()
        for i, (sb, cb) in enumerate(st_bufs):
            pst[i] = dm.dm_layer_state(None, None, sb.data_ptr(), cb.data_ptr())
        ptok = tokens(prefix, 1)[0]
        amax_p = torch.empty((B, prefix), device="cuda", dtype=torch.int32)
        denoise(pcfg, ptok.data_ptr(), amax_p.data_ptr(), pst)
        dm.dm_check(stream)
        states = (dm.dm_layer_state * layers)()
        for i, (sb, cb) in enumerate(st_bufs):
            states[i] = dm.dm_layer_state(sb.data_ptr(), cb.data_ptr(), None, None)
    else:
        ws = G.workspace(nb)
    toks = tokens(Lb, 4)
    amax = torch.empty((B, Lb), device="cuda", dtype=torch.int32)
    loop, gen = spec.get("loop"), spec.get("generate")
    passes_per_step = 1                                   # denoiser evaluations in one step

    def step(i):
        denoise(scfg, toks[i % 4].data_ptr(), amax.data_ptr(), states)

    if loop:
        # second set of state buffers; block i reads set i % 2 in its denoising passes and commits into the other one
        st_bufs2 = [(torch.empty_like(sb), torch.empty_like(cb)) for sb, cb in st_bufs]
        sets = (st_bufs, st_bufs2)
        read_st, commit_st = [], []
        for par in range(2):
            rd, cm = (dm.dm_layer_state * layers)(), (dm.dm_layer_state * layers)()
            for i in range(layers):
                (si, ci), (so, co) = sets[par][i], sets[1 - par][i]
                rd[i] = dm.dm_layer_state(si.data_ptr(), ci.data_ptr(), None, None)
                cm[i] = dm.dm_layer_state(si.data_ptr(), ci.data_ptr(), so.data_ptr(), co.data_ptr())
            read_st.append(rd); commit_st.append(cm)
        passes_per_step = loop["passes"] + 1

        def step(i):                                      # one block: its denoising passes, then the commit pass over its final tokens
            for p in range(loop["passes"]):
                denoise(scfg, toks[(i + p) % 4].data_ptr(), amax.data_ptr(), read_st[i % 2])
            denoise(scfg, toks[(i + 3) % 4].data_ptr(), amax.data_ptr(), commit_st[i % 2])
    if gen:
        K = Lb // gen["p"]
        gcfg = dm.dm_generate_cfg(K, 1e-3, 50257, 50258)
        g2 = torch.Generator(device="cuda").manual_seed(2)
        gu_keep = torch.rand(K + 1, B, Lb, generator=g2, device="cuda")
        gu_cat = torch.rand(K + 1, B, Lb, generator=g2, device="cuda")
        gtau = torch.from_numpy(np.stack([I.make_timestep_embedding(B, cond["d_cond"], seed=k) for k in range(K + 1)])).cuda() if cond else None
        gstart = torch.full((B, Lb), 50257, device="cuda", dtype=torch.int32)
        nbg = dm.dm_generate_workspace_bytes(scfg, blk if cond else None)
        ws = G.workspace(max(nb, nbg))
        passes_per_step = K + 1

        def step(i):                                      # one generation from an all-mask start: K reverse steps + the clean-up pass
            dm.dm_generate(scfg, blk if cond else None, csw, cbw if cond else None, gcfg, gstart.data_ptr(), gtau.data_ptr() if cond else 0,
                           gu_keep.data_ptr(), gu_cat.data_ptr(), amax.data_ptr(), 0, ws.data_ptr(), ws.numel(), stream_box[0])

    def timed(fn, n):
        for i in range(args.warmup):
            fn(i)
        dm.dm_check(stream)
        D.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        timed.launches0 = dm.dm_kernel_launch_count()
        e0.record()
        for i in range(n):
            fn(i)
        e1.record()
        timed.launches = dm.dm_kernel_launch_count() - timed.launches0      # kernels enqueued inside the timed region
        D.barrier()
        torch.cuda.synchronize()
        return D.max_over_ranks(e0.elapsed_time(e1), "cuda")

    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_total = timed(step, args.steps)
    launches = timed.launches
    # per-stage times: the same steps once more with the library's stage events switched on (a step of a stack records some 150 of them, which
    # costs a short-kernel workload a third of its time: they stay out of the region `value` is taken from)
    dm.dm_profile_enable(True)
    dm.dm_profile_read()
    ms_staged = timed(step, args.steps) / args.steps
    stage_ms, stage_n = dm.dm_profile_read()          # includes the warm-up steps
    dm.dm_profile_enable(False)
    clocks = sampler.stop() if sampler else None
    dm.dm_check(stream)
    T = B * Lb
    ms_step = ms_total / args.steps
    if args.graph:
        # the same step recorded once per token buffer into a CUDA graph and replayed: no launch work on the host
        graphs, cap = [], torch.cuda.Stream()
        for i in range(4):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap):
                stream_box[0] = torch.cuda.current_stream().cuda_stream
                step(i)
            stream_box[0] = stream
            graphs.append(g)
        if loop:                                          # same starting state for the eager block and the replayed one
            saved = [(sb.clone(), cb.clone()) for sb, cb in st_bufs]
        step(0)
        torch.cuda.synchronize()
        eager = amax.clone()
        amax.fill_(-1)
        if loop:
            for (sb, cb), (s0, c0) in zip(st_bufs, saved):
                sb.copy_(s0); cb.copy_(c0)
        graphs[0].replay()
        torch.cuda.synchronize()
        if not torch.equal(eager, amax):
            raise RuntimeError("the step replayed from the CUDA graph does not reproduce the eager step's token ids")
        ms_graph = timed(lambda i: graphs[i % 4].replay(), args.steps) / args.steps
        dm.dm_check(stream)
        extra = dict(extra, cuda_graph_ms_per_step=ms_graph)
    if prefix:
        # the alternative without a cache: re-encode prefix + block
        fcfg = stack_cfg(prefix + Lb)
        ftok = tokens(prefix + Lb, 2)
        famax = torch.empty((B, prefix + Lb), device="cuda", dtype=torch.int32)
        ms_full = timed(lambda i: denoise(fcfg, ftok[i % 2].data_ptr(), famax.data_ptr(), None), max(2, args.steps // 4)) / max(2, args.steps // 4)
        extra = dict(extra, prefix=prefix, full_reencode_ms_per_pass=ms_full, state_carry_speedup=ms_full / (ms_step / passes_per_step))
    # end to end: token ids from pinned host memory in, arg-max ids back, inside the timed region
    e2e = None
    if not args.no_e2e:
        th = torch.from_numpy(I.make_tokens(B, Lb, 50257, 50257, seed=9)).pin_memory()
        ah = torch.empty((B, Lb), dtype=torch.int32).pin_memory()
        td = torch.empty((B, Lb), device="cuda", dtype=torch.int32)

        def host_step(i):
            td.copy_(th, non_blocking=True)
            if loop or gen:                               # the block's / the generation's start tokens in, its final ids out
                (gstart if gen else toks[i % 4]).copy_(td, non_blocking=True)
                step(i)
            else:
                denoise(scfg, td.data_ptr(), amax.data_ptr(), states)
            ah.copy_(amax, non_blocking=True)
            torch.cuda.synchronize()
        for i in range(2):
            host_step(i)
        t0 = time.perf_counter()
        for i in range(args.steps):
            host_step(i)
        sec = time.perf_counter() - t0
        e2e = {"value": world * T * passes_per_step * layers * args.steps / sec, "unit": UNIT, "h2d_bytes_per_step": T * 4, "d2h_bytes_per_step": T * 4}
    if rank != 0:
        D.shutdown()
        return
    peaks = load_peaks()
    n_calls = max(stage_n[dm.DM_STAGE_SCAN], 1)       # mixer calls profiled (warm-up included)
    inp = stage_ms[dm.DM_STAGE_IN_PROJ] / n_calls
    scn = stage_ms[dm.DM_STAGE_SCAN] / n_calls
    outp = stage_ms[dm.DM_STAGE_OUT_PROJ] / n_calls
    n_mamba = layers - ((layers + hyb["period"] - 1) // hyb["period"] if hyb else 0)      # the other layers are attention
    f_in, f_out = gemm_flops_per_token(shape)
    in_tf, out_tf = f_in * T / (inp * 1e-3) / 1e12, f_out * T / (outp * 1e-3) / 1e12
    scan_bytes = scan_bytes_per_token(shape, 2) * T
    if prefix:
        scan_bytes += B * shape.n_heads * shape.headdim * shape.d_state * 4        # one read of the carried state
    scan_gbs = scan_bytes / (scn * 1e-3) / 1e9
    kernels = {"in_proj_per_layer": {"ms": inp, "tflops": in_tf}, "scan_per_layer": {"ms": scn, "gbs": scan_gbs},
               "out_proj_per_layer": {"ms": outp, "tflops": out_tf},
               "rest_of_step_ms": ms_step - passes_per_step * n_mamba * (inp + scn + outp)}
    burst = ms_total < 1000.0
    tpk = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    tsrc = peaks["source"] + (" (burst bf16: timed region under 1 s)" if burst else " (sustained bf16: timed region over 1 s)")
    scan_entry = {"kernel": "fused conv+scan+gate (per layer)", "bound": "hbm", "achieved": scan_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                  "frac": scan_gbs / peaks["hbm_gbs"], "frac_of_8tbs": scan_gbs / 8000.0, "ms": scn, "algorithmic_bytes": scan_bytes,
                  "traffic": None, "peak_source": peaks["source"] + " (copy bandwidth)"}
    if scn >= max(inp, outp):
        roofline = dict(scan_entry)
    else:
        tf = in_tf if inp >= outp else out_tf
        roofline = {"kernel": ("in_proj" if inp >= outp else "out_proj") + " GEMM (per layer)", "bound": "tensor", "achieved": tf,
                    "peak": tpk, "unit": "TFLOP/s", "frac": tf / tpk, "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                    "traffic": None, "peak_source": tsrc}
    roofline["scan"] = scan_entry
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline and not hyb:
        n_tok = min(Lb, 128)
        sec, nl = oracle_stack_sample_seconds(spec, n_tok)
        cpu_baseline = {"value": n_tok * nl / sec, "unit": UNIT, "cores": host_cores(), "threads_used": blas_threads(), "kind": "oracle",
                        "sample": f"batch row 0, first {n_tok} tokens, first {nl} layers + output head of {args.workload} (full widths), {sec:.1f} s; "
                                  "the metric is per layer"}
    npass = passes_per_step
    line = {"metric": METRIC, "value": world * T * npass * layers / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": dict({"workload": args.workload, "batch": B, "seq_len": Lb, "d_model": shape.d_model, "d_state": shape.d_state,
                            "heads": shape.n_heads, "layers": layers, "vocab": vocab, "block": "AdaLN + mixer + MLP (d_ff %d, d_cond %d)" % (cond["d_ff"], cond["d_cond"]) if cond else "RMSNorm pre-norm + mixer", "tokens_per_s_whole_stack": world * T * npass / (ms_step * 1e-3),
                            "ms_per_step_with_stage_events": ms_staged,
                            "parallelism": "replicas only" if world > 1 else "1 GPU",
                            "l2": "weights of 24 layers and the vocabulary projection exceed the 126 MB L2; token ids rotate over 4 buffers"},
                           **({"hybrid": "attention mixer (%d heads of %d) in every %dth layer, %d Mamba layers; the attention layers are inside rest_of_step_ms"
                                         % (hyb["heads"], shape.d_model // hyb["heads"], hyb["period"], n_mamba)} if hyb else {}),
                           **({"sample": "half of the positions masked, p = %d drawn per sequence and step" % smp["p"],
                               "generated_tokens_per_s_at_K_eq_L_over_p": world * T / ((Lb // smp["p"]) * ms_step * 1e-3)} if smp else {}),
                           **({"loop": "step = one block of %d tokens per sequence: %d denoising passes reading the carried state + 1 commit pass; "
                                       "%d blocks after a %d-token prefix" % (Lb, loop["passes"], loop["blocks"], prefix),
                               "generated_tokens_per_s": world * T / (ms_step * 1e-3), "ms_per_pass": ms_step / npass} if loop else {}),
                           **({"generate": "step = one generation of %d tokens per sequence from an all-mask start: K = L / %d = %d reverse steps "
                                           "(Eq. 3) + the clean-up pass, one dm_generate call" % (Lb, gen["p"], Lb // gen["p"]),
                               "generated_tokens_per_s": world * T / (ms_step * 1e-3), "ms_per_pass": ms_step / npass} if gen else {}),
                           **extra),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "kernels": kernels, "cpu_baseline": cpu_baseline}
    print(json.dumps(line), flush=True)
    D.shutdown()


def fit_latency(lengths, ms):
    """Non-negative least-squares fit of the per-step latency t(L) = a L^2 + b L + c (Sec. 4.3, latency decomposition: the
    quadratic term is what attention adds; a linear-time mixer should give a ~ 0).  L is scaled to units of 1024 tokens so
    that the three columns have comparable size.  Returns a, b, c in ms per (1024 tokens)^2, ms per 1024 tokens, ms."""
    from scipy.optimize import nnls
    x = np.asarray(lengths, np.float64) / 1024.0
    A = np.stack([x * x, x, np.ones_like(x)], axis=1)
    coef, resid = nnls(A, np.asarray(ms, np.float64))
    return [float(v) for v in coef], float(resid)


def run_lsweep(args, rank, local_rank, world):
    """cfg 3's sweep over L at batch 1 (the paper's throughput axis, Sec. 4.3, up to its longest context 65 536) with the
    fit of fit_latency() over the whole mixer step and over the fused scan alone."""
    import torch
    from paper_2511_15927_b200 import build
    if rank == 0 or world == 1:
        build.build()
    from paper_2511_15927_b200 import dist_util as D
    D.init("nccl", local_rank)
    from paper_2511_15927_b200 import binding as dm
    torch.cuda.set_device(local_rank)
    from paper_2511_15927_b200 import torch_io as G
    lengths = [2048, 4096, 8192, 16384, 32768, 65536]
    base, dtype = I.CONFIGS["cfg3_8k"]
    wf, wr = I.make_mixer_weights(base, 0, dtype)
    cw = (dm.make_dir_weights(G.dev_dir_weights(wf, dtype)), dm.make_dir_weights(G.dev_dir_weights(wr, dtype)))
    keep = cw
    stream = torch.cuda.current_stream().cuda_stream
    sampler = ClockSampler(local_rank) if rank == 0 else None
    rows, launches = [], 0
    for L in lengths:
        shape = I.MixerShape(1, L, base.d_model, base.expand, base.d_state, base.d_conv, base.n_heads)
        cfg = G.cfg_of(shape, dtype)
        g = torch.Generator(device="cuda").manual_seed(L)
        xs = [torch.randn(1, L, shape.d_model, generator=g, device="cuda").to(torch.bfloat16) for _ in range(4)]
        y = torch.empty_like(xs[0])
        nb = dm.dm_bimamba_workspace_bytes(cfg)
        ws = G.workspace(nb)
        for i in range(args.warmup):
            dm.dm_bimamba_forward(cfg, cw, xs[i % 4].data_ptr(), y.data_ptr(), ws.data_ptr(), nb, stream)
        dm.dm_check(stream)
        D.barrier(); torch.cuda.synchronize()
        dm.dm_profile_enable(True); dm.dm_profile_read()
        l0 = dm.dm_kernel_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.steps):
            dm.dm_bimamba_forward(cfg, cw, xs[i % 4].data_ptr(), y.data_ptr(), ws.data_ptr(), nb, stream)
        e1.record()
        D.barrier(); torch.cuda.synchronize()
        launches += dm.dm_kernel_launch_count() - l0
        stage_ms, stage_n = dm.dm_profile_read()
        dm.dm_profile_enable(False)
        dm.dm_check(stream)
        ms = D.max_over_ranks(e0.elapsed_time(e1), "cuda") / args.steps
        rows.append({"L": L, "ms_per_step": ms, "scan_ms": stage_ms[dm.DM_STAGE_SCAN] / max(stage_n[dm.DM_STAGE_SCAN], 1),
                     "tokens_per_s": world * L / (ms * 1e-3)})
        del xs, y, ws
    clocks = sampler.stop() if sampler else None
    if rank != 0:
        D.shutdown()
        return
    (a, b, c), resid = fit_latency([r["L"] for r in rows], [r["ms_per_step"] for r in rows])
    (sa, sb, sc), sresid = fit_latency([r["L"] for r in rows], [r["scan_ms"] for r in rows])
    last = rows[-1]
    peaks = load_peaks()
    es = 2
    shape = I.MixerShape(1, last["L"], base.d_model, base.expand, base.d_state, base.d_conv, base.n_heads)
    scan_bytes = scan_bytes_per_token(shape, es) * last["L"]
    scan_gbs = scan_bytes / (last["scan_ms"] * 1e-3) / 1e9
    line = {"metric": METRIC, "value": last["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": last["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": "lsweep_fit", "batch": 1, "seq_len": last["L"], "d_model": base.d_model, "d_state": base.d_state,
                       "heads": base.n_heads, "sweep": rows,
                       "latency_fit": {"model": "t(L) = a (L/1024)^2 + b (L/1024) + c, non-negative least squares, ms",
                                       "mixer_step": {"a": a, "b": b, "c": c, "residual_ms": resid,
                                                      "quadratic_share_at_65536": a * 64 * 64 / max(a * 64 * 64 + b * 64 + c, 1e-30)},
                                       "fused_scan": {"a": sa, "b": sb, "c": sc, "residual_ms": sresid}},
                       "l2": "inputs rotate over 4 buffers; every length's working set exceeds the 126 MB L2 from L = 4096 up",
                       "parallelism": "replicas only" if world > 1 else "1 GPU"},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
            "roofline": {"kernel": "fused conv+scan+gate at the longest length", "bound": "hbm", "achieved": scan_gbs, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": scan_gbs / peaks["hbm_gbs"], "frac_of_8tbs": scan_gbs / 8000.0, "ms": last["scan_ms"],
                         "algorithmic_bytes": scan_bytes, "traffic": ncu_traffic("scan", shape, I.BF16, last["L"]),
                         "peak_source": peaks["source"] + " (copy bandwidth)"},
            "cpu_baseline": None}
    print(json.dumps(line), flush=True)
    D.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 10; 64 blocks for cfg4_loop; 3 generations for the *_generate workloads)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg1", choices=sorted(I.CONFIGS) + sorted(STACKS) + ["lsweep_fit", "cfg1_tied", "cfg3_8k_tied"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=128, help="tokens per step of the reference arm's sample")
    ap.add_argument("--cpu-baseline-tokens", type=int, default=2048)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph", action="store_true", help="stack workloads: also time the step replayed from a captured CUDA graph")
    args = ap.parse_args()
    if args.steps is None:
        spec = STACKS.get(args.workload, {})
        args.steps = spec["loop"]["blocks"] if spec.get("loop") else 3 if spec.get("generate") else 10
    if args.warmup < 3:
        args.warmup = max(args.warmup, 1) if args.impl == "reference" else 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.workload == "lsweep_fit":
        if args.impl == "reference":
            if rank == 0:
                print(json.dumps({"impl": "reference", "unavailable": "the sweep is a post-processing workload of cfg3; run the reference arm on cfg3_8k"}), flush=True)
            return
        run_lsweep(args, rank, local_rank, world)
        return
    if args.workload in STACKS:
        if args.impl == "reference":
            if rank == 0:
                run_reference_stack(args)
            return
        run_stack(args, rank, local_rank, world)
        return
    # *_tied: the same shape with the directions sharing in_proj and out_proj (App. A.1 "bidirectional weight tie")
    tied = args.workload.endswith("_tied")
    shape, dtype = I.CONFIGS[args.workload[:-5] if tied else args.workload]

    if args.impl == "reference":
        run_reference(args, shape, dtype, rank)
        return

    import torch
    from paper_2511_15927_b200 import build
    if rank == 0 or world == 1:
        build.build()
    from paper_2511_15927_b200 import dist_util as D
    D.init("nccl", local_rank)
    from paper_2511_15927_b200 import binding as dm
    torch.cuda.set_device(local_rank)
    from paper_2511_15927_b200 import torch_io as G

    es = 2 if dtype == I.BF16 else 4
    T = shape.batch * shape.seqlen
    cfg = G.cfg_of(shape, dtype, flags=dm.DM_FLAGS_DEFAULT | (dm.DM_FLAG_TIED_PROJ if tied else 0))
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
        D.barrier()
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
    ms_total = D.max_over_ranks(ms_total, "cuda")
    ms_step = ms_total / args.steps
    value = D.whole_job_value(T, args.steps, ms_total)

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
        sec = D.max_over_ranks(sec, "cuda")
        e2e = {"value": D.whole_job_value(T, args.steps, sec * 1e3), "unit": UNIT, "h2d_bytes_per_step": T * shape.d_model * es,
               "d2h_bytes_per_step": T * shape.d_model * es}

    if rank != 0:
        D.shutdown()
        return

    peaks = load_peaks()
    scan_ms = stage_ms[dm.DM_STAGE_SCAN] / max(stage_n[dm.DM_STAGE_SCAN], 1)
    inp_ms = stage_ms[dm.DM_STAGE_IN_PROJ] / args.steps
    outp_ms = stage_ms[dm.DM_STAGE_OUT_PROJ] / args.steps
    scan_bytes = scan_bytes_per_token(shape, es) * T
    f_in, f_out = gemm_flops_per_token(shape)
    if tied:                                               # one shared in_proj and one out_proj over the summed directions
        f_in, f_out = f_in // 2, f_out // 2
    scan_gbs = scan_bytes / (scan_ms * 1e-3) / 1e9
    in_tf = f_in * T / (inp_ms * 1e-3) / 1e12
    out_tf = f_out * T / (outp_ms * 1e-3) / 1e12
    def tfrac(tf):
        return {"frac_of_%s_burst_tensor_peak" % peaks["source"]: tf / peaks["bf16_tflops"] if dtype == I.BF16 else None,
                "frac_of_%s_sustained_tensor_peak" % peaks["source"]: tf / peaks["bf16_tflops_sustained"] if dtype == I.BF16 else None}
    kernels = {
        "in_proj": dict({"ms": inp_ms, "tflops": in_tf}, **tfrac(in_tf)),
        "scan": {"ms": scan_ms, "gbs": scan_gbs, "frac_of_%s_hbm_peak" % peaks["source"]: scan_gbs / peaks["hbm_gbs"],
                 "frac_of_nominal_8tbs": scan_gbs / 8000.0, "algorithmic_bytes": scan_bytes},
        "out_proj": dict({"ms": outp_ms, "tflops": out_tf}, **tfrac(out_tf)),
    }
    # Tensor peak for the GEMMs: the timed region is tens of milliseconds at full clocks, i.e. the burst figure's regime;
    # the sustained figure (a seconds-long loop under the power cap) is printed beside it.
    burst = ms_total < 1000.0
    tpk = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    tsrc = peaks["source"] + (" (burst bf16: timed region under 1 s)" if burst else " (sustained bf16)")
    scan_entry = {"kernel": "fused conv+scan+gate", "bound": "hbm", "achieved": scan_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                  "frac": scan_gbs / peaks["hbm_gbs"], "frac_of_8tbs": scan_gbs / 8000.0, "ms": scan_ms, "algorithmic_bytes": scan_bytes,
                  "traffic": ncu_traffic("scan", shape, dtype, T), "peak_source": peaks["source"] + " (copy bandwidth)"}

    def gemm_entry(name, tf, ms):
        return {"kernel": name + " GEMM (one launch per direction)", "bound": "tensor", "achieved": tf, "peak": tpk, "unit": "TFLOP/s",
                "frac": tf / tpk, "frac_of_sustained": tf / peaks["bf16_tflops_sustained"], "ms": ms,
                "traffic": ncu_traffic(name, shape, dtype, T), "peak_source": tsrc}
    dominant = max(("in_proj", inp_ms), ("scan", scan_ms), ("out_proj", outp_ms), key=lambda kv: kv[1])[0]
    if dominant == "scan" or dtype != I.BF16:
        roofline = dict(scan_entry)
    else:
        roofline = gemm_entry(dominant, in_tf if dominant == "in_proj" else out_tf, inp_ms if dominant == "in_proj" else outp_ms)
    # the dominant kernel above; the kernel the metric names (the fused scan) and the other GEMM always ride along
    roofline["scan"] = scan_entry
    if dtype == I.BF16:
        roofline["in_proj"] = gemm_entry("in_proj", in_tf, inp_ms)
        roofline["out_proj"] = gemm_entry("out_proj", out_tf, outp_ms)

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        n_tok = min(shape.seqlen, args.cpu_baseline_tokens)
        sec = oracle_sample_seconds(shape, dtype, n_tok)
        cpu_baseline = {"value": n_tok / sec, "unit": UNIT, "cores": host_cores(), "threads_used": blas_threads(), "kind": "oracle",
                        "sample": f"batch row 0, first {n_tok} tokens of {args.workload} (full widths, both directions), {sec:.1f} s; "
                                  "the token loop of the oracle is one Python thread, its matrix products use the BLAS threads"}

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
    D.shutdown()


if __name__ == "__main__":
    main()
