"""Helpers for the GPU parity tests: move the seeded host inputs to the device, call the library through
its C ABI (via the ctypes binding) and bring results back as float64 numpy arrays."""
from __future__ import annotations

import numpy as np
import torch

from paper_2511_15927_b200 import binding as dm
from paper_2511_15927_b200 import inputs as I
from paper_2511_15927_b200.torch_io import (cfg_of, dev, dev_block_weights, dev_dir_weights, dev_stack_weights, dm_dtype,  # noqa: F401
                                            tdtype, workspace)


def run_forward(shape, dtype, wf, wr, x, flags=dm.DM_FLAGS_DEFAULT, dir_mask=dm.DM_DIR_BOTH, chunk=0):
    cfg = cfg_of(shape, dtype, flags, dir_mask, chunk)
    dwf, dwr = dev_dir_weights(wf, dtype), dev_dir_weights(wr, dtype)
    xd = dev(x, dtype)
    yd = torch.empty_like(xd)
    nb = dm.dm_bimamba_workspace_bytes(cfg)
    ws = workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_bimamba_forward(cfg, (dm.make_dir_weights(dwf), dm.make_dir_weights(dwr)), xd.data_ptr(), yd.data_ptr(),
                          ws.data_ptr(), nb, st)
    dm.dm_check(st)
    return yd.float().cpu().numpy().astype(np.float64)


def run_forward_host(shape, dtype, wf, wr, x, pinned=True):
    """dm_bimamba_forward_host: x and y live in host memory, the library stages them through its workspace."""
    cfg = cfg_of(shape, dtype)
    dwf, dwr = dev_dir_weights(wf, dtype), dev_dir_weights(wr, dtype)
    xh = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(tdtype(dtype))
    yh = torch.empty_like(xh)
    if pinned:
        xh, yh = xh.pin_memory(), yh.pin_memory()
    act = (xh.numel() * xh.element_size() + 255) // 256 * 256
    nb = dm.dm_bimamba_workspace_bytes(cfg) + 2 * act
    ws = workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_bimamba_forward_host(cfg, (dm.make_dir_weights(dwf), dm.make_dir_weights(dwr)), xh.data_ptr(), yh.data_ptr(),
                               ws.data_ptr(), nb, st)
    dm.dm_check(st)
    return yh.float().numpy().astype(np.float64)


def run_block_step(shape, dtype, wf, wr, x_blk, ssm_in=None, conv_in=None, want_state=True, flags=dm.DM_FLAGS_DEFAULT,
                   dir_mask=dm.DM_DIR_BOTH, chunk=0):
    cfg = cfg_of(shape, dtype, flags, dir_mask, chunk)
    dwf, dwr = dev_dir_weights(wf, dtype), dev_dir_weights(wr, dtype)
    xd = dev(x_blk, dtype)
    yd = torch.empty_like(xd)
    s_in = dev(ssm_in.astype(np.float32)) if ssm_in is not None else None
    c_in = dev(conv_in.astype(np.float32), dtype) if conv_in is not None else None
    s_out = torch.full((shape.batch, shape.n_heads, shape.headdim, shape.d_state), float("nan"), device="cuda") if want_state else None
    c_out = torch.full((shape.batch, shape.d_conv - 1, shape.conv_ch), float("nan"), device="cuda", dtype=tdtype(dtype)) if want_state else None
    nb = dm.dm_bimamba_workspace_bytes(cfg)
    ws = workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    p = lambda t: t.data_ptr() if t is not None else 0
    dm.dm_bimamba_block_step(cfg, (dm.make_dir_weights(dwf), dm.make_dir_weights(dwr)), xd.data_ptr(), p(s_in), p(c_in),
                             p(s_out), p(c_out), yd.data_ptr(), ws.data_ptr(), nb, st)
    dm.dm_check(st)
    f = lambda t: None if t is None else t.float().cpu().numpy().astype(np.float64)
    return f(yd), f(s_out), f(c_out)


def run_denoise(shape, dtype, sw, tokens, vocab, want_logits=True, want_argmax=True, states_in=None, want_states=False,
                flags=dm.DM_FLAGS_DEFAULT, dir_mask=dm.DM_DIR_BOTH, rms_eps=1e-5, tau=None, d_ff=0, ln_eps=1e-5):
    """tau given: the timestep-conditioned stack (dm_denoise_step_cond), whose block weights are in sw's layers."""
    n_layers = len(sw["layers"])
    scfg = dm.dm_stack_cfg(cfg_of(shape, dtype, flags, dir_mask), n_layers, vocab, rms_eps)
    dsw = dev_stack_weights(sw, dtype)
    csw, keep = dm.make_stack_weights(dsw)
    tok = dev(tokens.astype(np.int32))
    T = shape.batch * shape.seqlen
    logits = torch.empty((shape.batch, shape.seqlen, vocab), device="cuda", dtype=tdtype(dtype)) if want_logits else None
    amax = torch.full((shape.batch, shape.seqlen), -1, device="cuda", dtype=torch.int32) if want_argmax else None
    states = None
    bufs = []
    if states_in is not None or want_states:
        states = (dm.dm_layer_state * n_layers)()
        for i in range(n_layers):
            s_in = c_in = None
            if states_in is not None and states_in[i] is not None:
                s_in = dev(states_in[i][0].astype(np.float32)); c_in = dev(states_in[i][1].astype(np.float32), dtype)
            s_out = torch.empty((shape.batch, shape.n_heads, shape.headdim, shape.d_state), device="cuda") if want_states else None
            c_out = torch.empty((shape.batch, shape.d_conv - 1, shape.conv_ch), device="cuda", dtype=tdtype(dtype)) if want_states else None
            bufs.append((s_in, c_in, s_out, c_out))
            p = lambda t: t.data_ptr() if t is not None else None
            states[i] = dm.dm_layer_state(p(s_in), p(c_in), p(s_out), p(c_out))
    st = torch.cuda.current_stream().cuda_stream
    if tau is None:
        nb = dm.dm_denoise_workspace_bytes(scfg)
        ws = workspace(nb)
        dm.dm_denoise_step(scfg, csw, tok.data_ptr(), logits.data_ptr() if want_logits else 0,
                           amax.data_ptr() if want_argmax else 0, states, ws.data_ptr(), nb, st)
    else:
        blk = dm.dm_block_cfg(d_ff, tau.shape[1], ln_eps)
        dbw = dev_block_weights(sw, dtype)
        cbw = dm.make_block_weights(dbw)
        taud = dev(np.asarray(tau, np.float32))
        nb = dm.dm_denoise_cond_workspace_bytes(scfg, blk)
        ws = workspace(nb)
        dm.dm_denoise_step_cond(scfg, blk, csw, cbw, tok.data_ptr(), taud.data_ptr(), logits.data_ptr() if want_logits else 0,
                                amax.data_ptr() if want_argmax else 0, states, ws.data_ptr(), nb, st)
    dm.dm_check(st)
    f = lambda t: None if t is None else t.float().cpu().numpy().astype(np.float64)
    out_states = [(f(b[2]), f(b[3])) for b in bufs] if want_states else None
    return f(logits), (amax.cpu().numpy() if want_argmax else None), out_states


def rel_l2(a, b):
    return float(np.linalg.norm(np.asarray(a, np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - b)))


def oracle_kwargs(shape, flags=dm.DM_FLAGS_DEFAULT, eps=1e-5):
    return dict(expand=shape.expand, d_state=shape.d_state, n_heads=shape.n_heads, n_groups=shape.n_groups,
                gated_norm=bool(flags & dm.DM_FLAG_GATED_RMSNORM), conv_bias=bool(flags & dm.DM_FLAG_CONV_BIAS),
                d_skip=bool(flags & dm.DM_FLAG_D_SKIP), norm_eps=eps)


def run_sample_step(shape, dtype, sw, tokens, vocab, u_keep, u_cat, keep_prob, mask_id, vocab_real, tau=None, d_ff=0,
                    rms_eps=1e-5, ln_eps=1e-5):
    """dm_denoise_sample_step on host arrays; returns tokens_out [B, L] int32."""
    n_layers = len(sw["layers"])
    scfg = dm.dm_stack_cfg(cfg_of(shape, dtype), n_layers, vocab, rms_eps)
    dsw = dev_stack_weights(sw, dtype)
    csw, keep = dm.make_stack_weights(dsw)
    blk = cbw = taud = None
    if tau is not None:
        blk = dm.dm_block_cfg(d_ff, tau.shape[1], ln_eps)
        dbw = dev_block_weights(sw, dtype)
        cbw = dm.make_block_weights(dbw)
        taud = dev(np.asarray(tau, np.float32))
    tok = dev(np.asarray(tokens, np.int32))
    out = torch.full_like(tok, -7)
    uk, uc = dev(np.asarray(u_keep, np.float32)), dev(np.asarray(u_cat, np.float32))
    nb = dm.dm_denoise_sample_workspace_bytes(scfg, blk)
    ws = workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_denoise_sample_step(scfg, blk, csw, cbw, tok.data_ptr(), taud.data_ptr() if taud is not None else 0,
                              dm.dm_sample_cfg(mask_id, vocab_real, keep_prob), uk.data_ptr(), uc.data_ptr(), out.data_ptr(), None,
                              ws.data_ptr(), nb, st)
    dm.dm_check(st)
    return out.cpu().numpy()


def run_denoise_hybrid(shape, dtype, sw, tokens, vocab, attn_period, attn_heads, tau=None, d_ff=0, rms_eps=1e-5, ln_eps=1e-5):
    """dm_denoise_step_hybrid on host arrays; layers of sw that are attention carry "w_qkv" and "w_o".  Returns logits."""
    n_layers = len(sw["layers"])
    scfg = dm.dm_stack_cfg(cfg_of(shape, dtype), n_layers, vocab, rms_eps)
    dsw = dev_stack_weights(sw, dtype)
    csw, keep = dm.make_stack_weights(dsw)
    blk = cbw = taud = None
    if tau is not None:
        blk = dm.dm_block_cfg(d_ff, tau.shape[1], ln_eps)
        dbw = dev_block_weights(sw, dtype)
        cbw = dm.make_block_weights(dbw)
        taud = dev(np.asarray(tau, np.float32))
    daw = [({"w_qkv": dev(l["w_qkv"], dtype), "w_o": dev(l["w_o"], dtype)} if "w_qkv" in l else None) for l in sw["layers"]]
    caw = dm.make_attn_weights(daw)
    tok = dev(np.asarray(tokens, np.int32))
    logits = torch.empty((shape.batch, shape.seqlen, vocab), device="cuda", dtype=tdtype(dtype))
    nb = dm.dm_denoise_hybrid_workspace_bytes(scfg, blk)
    ws = workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_denoise_step_hybrid(scfg, blk, dm.dm_hybrid_cfg(attn_period, attn_heads), csw, cbw, caw, tok.data_ptr(),
                              taud.data_ptr() if taud is not None else 0, logits.data_ptr(), 0, ws.data_ptr(), nb, st)
    dm.dm_check(st)
    return logits.float().cpu().numpy().astype(np.float64)


def run_generate(shape, dtype, sw, tokens, vocab, u_keep, u_cat, steps, mask_id, vocab_real, t_eps=1e-3, tau=None, d_ff=0,
                 want_trace=True, rms_eps=1e-5, ln_eps=1e-5):
    """dm_generate on host arrays: u_keep, u_cat [steps + 1, B, L]; tau [steps + 1, B, d_c] or None.  Returns (tokens_out, trace)."""
    n_layers = len(sw["layers"])
    scfg = dm.dm_stack_cfg(cfg_of(shape, dtype), n_layers, vocab, rms_eps)
    dsw = dev_stack_weights(sw, dtype)
    csw, keep = dm.make_stack_weights(dsw)
    blk = cbw = taud = None
    if tau is not None:
        blk = dm.dm_block_cfg(d_ff, tau.shape[-1], ln_eps)
        dbw = dev_block_weights(sw, dtype)
        cbw = dm.make_block_weights(dbw)
        taud = dev(np.asarray(tau, np.float32))
    tok = dev(np.asarray(tokens, np.int32))
    out = torch.full_like(tok, -7)
    trace = torch.full((steps + 1,) + tuple(tok.shape), -7, device="cuda", dtype=torch.int32) if want_trace else None
    uk, uc = dev(np.asarray(u_keep, np.float32)), dev(np.asarray(u_cat, np.float32))
    nb = dm.dm_generate_workspace_bytes(scfg, blk)
    ws = workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_generate(scfg, blk, csw, cbw, dm.dm_generate_cfg(steps, t_eps, mask_id, vocab_real), tok.data_ptr(),
                   taud.data_ptr() if taud is not None else 0, uk.data_ptr(), uc.data_ptr(), out.data_ptr(),
                   trace.data_ptr() if want_trace else 0, ws.data_ptr(), nb, st)
    dm.dm_check(st)
    return out.cpu().numpy(), (trace.cpu().numpy() if want_trace else None)
