"""Thin ctypes binding of libdm_bimamba.so: argument marshalling only.

Every function here has the name and the arguments of the C entry point it calls (see
include/dm_bimamba.h).  Device buffers are passed as integer addresses (`tensor.data_ptr()`), host
buffers likewise; this module never computes anything and there is no fallback: if the compiled
library is missing, importing the module raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
# DM_BIMAMBA_LIB selects another build of the same library (e.g. one compiled with different flags).
LIB_PATH = os.environ.get("DM_BIMAMBA_LIB") or os.path.join(_HERE, "libdm_bimamba.so")

DM_OK, DM_ERR_INVALID_ARG, DM_ERR_UNSUPPORTED, DM_ERR_WORKSPACE, DM_ERR_CUDA, DM_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5
DM_F32, DM_BF16 = 0, 1
DM_FLAG_GATED_RMSNORM, DM_FLAG_CONV_BIAS, DM_FLAG_D_SKIP, DM_FLAG_TIED_PROJ = 1, 2, 4, 8
DM_DIR_FWD, DM_DIR_REV, DM_DIR_BOTH = 1, 2, 3
DM_FLAGS_DEFAULT = DM_FLAG_GATED_RMSNORM | DM_FLAG_CONV_BIAS | DM_FLAG_D_SKIP


class dm_mixer_cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "seqlen", "d_model", "expand", "d_state", "d_conv", "n_heads",
                                         "n_groups", "dtype", "flags", "dir_mask", "chunk")] + [("norm_eps", C.c_float)]


class dm_dir_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_in", "conv_w", "conv_b", "dt_bias", "A_log", "D", "norm_w", "w_out")]


class dm_layer_weights(C.Structure):
    _fields_ = [("norm_w", C.c_void_p), ("dir", dm_dir_weights * 2)]


class dm_stack_cfg(C.Structure):
    _fields_ = [("mixer", dm_mixer_cfg), ("n_layers", C.c_int32), ("vocab", C.c_int32), ("rms_eps", C.c_float)]


class dm_stack_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("layers", C.POINTER(dm_layer_weights)), ("final_norm_w", C.c_void_p),
                ("w_vocab", C.c_void_p)]


class dm_layer_state(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ssm_in", "conv_in", "ssm_out", "conv_out")]


class dm_block_cfg(C.Structure):
    _fields_ = [("d_ff", C.c_int32), ("d_cond", C.c_int32), ("ln_eps", C.c_float)]


class dm_hybrid_cfg(C.Structure):
    _fields_ = [("attn_period", C.c_int32), ("attn_heads", C.c_int32)]


class dm_attn_weights(C.Structure):
    _fields_ = [("w_qkv", C.c_void_p), ("w_o", C.c_void_p)]


class dm_attn_state(C.Structure):
    _fields_ = [("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("len", C.c_int32), ("cap", C.c_int32)]


class dm_sample_cfg(C.Structure):
    _fields_ = [("mask_id", C.c_int32), ("vocab_real", C.c_int32), ("keep_prob", C.c_float)]


class dm_generate_cfg(C.Structure):
    _fields_ = [("steps", C.c_int32), ("t_eps", C.c_float), ("mask_id", C.c_int32), ("vocab_real", C.c_int32)]


class dm_block_weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_cond", "b_cond", "w_up", "b_up", "w_down", "b_down")]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_15927_b200.build` "
                      "(or __graft_entry__.build()); there is no fallback path")
_lib = C.CDLL(LIB_PATH)

_vp, _sz = C.c_void_p, C.c_size_t
_lib.dm_status_string.restype = C.c_char_p
_lib.dm_status_string.argtypes = [C.c_int]
_lib.dm_last_error_message.restype = C.c_char_p
_lib.dm_last_error_message.argtypes = []
_lib.dm_kernel_launch_count.restype = C.c_uint64
_lib.dm_kernel_launch_count.argtypes = []
_lib.dm_bimamba_workspace_bytes.argtypes = [C.POINTER(dm_mixer_cfg), C.POINTER(_sz)]
_lib.dm_denoise_workspace_bytes.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(_sz)]
_lib.dm_check.argtypes = [_vp]
_lib.dm_bimamba_forward.argtypes = [C.POINTER(dm_mixer_cfg), C.POINTER(dm_dir_weights), _vp, _vp, _vp, _sz, _vp]
_lib.dm_bimamba_forward_host.argtypes = [C.POINTER(dm_mixer_cfg), C.POINTER(dm_dir_weights), _vp, _vp, _vp, _sz, _vp]
_lib.dm_bimamba_forward_static.argtypes = [C.POINTER(dm_mixer_cfg), C.POINTER(dm_dir_weights), _vp, _vp, _vp]
_lib.dm_bimamba_forward_static.restype = C.c_int
_lib.dm_bimamba_block_step.argtypes = [C.POINTER(dm_mixer_cfg), C.POINTER(dm_dir_weights), _vp, _vp, _vp, _vp, _vp, _vp,
                                       _vp, _sz, _vp]
_lib.dm_denoise_step.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_stack_weights), _vp, _vp, _vp,
                                 C.POINTER(dm_layer_state), _vp, _sz, _vp]
_lib.dm_denoise_cond_workspace_bytes.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(_sz)]
_lib.dm_denoise_cond_workspace_bytes.restype = C.c_int
_lib.dm_denoise_step_cond.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(dm_stack_weights),
                                      C.POINTER(dm_block_weights), _vp, _vp, _vp, _vp, C.POINTER(dm_layer_state), _vp, _sz, _vp]
_lib.dm_denoise_step_cond.restype = C.c_int
_lib.dm_denoise_sample_workspace_bytes.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(_sz)]
_lib.dm_denoise_sample_workspace_bytes.restype = C.c_int
_lib.dm_denoise_sample_step.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(dm_stack_weights),
                                        C.POINTER(dm_block_weights), _vp, _vp, C.POINTER(dm_sample_cfg), _vp, _vp, _vp,
                                        C.POINTER(dm_layer_state), _vp, _sz, _vp]
_lib.dm_denoise_sample_step.restype = C.c_int
_lib.dm_generate_workspace_bytes.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(_sz)]
_lib.dm_generate_workspace_bytes.restype = C.c_int
_lib.dm_generate.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(dm_stack_weights), C.POINTER(dm_block_weights),
                             C.POINTER(dm_generate_cfg), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.dm_generate.restype = C.c_int
_lib.dm_denoise_hybrid_workspace_bytes.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(_sz)]
_lib.dm_denoise_hybrid_workspace_bytes.restype = C.c_int
_lib.dm_denoise_step_hybrid.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(dm_hybrid_cfg), C.POINTER(dm_stack_weights),
                                        C.POINTER(dm_block_weights), C.POINTER(dm_attn_weights), _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.dm_denoise_step_hybrid.restype = C.c_int
_lib.dm_denoise_step_hybrid_block.argtypes = [C.POINTER(dm_stack_cfg), C.POINTER(dm_block_cfg), C.POINTER(dm_hybrid_cfg), C.POINTER(dm_stack_weights),
                                              C.POINTER(dm_block_weights), C.POINTER(dm_attn_weights), _vp, _vp, _vp, _vp,
                                              C.POINTER(dm_layer_state), C.POINTER(dm_attn_state), _vp, _sz, _vp]
_lib.dm_denoise_step_hybrid_block.restype = C.c_int
_lib.dm_attention_block_step.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32,
                                         _vp, _vp, _sz, _vp]
_lib.dm_attention_block_step.restype = C.c_int
_lib.dm_attention_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(_sz)]
_lib.dm_attention_workspace_bytes.restype = C.c_int
_lib.dm_attention_forward.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.dm_attention_forward.restype = C.c_int
_lib.dm_selftest_wait_timeout.argtypes = [C.c_uint32, _vp, _vp]
_lib.dm_selftest_wait_timeout.restype = C.c_int
_lib.dm_linear.argtypes = [C.c_int, _vp, _vp, _vp, C.c_int, C.c_int64, C.c_int32, C.c_int32, _vp, _vp, _vp]
_lib.dm_linear.restype = C.c_int
_lib.dm_profile_enable.argtypes = [C.c_int]
_lib.dm_profile_read.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_uint64)]
for _f in ("dm_profile_enable", "dm_profile_read", "dm_bimamba_workspace_bytes", "dm_denoise_workspace_bytes", "dm_check", "dm_bimamba_forward",
           "dm_bimamba_forward_host", "dm_bimamba_block_step", "dm_denoise_step"):
    getattr(_lib, _f).restype = C.c_int

EXPORTS = ("dm_status_string", "dm_last_error_message", "dm_kernel_launch_count", "dm_bimamba_workspace_bytes",
           "dm_denoise_workspace_bytes", "dm_check", "dm_bimamba_forward", "dm_bimamba_forward_host",
           "dm_bimamba_block_step", "dm_denoise_step", "dm_profile_enable", "dm_profile_read", "dm_linear", "dm_bimamba_forward_static",
           "dm_denoise_cond_workspace_bytes", "dm_denoise_step_cond", "dm_denoise_sample_workspace_bytes", "dm_denoise_sample_step",
           "dm_attention_workspace_bytes", "dm_attention_forward", "dm_denoise_hybrid_workspace_bytes", "dm_denoise_step_hybrid",
           "dm_denoise_step_hybrid_block", "dm_attention_block_step", "dm_generate_workspace_bytes", "dm_generate", "dm_selftest_wait_timeout", "dm_selftest_withhold_prep")
DM_STATIC_WORKSPACE_BYTES = 32 << 20
DM_STAGE_IN_PROJ, DM_STAGE_SCAN, DM_STAGE_OUT_PROJ, DM_STAGE_COUNT = 0, 1, 2, 3


class DmError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"{dm_status_string(status)} ({status}): {dm_last_error_message()}")


def _ok(status: int) -> None:
    if status != DM_OK:
        raise DmError(status)


def dm_status_string(status: int) -> str:
    return _lib.dm_status_string(int(status)).decode()


def dm_last_error_message() -> str:
    return _lib.dm_last_error_message().decode()


def dm_kernel_launch_count() -> int:
    return int(_lib.dm_kernel_launch_count())


def dm_profile_enable(on: bool) -> None:
    _ok(_lib.dm_profile_enable(1 if on else 0))


def dm_profile_read():
    """Returns (ms, spans): two lists indexed by DM_STAGE_*."""
    ms = (C.c_float * DM_STAGE_COUNT)()
    n = (C.c_uint64 * DM_STAGE_COUNT)()
    _ok(_lib.dm_profile_read(ms, n))
    return list(ms), [int(v) for v in n]


def dm_bimamba_workspace_bytes(cfg: dm_mixer_cfg) -> int:
    n = _sz(0)
    _ok(_lib.dm_bimamba_workspace_bytes(C.byref(cfg), C.byref(n)))
    return int(n.value)


def dm_denoise_workspace_bytes(cfg: dm_stack_cfg) -> int:
    n = _sz(0)
    _ok(_lib.dm_denoise_workspace_bytes(C.byref(cfg), C.byref(n)))
    return int(n.value)


def dm_check(cuda_stream: int = 0) -> None:
    _ok(_lib.dm_check(_vp(cuda_stream)))


def _dirs(w) -> C.Array:
    arr = (dm_dir_weights * 2)()
    for i in range(2):
        arr[i] = w[i]
    return arr


def dm_bimamba_forward(cfg, w, x: int, y: int, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    _ok(_lib.dm_bimamba_forward(C.byref(cfg), _dirs(w), _vp(x), _vp(y), _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_bimamba_forward_host(cfg, w, x_host: int, y_host: int, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    _ok(_lib.dm_bimamba_forward_host(C.byref(cfg), _dirs(w), _vp(x_host), _vp(y_host), _vp(workspace), _sz(workspace_bytes),
                                     _vp(cuda_stream)))


def dm_bimamba_forward_static(cfg, w, x: int, y: int, cuda_stream: int = 0) -> None:
    """dm_bimamba_forward on the library's built-in scratch array (no workspace argument, nothing allocated)."""
    _ok(_lib.dm_bimamba_forward_static(C.byref(cfg), _dirs(w), _vp(x), _vp(y), _vp(cuda_stream)))


def dm_linear(dtype: int, x: int, w: int, y: int, y_dtype: int, rows: int, in_features: int, out_features: int,
              row_scale: int = 0, addend: int = 0, cuda_stream: int = 0) -> None:
    _ok(_lib.dm_linear(dtype, _vp(x), _vp(w), _vp(y), y_dtype, rows, in_features, out_features, _vp(row_scale or None),
                       _vp(addend or None), _vp(cuda_stream)))


def dm_bimamba_block_step(cfg, w, x_blk: int, ssm_state_in: int, conv_state_in: int, ssm_state_out: int,
                          conv_state_out: int, y_blk: int, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    _ok(_lib.dm_bimamba_block_step(C.byref(cfg), _dirs(w), _vp(x_blk), _vp(ssm_state_in or None), _vp(conv_state_in or None),
                                   _vp(ssm_state_out or None), _vp(conv_state_out or None), _vp(y_blk), _vp(workspace),
                                   _sz(workspace_bytes), _vp(cuda_stream)))


def dm_denoise_step(cfg, weights, tokens: int, logits: int, argmax_out: int, states, workspace: int,
                    workspace_bytes: int, cuda_stream: int = 0) -> None:
    """`states`: None, or a ctypes array (dm_layer_state * n_layers)."""
    _ok(_lib.dm_denoise_step(C.byref(cfg), C.byref(weights), _vp(tokens), _vp(logits or None), _vp(argmax_out or None),
                             states, _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_denoise_cond_workspace_bytes(cfg: dm_stack_cfg, blk: dm_block_cfg) -> int:
    n = _sz(0)
    _ok(_lib.dm_denoise_cond_workspace_bytes(C.byref(cfg), C.byref(blk), C.byref(n)))
    return n.value


def dm_denoise_step_cond(cfg, blk, weights, block_weights, tokens: int, tau: int, logits: int, argmax_out: int, states,
                         workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    """`block_weights`: ctypes array (dm_block_weights * n_layers); `states`: None or (dm_layer_state * n_layers)."""
    _ok(_lib.dm_denoise_step_cond(C.byref(cfg), C.byref(blk), C.byref(weights), block_weights, _vp(tokens), _vp(tau),
                                  _vp(logits or None), _vp(argmax_out or None), states, _vp(workspace), _sz(workspace_bytes),
                                  _vp(cuda_stream)))


def dm_denoise_sample_workspace_bytes(cfg: dm_stack_cfg, blk=None) -> int:
    n = _sz(0)
    _ok(_lib.dm_denoise_sample_workspace_bytes(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(n)))
    return n.value


def dm_denoise_sample_step(cfg, blk, weights, block_weights, tokens_in: int, tau: int, sample: dm_sample_cfg, u_keep: int,
                           u_cat: int, tokens_out: int, states, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    """blk / block_weights / tau: None (or 0) for the plain stack, else as in dm_denoise_step_cond."""
    _ok(_lib.dm_denoise_sample_step(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(weights), block_weights,
                                    _vp(tokens_in), _vp(tau or None), C.byref(sample), _vp(u_keep), _vp(u_cat), _vp(tokens_out),
                                    states, _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_selftest_withhold_prep(on: bool) -> None:
    _lib.dm_selftest_withhold_prep.argtypes = [C.c_int]
    _lib.dm_selftest_withhold_prep.restype = C.c_int
    _ok(_lib.dm_selftest_withhold_prep(1 if on else 0))


def dm_selftest_wait_timeout(limit_us: int, out: int, cuda_stream: int = 0) -> None:
    """out: device pointer to 3 uint64."""
    _ok(_lib.dm_selftest_wait_timeout(int(limit_us), _vp(out), _vp(cuda_stream)))


def dm_generate_workspace_bytes(cfg: dm_stack_cfg, blk=None) -> int:
    n = _sz(0)
    _ok(_lib.dm_generate_workspace_bytes(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(n)))
    return n.value


def dm_generate(cfg, blk, weights, block_weights, gen: dm_generate_cfg, tokens_in: int, tau: int, u_keep: int, u_cat: int,
                tokens_out: int, trace: int, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    """u_keep, u_cat: [steps + 1, B, L]; tau: [steps + 1, B, d_cond] or 0; trace: [steps + 1, B, L] or 0."""
    _ok(_lib.dm_generate(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(weights), block_weights, C.byref(gen),
                         _vp(tokens_in), _vp(tau or None), _vp(u_keep), _vp(u_cat), _vp(tokens_out), _vp(trace or None),
                         _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_denoise_hybrid_workspace_bytes(cfg: dm_stack_cfg, blk=None) -> int:
    n = _sz(0)
    _ok(_lib.dm_denoise_hybrid_workspace_bytes(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(n)))
    return n.value


def dm_denoise_step_hybrid(cfg, blk, hybrid: dm_hybrid_cfg, weights, block_weights, attn_weights, tokens: int, tau: int, logits: int,
                           argmax_out: int, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    """attn_weights: ctypes array (dm_attn_weights * n_layers); blk / block_weights / tau: None (0) for the plain stack."""
    _ok(_lib.dm_denoise_step_hybrid(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(hybrid), C.byref(weights),
                                    block_weights, attn_weights, _vp(tokens), _vp(tau or None), _vp(logits or None),
                                    _vp(argmax_out or None), _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_denoise_step_hybrid_block(cfg, blk, hybrid: dm_hybrid_cfg, weights, block_weights, attn_weights, tokens: int, tau: int, logits: int,
                                 argmax_out: int, states, attn_states, workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    """states: (dm_layer_state * n_layers) or None; attn_states: (dm_attn_state * n_layers)."""
    _ok(_lib.dm_denoise_step_hybrid_block(C.byref(cfg), C.byref(blk) if blk is not None else None, C.byref(hybrid), C.byref(weights),
                                          block_weights, attn_weights, _vp(tokens), _vp(tau or None), _vp(logits or None),
                                          _vp(argmax_out or None), states, attn_states, _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_attention_block_step(batch: int, block_len: int, d_model: int, n_heads: int, dtype: int, w_qkv: int, w_o: int, x_blk: int,
                            k_cache: int, v_cache: int, cache_len: int, cache_cap: int, y_blk: int, workspace: int,
                            workspace_bytes: int, cuda_stream: int = 0) -> None:
    _ok(_lib.dm_attention_block_step(batch, block_len, d_model, n_heads, dtype, _vp(w_qkv), _vp(w_o), _vp(x_blk), _vp(k_cache), _vp(v_cache),
                                     cache_len, cache_cap, _vp(y_blk), _vp(workspace), _sz(workspace_bytes), _vp(cuda_stream)))


def dm_attention_workspace_bytes(batch: int, seqlen: int, d_model: int, dtype: int) -> int:
    n = _sz(0)
    _ok(_lib.dm_attention_workspace_bytes(batch, seqlen, d_model, dtype, C.byref(n)))
    return n.value


def dm_attention_forward(batch: int, seqlen: int, d_model: int, n_heads: int, dtype: int, w_qkv: int, w_o: int, x: int, y: int,
                         workspace: int, workspace_bytes: int, cuda_stream: int = 0) -> None:
    _ok(_lib.dm_attention_forward(batch, seqlen, d_model, n_heads, dtype, _vp(w_qkv), _vp(w_o), _vp(x), _vp(y), _vp(workspace),
                                  _sz(workspace_bytes), _vp(cuda_stream)))


# ------------------------------------------------------------------------------------------------
# Marshalling helpers (no arithmetic): build the C structs from shapes and from dicts of tensors.
# ------------------------------------------------------------------------------------------------

def make_mixer_cfg(batch, seqlen, d_model, expand, d_state, d_conv, n_heads, dtype, n_groups=1,
                   flags=DM_FLAGS_DEFAULT, dir_mask=DM_DIR_BOTH, chunk=0, norm_eps=1e-5) -> dm_mixer_cfg:
    return dm_mixer_cfg(batch, seqlen, d_model, expand, d_state, d_conv, n_heads, n_groups, dtype, flags, dir_mask,
                        chunk, norm_eps)


def make_dir_weights(t: dict) -> dm_dir_weights:
    """t maps the field names of dm_dir_weights to objects with .data_ptr() (device tensors) or None."""
    return dm_dir_weights(*[(t[n].data_ptr() if t.get(n) is not None else None)
                            for n in ("w_in", "conv_w", "conv_b", "dt_bias", "A_log", "D", "norm_w", "w_out")])


def make_stack_weights(t: dict):
    """t: {"embed", "w_vocab", "final_norm_w", "layers": [{"norm_w", "fwd": {...}, "rev": {...}}]} of device tensors.
    Returns (dm_stack_weights, keepalive) -- keep the second object alive while the first is in use."""
    n = len(t["layers"])
    arr = (dm_layer_weights * n)()
    for i, l in enumerate(t["layers"]):
        arr[i].norm_w = l["norm_w"].data_ptr()
        arr[i].dir[0] = make_dir_weights(l["fwd"])
        arr[i].dir[1] = make_dir_weights(l["rev"])
    sw = dm_stack_weights(t["embed"].data_ptr(), C.cast(arr, C.POINTER(dm_layer_weights)), t["final_norm_w"].data_ptr(),
                          t["w_vocab"].data_ptr())
    return sw, arr


def make_block_weights(layers):
    """layers: list of {"w_cond", "b_cond", "w_up", "b_up", "w_down", "b_down"} of device tensors (biases may be None).
    Returns the ctypes array (dm_block_weights * n_layers)."""
    arr = (dm_block_weights * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = dm_block_weights(*[(l[n].data_ptr() if l.get(n) is not None else None)
                                    for n in ("w_cond", "b_cond", "w_up", "b_up", "w_down", "b_down")])
    return arr


def make_attn_weights(layers):
    """layers: list of {"w_qkv", "w_o"} of device tensors, or None for layers that are not attention."""
    arr = (dm_attn_weights * len(layers))()
    for i, l in enumerate(layers):
        if l is not None:
            arr[i] = dm_attn_weights(l["w_qkv"].data_ptr(), l["w_o"].data_ptr())
    return arr
