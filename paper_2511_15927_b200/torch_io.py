"""Marshalling between host numpy arrays and device tensors for callers of the binding (torch is used for
device memory and streams only)."""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from paper_2511_15927_b200 import binding as dm
from paper_2511_15927_b200 import inputs as I

TYPED = ("w_in", "conv_w", "conv_b", "norm_w", "w_out")


def tdtype(dtype):
    return torch.bfloat16 if dtype == I.BF16 else torch.float32


def dm_dtype(dtype):
    return dm.DM_BF16 if dtype == I.BF16 else dm.DM_F32


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(tdtype(dtype)) if dtype is not None else t


def dev_dir_weights(w: dict, dtype) -> dict:
    return {k: (dev(v, dtype if k in TYPED else None) if v is not None else None) for k, v in w.items()}


def cfg_of(shape: I.MixerShape, dtype, flags=dm.DM_FLAGS_DEFAULT, dir_mask=dm.DM_DIR_BOTH, chunk=0, eps=1e-5):
    return dm.make_mixer_cfg(shape.batch, shape.seqlen, shape.d_model, shape.expand, shape.d_state, shape.d_conv,
                             shape.n_heads, dm_dtype(dtype), shape.n_groups, flags, dir_mask, chunk, eps)


def workspace(nbytes: int) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")


def dev_stack_weights(sw: dict, dtype) -> dict:
    return {"embed": dev(sw["embed"], dtype), "w_vocab": dev(sw["w_vocab"], dtype),
            "final_norm_w": dev(sw["final_norm_w"], dtype),
            "layers": [{"norm_w": dev(l["norm_w"], dtype), "fwd": dev_dir_weights(l["fwd"], dtype),
                        "rev": dev_dir_weights(l["rev"], dtype)} for l in sw["layers"]]}


def dev_block_weights(sw: dict, dtype) -> list:
    """The timestep-conditioned block's parameters of every layer: matrices in the I/O dtype, biases in fp32."""
    f32 = lambda a: None if a is None else dev(np.asarray(a, np.float32))
    return [{"w_cond": dev(l["w_cond"], dtype), "b_cond": f32(l.get("b_cond")), "w_up": dev(l["w_up"], dtype),
             "b_up": f32(l.get("b_up")), "w_down": dev(l["w_down"], dtype), "b_down": f32(l.get("b_down"))}
            for l in sw["layers"]]


