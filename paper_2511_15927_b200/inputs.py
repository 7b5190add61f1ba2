"""Seeded synthetic inputs for the bidirectional Mamba-2 mixer and its layer stack.

This module only *draws numbers*: activations, weights, token ids.  It holds none of the
mixer's arithmetic, so both the CPU oracle's tests and the CUDA path's tests can feed the very
same host buffers to their side without sharing any of the method's code.

Distributions (per direction, forward and reverse drawn independently):

    x            ~ N(0, 1)
    w_in, w_out  ~ N(0, 0.02)          (also embeddings and the vocabulary projection)
    A_log        = log U[1, 16]        one value per head
    dt_bias      = softplus^-1(exp U[log 1e-3, log 1e-1])   one value per head
    conv_w/b     ~ U(-k^-1/2, k^-1/2)  k = d_conv
    D, norm_w    = 1                   (or U[0.5, 1.5] with perturb=True, so that a test notices
                                        a kernel that ignores them)

Every tensor comes from its own Philox (counter-based) stream keyed by (seed, tensor name), so
drawing one tensor never shifts another.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass

import numpy as np

F32 = "f32"
BF16 = "bf16"


@dataclass(frozen=True)
class MixerShape:
    """Sizes of one bidirectional mixer call, in the paper's notation (App. C table)."""
    batch: int
    seqlen: int
    d_model: int
    expand: int = 2
    d_state: int = 16
    d_conv: int = 4
    n_heads: int = 8
    n_groups: int = 1

    @property
    def d_inner(self) -> int:
        return self.expand * self.d_model

    @property
    def headdim(self) -> int:
        return self.d_inner // self.n_heads

    @property
    def conv_ch(self) -> int:
        return self.d_inner + 2 * self.n_groups * self.d_state

    @property
    def d_in_proj(self) -> int:
        return 2 * self.d_inner + 2 * self.n_groups * self.d_state + self.n_heads


def _rng(seed: int, name: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), zlib.crc32(name.encode())]))


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(bf16_bits(a)).reshape(np.shape(a))


def _typed(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == BF16 else a


def make_activations(shape: MixerShape, seed: int = 0, dtype: str = F32, name: str = "x") -> np.ndarray:
    """x [B, L, d_model] ~ N(0,1); float32 values (bf16-representable when dtype is bf16)."""
    g = _rng(seed, name)
    x = g.standard_normal((shape.batch, shape.seqlen, shape.d_model), dtype=np.float32)
    return _typed(x, dtype)


def make_dir_weights(shape: MixerShape, seed: int = 0, direction: str = "fwd", dtype: str = F32,
                     perturb: bool = False, prefix: str = "") -> dict:
    """One direction's parameter set.  Matrices are [out_features, in_features], row-major."""
    s = shape
    tag = f"{prefix}{direction}."
    k = s.d_conv
    bound = k ** -0.5
    w = {}
    w["w_in"] = _typed(0.02 * _rng(seed, tag + "w_in").standard_normal((s.d_in_proj, s.d_model), dtype=np.float32), dtype)
    w["conv_w"] = _typed(_rng(seed, tag + "conv_w").uniform(-bound, bound, (s.conv_ch, k)), dtype)
    w["conv_b"] = _typed(_rng(seed, tag + "conv_b").uniform(-bound, bound, (s.conv_ch,)), dtype)
    w["A_log"] = np.log(_rng(seed, tag + "A_log").uniform(1.0, 16.0, (s.n_heads,))).astype(np.float32)
    dt = np.exp(_rng(seed, tag + "dt").uniform(np.log(1e-3), np.log(1e-1), (s.n_heads,)))
    w["dt_bias"] = (dt + np.log(-np.expm1(-dt))).astype(np.float32)   # inverse of softplus
    if perturb:
        w["D"] = _rng(seed, tag + "D").uniform(0.5, 1.5, (s.n_heads,)).astype(np.float32)
        w["norm_w"] = _typed(_rng(seed, tag + "norm_w").uniform(0.5, 1.5, (s.d_inner,)), dtype)
    else:
        w["D"] = np.ones((s.n_heads,), dtype=np.float32)
        w["norm_w"] = np.ones((s.d_inner,), dtype=np.float32)
    w["w_out"] = _typed(0.02 * _rng(seed, tag + "w_out").standard_normal((s.d_model, s.d_inner), dtype=np.float32), dtype)
    return w


def make_mixer_weights(shape: MixerShape, seed: int = 0, dtype: str = F32, perturb: bool = False,
                       prefix: str = "") -> tuple:
    """(forward weights, reverse weights): untied, drawn independently."""
    return (make_dir_weights(shape, seed, "fwd", dtype, perturb, prefix),
            make_dir_weights(shape, seed, "rev", dtype, perturb, prefix))


def make_states(shape: MixerShape, seed: int = 0, dtype: str = F32, scale: float = 0.5) -> tuple:
    """A non-trivial carried state: ssm [B,H,P,N] float32 and conv [B, d_conv-1, conv_ch]."""
    s = shape
    ssm = scale * _rng(seed, "ssm_state").standard_normal((s.batch, s.n_heads, s.headdim, s.d_state), dtype=np.float32)
    conv = _rng(seed, "conv_state").standard_normal((s.batch, s.d_conv - 1, s.conv_ch), dtype=np.float32)
    return ssm.astype(np.float32), _typed(conv, dtype)


def make_tokens(batch: int, seqlen: int, vocab_real: int, mask_id: int, seed: int = 0) -> np.ndarray:
    """Token ids uniform over [0, vocab_real); in row b each position is replaced by mask_id with
    probability t_b, t_b ~ U[0,1] (the forward masking process, Eq. 1)."""
    g = _rng(seed, "tokens")
    ids = g.integers(0, vocab_real, (batch, seqlen), dtype=np.int64)
    t = g.uniform(0.0, 1.0, (batch, 1))
    masked = g.uniform(0.0, 1.0, (batch, seqlen)) < t
    ids[masked] = mask_id
    return ids.astype(np.int32)


def make_stack_weights(shape: MixerShape, n_layers: int, vocab: int, seed: int = 0, dtype: str = F32,
                       perturb: bool = False) -> dict:
    """Embedding [V,d], per layer (pre-norm weight [d], forward and reverse mixer weights), final norm
    weight [d], vocabulary projection [V,d]."""
    s = shape
    sw = {"embed": _typed(0.02 * _rng(seed, "embed").standard_normal((vocab, s.d_model), dtype=np.float32), dtype),
          "w_vocab": _typed(0.02 * _rng(seed, "w_vocab").standard_normal((vocab, s.d_model), dtype=np.float32), dtype),
          "layers": []}
    for i in range(n_layers):
        if perturb:
            nw = _typed(_rng(seed, f"L{i}.norm").uniform(0.5, 1.5, (s.d_model,)), dtype)
        else:
            nw = np.ones((s.d_model,), dtype=np.float32)
        f, r = make_mixer_weights(s, seed, dtype, perturb, prefix=f"L{i}.")
        sw["layers"].append({"norm_w": nw, "fwd": f, "rev": r})
    sw["final_norm_w"] = (_typed(_rng(seed, "final_norm").uniform(0.5, 1.5, (s.d_model,)), dtype)
                          if perturb else np.ones((s.d_model,), dtype=np.float32))
    return sw


def add_block_weights(sw: dict, shape: MixerShape, d_ff: int, d_cond: int, seed: int = 0, dtype: str = F32) -> dict:
    """Adds the timestep-conditioned block's parameters to every layer of `sw` (App. A.1): the modulation
    map W_cond [6 d, d_c] with its bias (shift rows start at 0, scale and gate rows at 1, so that the block
    is not degenerate at tau = 0) and the MLP d -> d_ff -> d with biases."""
    d = shape.d_model
    for i, layer in enumerate(sw["layers"]):
        g = lambda name: _rng(seed, f"L{i}.{name}")
        layer["w_cond"] = _typed(0.02 * g("w_cond").standard_normal((6 * d, d_cond), dtype=np.float32), dtype)
        base = np.tile(np.repeat(np.array([0.0, 1.0, 1.0], np.float32), d), 2)
        layer["b_cond"] = (base + 0.1 * g("b_cond").standard_normal((6 * d,), dtype=np.float32)).astype(np.float32)
        layer["w_up"] = _typed(0.02 * g("w_up").standard_normal((d_ff, d), dtype=np.float32), dtype)
        layer["b_up"] = (0.02 * g("b_up").standard_normal((d_ff,), dtype=np.float32)).astype(np.float32)
        layer["w_down"] = _typed(0.02 * g("w_down").standard_normal((d, d_ff), dtype=np.float32), dtype)
        layer["b_down"] = (0.02 * g("b_down").standard_normal((d,), dtype=np.float32)).astype(np.float32)
    return sw


def make_timestep_embedding(batch: int, d_cond: int, seed: int = 0) -> np.ndarray:
    """tau_t of each sequence, [B, d_c] fp32 (stands in for the output of the paper's timestep MLP)."""
    return _rng(seed, "tau").standard_normal((batch, d_cond), dtype=np.float32)


# The benchmark configurations (batch, L, d_model, heads, d_state) with their I/O dtype.
CONFIGS = {
    "cfg0": (MixerShape(1, 256, 128, 2, 16, 4, 8), F32),
    "cfg1": (MixerShape(8, 2048, 2048, 2, 128, 4, 64), BF16),
    "cfg2_layer": (MixerShape(4, 4096, 1024, 2, 16, 4, 32), BF16),
    "cfg3_8k": (MixerShape(1, 8192, 2048, 2, 128, 4, 64), BF16),
    "cfg3_16k": (MixerShape(1, 16384, 2048, 2, 128, 4, 64), BF16),
    "cfg3_32k": (MixerShape(1, 32768, 2048, 2, 128, 4, 64), BF16),
    "cfg3_64k": (MixerShape(1, 65536, 2048, 2, 128, 4, 64), BF16),      # the longest context of the paper's throughput sweep (Sec. 4.3)
    "cfg4_block": (MixerShape(16, 32, 2048, 2, 128, 4, 64), BF16),
    "paper_1p3b": (MixerShape(1, 1024, 1920, 2, 128, 4, 120), BF16),
    "paper_1p3b_8k": (MixerShape(1, 8192, 1920, 2, 128, 4, 120), BF16),
}
