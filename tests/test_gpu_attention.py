"""GPU parity of dm_attention_forward (the hybrid's bidirectional multi-head attention mixer, Sec. 3.3) against the CPU
oracle: lengths around the 128-token tiles, several heads and sequences, a peaked and a flat score distribution."""
import numpy as np
import pytest
import torch

from oracle import bimamba_oracle as O
from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu
BF16_REL, BF16_ABS = 1e-2, 5e-2


@pytest.fixture(scope="module")
def G():
    from paper_2511_15927_b200 import build
    build.build()
    import tests.gpu_util as g
    return g


def _run(G, x, w_qkv, w_o, H):
    from paper_2511_15927_b200 import binding as dm
    B, L, d = x.shape
    xd, wq, wo = G.dev(x, I.BF16), G.dev(w_qkv, I.BF16), G.dev(w_o, I.BF16)
    yd = torch.empty_like(xd)
    nb = dm.dm_attention_workspace_bytes(B, L, d, dm.DM_BF16)
    ws = G.workspace(nb)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_attention_forward(B, L, d, H, dm.DM_BF16, wq.data_ptr(), wo.data_ptr(), xd.data_ptr(), yd.data_ptr(), ws.data_ptr(), nb, st)
    dm.dm_check(st)
    return yd.float().cpu().numpy().astype(np.float64)


def _case(B, L, H, seed, w_scale):
    d = 64 * H
    r = np.random.default_rng(seed)
    x = I.round_to_bf16(r.standard_normal((B, L, d), dtype=np.float32))
    w_qkv = I.round_to_bf16((w_scale / np.sqrt(d)) * r.standard_normal((3 * d, d), dtype=np.float32))
    w_o = I.round_to_bf16((1.0 / np.sqrt(d)) * r.standard_normal((d, d), dtype=np.float32))
    return x, w_qkv, w_o


@pytest.mark.parametrize("L", [1, 5, 127, 128, 129, 256, 300, 1000])
def test_lengths_around_the_tiles(G, L):
    x, wq, wo = _case(2, L, 2, L, 1.0)
    got = _run(G, x, wq, wo, 2)
    want = O.attention_mixer(x, wq, wo, 2)
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= BF16_REL, G.rel_l2(got, want)
    assert G.max_abs(got, want) <= BF16_ABS, G.max_abs(got, want)


@pytest.mark.parametrize("w_scale", [0.05, 2.0])
def test_flat_and_peaked_scores_many_heads(G, w_scale):
    """Small projections give nearly uniform attention (every output close to the mean value); large ones give scores with a
    standard deviation of 4 and maxima near 15, where the running maximum matters.  (Larger still, and the bf16 rounding of
    the stored Q and K alone moves the scores by more than the tolerance allows: an error of 2^-9 on a score of 50 is 0.1 in
    the exponent.)"""
    x, wq, wo = _case(3, 400, 8, 11, w_scale)
    got = _run(G, x, wq, wo, 8)
    want = O.attention_mixer(x, wq, wo, 8)
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= BF16_REL, G.rel_l2(got, want)
    assert G.max_abs(got, want) <= BF16_ABS * max(1.0, np.abs(want).max()), G.max_abs(got, want)


def test_permutation_equivariance_and_determinism(G):
    """No position encoding, no mask: permuting the tokens permutes the outputs (up to the order of the fp32 sums)."""
    x, wq, wo = _case(1, 333, 2, 12, 1.0)
    a = _run(G, x, wq, wo, 2)
    np.testing.assert_array_equal(a, _run(G, x, wq, wo, 2))
    perm = np.random.default_rng(3).permutation(333)
    bperm = _run(G, np.ascontiguousarray(x[:, perm]), wq, wo, 2)
    assert G.rel_l2(bperm, a[:, perm]) <= 5e-3


def test_attention_argument_checks(G):
    from paper_2511_15927_b200 import binding as dm
    x, wq, wo = _case(1, 16, 2, 13, 1.0)
    before = dm.dm_kernel_launch_count()
    with pytest.raises(dm.DmError):
        _run(G, x, wq, wo, 4)                                # heads of width 32: unsupported
    assert dm.dm_kernel_launch_count() == before


def _hybrid_stack(shape, layers, V, seed, cond):
    sw = I.make_stack_weights(shape, layers, V, seed=seed, dtype=I.BF16, perturb=True)
    d = shape.d_model
    r = np.random.default_rng(seed)
    for i, l in enumerate(sw["layers"]):
        l["w_qkv"] = I.round_to_bf16((1.0 / np.sqrt(d)) * r.standard_normal((3 * d, d), dtype=np.float32))
        l["w_o"] = I.round_to_bf16((0.5 / np.sqrt(d)) * r.standard_normal((d, d), dtype=np.float32))
    tau, d_ff = None, 0
    if cond:
        d_ff = 2 * d
        I.add_block_weights(sw, shape, d_ff, 32, seed=seed, dtype=I.BF16)
        tau = I.make_timestep_embedding(shape.batch, 32, seed=seed)
    return sw, tau, d_ff


@pytest.mark.parametrize("cond", [False, True])
def test_hybrid_stack_against_the_oracle(G, cond):
    """Attention mixer in layers 0 and 3 of a 5-layer stack (period 3), bidirectional Mamba elsewhere."""
    shape = I.MixerShape(2, 150, 128, 2, 128, 4, 4)          # d_model 128 = 2 attention heads of 64
    V = 504
    sw, tau, d_ff = _hybrid_stack(shape, 5, V, 21, cond)
    tok = I.make_tokens(2, 150, V - 1, V - 1, seed=21)
    want = O.denoise_step_hybrid(tok, sw, attn_period=3, attn_heads=2, tau=tau, **G.oracle_kwargs(shape))
    got = G.run_denoise_hybrid(shape, I.BF16, sw, tok, V, 3, 2, tau=tau, d_ff=d_ff)
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= 1e-2, G.rel_l2(got, want)
    # period 0: no attention layer; identical to the stack without the hybrid entry point
    plain, _, _ = G.run_denoise(shape, I.BF16, sw, tok, V, want_argmax=False, tau=tau, d_ff=d_ff)
    np.testing.assert_array_equal(G.run_denoise_hybrid(shape, I.BF16, sw, tok, V, 0, 2, tau=tau, d_ff=d_ff), plain)
    assert np.any(got != plain)
