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


def _case(B, L, H, seed, w_scale, dh=64):
    d = dh * H
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


@pytest.mark.parametrize("L", [5, 129, 300, 1000])
def test_heads_of_80_channels(G, L):
    """The head width of the paper's 1.3B hybrid (d_model 1920 = 24 heads of 80): three heads, so that the first, a middle and the
    last head (whose second sub-tile runs past the end of the row) are all there."""
    x, wq, wo = _case(2, L, 3, 40 + L, 1.0, dh=80)
    got = _run(G, x, wq, wo, 3)
    want = O.attention_mixer(x, wq, wo, 3)
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= BF16_REL, G.rel_l2(got, want)
    assert G.max_abs(got, want) <= BF16_ABS, G.max_abs(got, want)


def test_heads_of_80_channels_peaked_scores(G):
    x, wq, wo = _case(2, 400, 6, 17, 2.0, dh=80)
    got = _run(G, x, wq, wo, 6)
    want = O.attention_mixer(x, wq, wo, 6)
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


def test_hybrid_stack_with_heads_of_80(G):
    """d_model 160 = 2 attention heads of 80 beside Mamba layers of 5 heads x 64 channels."""
    shape = I.MixerShape(2, 150, 160, 2, 128, 4, 5)
    V = 504
    sw, tau, d_ff = _hybrid_stack(shape, 4, V, 23, False)
    tok = I.make_tokens(2, 150, V - 1, V - 1, seed=23)
    want = O.denoise_step_hybrid(tok, sw, attn_period=3, attn_heads=2, tau=tau, **G.oracle_kwargs(shape))
    got = G.run_denoise_hybrid(shape, I.BF16, sw, tok, V, 3, 2, tau=tau, d_ff=d_ff)
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= 1e-2, G.rel_l2(got, want)


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


@pytest.mark.parametrize("dh", [64, 80])
def test_attention_block_step_with_cache(G, dh):
    """Prefix of 200 tokens through the block entry point with an empty cache, then a block of 40 that attends to the cached
    prefix and to itself: outputs and cache contents against the oracle; rows past the valid keys of the cache hold NaN on
    purpose (the kernel must not let them in)."""
    from paper_2511_15927_b200 import binding as dm
    B, H, cap = 2, 2, 300
    d = dh * H
    x, wq, wo = _case(B, 240, H, 31, 1.0, dh=dh)
    wqd, wod = G.dev(wq, I.BF16), G.dev(wo, I.BF16)
    kc = torch.full((B, cap, d), float("nan"), device="cuda", dtype=torch.bfloat16)
    vc = torch.full((B, cap, d), float("nan"), device="cuda", dtype=torch.bfloat16)
    st = torch.cuda.current_stream().cuda_stream

    def run(xb, cache_len):
        xd = G.dev(xb, I.BF16)
        yd = torch.empty_like(xd)
        nb = dm.dm_attention_workspace_bytes(B, xb.shape[1], d, dm.DM_BF16)
        ws = G.workspace(nb)
        dm.dm_attention_block_step(B, xb.shape[1], d, H, dm.DM_BF16, wqd.data_ptr(), wod.data_ptr(), xd.data_ptr(), kc.data_ptr(), vc.data_ptr(),
                                   cache_len, cap, yd.data_ptr(), ws.data_ptr(), nb, st)
        dm.dm_check(st)
        return yd.float().cpu().numpy().astype(np.float64)

    y1 = run(np.ascontiguousarray(x[:, :200]), 0)
    w1, k1, v1 = O.attention_block_step(x[:, :200], wq, wo, H)
    assert np.all(np.isfinite(y1)) and G.rel_l2(y1, w1) <= BF16_REL
    y2 = run(np.ascontiguousarray(x[:, 200:]), 200)
    # the oracle continues from the cache as the library stores it (bf16)
    k1r, v1r = kc[:, :200].float().cpu().numpy().astype(np.float64), vc[:, :200].float().cpu().numpy().astype(np.float64)
    assert G.rel_l2(k1r, k1) <= 5e-3 and G.rel_l2(v1r, v1) <= 5e-3
    w2, k2, v2 = O.attention_block_step(x[:, 200:], wq, wo, H, k1r, v1r)
    assert np.all(np.isfinite(y2)) and G.rel_l2(y2, w2) <= BF16_REL and G.max_abs(y2, w2) <= BF16_ABS
    assert G.rel_l2(kc[:, :240].float().cpu().numpy().astype(np.float64), k2) <= 5e-3
    assert torch.isnan(kc[:, 240:]).all() and torch.isnan(vc[:, 240:]).all()          # nothing written past the block
    before = dm.dm_kernel_launch_count()
    with pytest.raises(dm.DmError):
        run(np.ascontiguousarray(x[:, :100]), 250)                                     # 250 + 100 > cap
    assert dm.dm_kernel_launch_count() == before


def test_hybrid_stack_block_mode(G):
    """Prefix pass commits Mamba states and key/value caches, the next block starts from them (Sec. 4.3)."""
    from paper_2511_15927_b200 import binding as dm
    import tests.gpu_util as U
    B, G1, G2, V, layers, period, heads = 2, 96, 32, 504, 4, 2, 2
    full = I.MixerShape(B, G1 + G2, 128, 2, 128, 4, 4)
    sw, _, _ = _hybrid_stack(full, layers, V, 41, False)
    tok = I.make_tokens(B, G1 + G2, V - 1, V - 1, seed=41)
    kw = G.oracle_kwargs(full)
    want1, st_o = O.denoise_step_hybrid(tok[:, :G1], sw, attn_period=period, attn_heads=heads, return_states=True, **kw)
    d, cap = full.d_model, 160
    dsw = U.dev_stack_weights(sw, I.BF16)
    csw, keep = dm.make_stack_weights(dsw)
    daw = [{"w_qkv": G.dev(l["w_qkv"], I.BF16), "w_o": G.dev(l["w_o"], I.BF16)} for l in sw["layers"]]
    caw = dm.make_attn_weights(daw)
    caches = [(torch.zeros((B, cap, d), device="cuda", dtype=torch.bfloat16), torch.zeros((B, cap, d), device="cuda", dtype=torch.bfloat16)) for _ in range(layers)]
    ssm = [torch.zeros((B, full.n_heads, full.headdim, full.d_state), device="cuda") for _ in range(layers)]
    conv = [torch.zeros((B, full.d_conv - 1, full.conv_ch), device="cuda", dtype=torch.bfloat16) for _ in range(layers)]
    st = torch.cuda.current_stream().cuda_stream

    def step(tokens, L, cache_len, first):
        shape = I.MixerShape(B, L, full.d_model, 2, full.d_state, 4, full.n_heads)
        scfg = dm.dm_stack_cfg(U.cfg_of(shape, I.BF16), layers, V, 1e-5)
        states = (dm.dm_layer_state * layers)()
        ast = (dm.dm_attn_state * layers)()
        for i in range(layers):
            if first:
                states[i] = dm.dm_layer_state(None, None, ssm[i].data_ptr(), conv[i].data_ptr())       # commit
            else:
                states[i] = dm.dm_layer_state(ssm[i].data_ptr(), conv[i].data_ptr(), None, None)       # read only
            ast[i] = dm.dm_attn_state(caches[i][0].data_ptr(), caches[i][1].data_ptr(), cache_len, cap)
        td = G.dev(np.asarray(tokens, np.int32))
        logits = torch.empty((B, L, V), device="cuda", dtype=torch.bfloat16)
        nb = dm.dm_denoise_hybrid_workspace_bytes(scfg, None)
        ws = G.workspace(nb)
        dm.dm_denoise_step_hybrid_block(scfg, None, dm.dm_hybrid_cfg(period, heads), csw, None, caw, td.data_ptr(), 0, logits.data_ptr(), 0,
                                        states, ast, ws.data_ptr(), nb, st)
        dm.dm_check(st)
        return logits.float().cpu().numpy().astype(np.float64)

    got1 = step(tok[:, :G1], G1, 0, True)
    assert G.rel_l2(got1, want1) <= 1e-2, G.rel_l2(got1, want1)
    # the oracle continues from the states as the library holds them
    st_in = []
    for i in range(layers):
        if i % period == 0:
            st_in.append((caches[i][0][:, :G1].float().cpu().numpy().astype(np.float64), caches[i][1][:, :G1].float().cpu().numpy().astype(np.float64)))
        else:
            st_in.append((ssm[i].cpu().numpy().astype(np.float64), conv[i].float().cpu().numpy().astype(np.float64)))
    want2, _ = O.denoise_step_hybrid(tok[:, G1:], sw, attn_period=period, attn_heads=heads, states_in=st_in, return_states=True, **kw)
    got2 = step(tok[:, G1:], G2, G1, False)
    assert G.rel_l2(got2, want2) <= 1e-2, G.rel_l2(got2, want2)
