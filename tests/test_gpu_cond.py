"""GPU parity of dm_denoise_step_cond (the timestep-conditioned block of App. A.1 in every layer: AdaLN, mixer,
gated residual, AdaLN, MLP, gated residual) against the CPU oracle, full-sequence and block mode."""
import numpy as np
import pytest

from oracle import bimamba_oracle as O
from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    from paper_2511_15927_b200 import build
    build.build()
    import tests.gpu_util as g
    return g


def _stack(shape, layers, V, d_ff, d_c, seed, dtype):
    sw = I.make_stack_weights(shape, layers, V, seed=seed, dtype=dtype, perturb=True)
    I.add_block_weights(sw, shape, d_ff, d_c, seed=seed, dtype=dtype)
    return sw, I.make_timestep_embedding(shape.batch, d_c, seed=seed)


@pytest.mark.parametrize("dtype,N,d,H,layers,V,d_ff,d_c", [(I.F32, 16, 64, 4, 3, 200, 128, 24),      # CUDA-core GEMMs, sequential scan
                                                          (I.BF16, 128, 128, 4, 2, 1000, 256, 128),   # tensor-core GEMMs and scan
                                                          (I.BF16, 16, 256, 8, 2, 304, 520, 40)])      # padded d_state, odd widths
def test_conditioned_step_full_sequence(G, dtype, N, d, H, layers, V, d_ff, d_c):
    shape = I.MixerShape(3, 70, d, 2, N, 4, H)
    sw, tau = _stack(shape, layers, V, d_ff, d_c, 3, dtype)
    tok = I.make_tokens(3, 70, V - 1, V - 1, seed=3)
    want = O.denoise_step_cond(tok, tau, sw, **G.oracle_kwargs(shape))
    logits, amax, _ = G.run_denoise(shape, dtype, sw, tok, V, tau=tau, d_ff=d_ff)
    tol = 1e-4 if dtype == I.F32 else 1e-2
    assert np.all(np.isfinite(logits))
    assert G.rel_l2(logits, want) <= tol, G.rel_l2(logits, want)
    np.testing.assert_array_equal(amax.reshape(-1), np.argmax(logits.reshape(-1, V), axis=1))   # decided on the stored logits
    # each sequence is modulated by its own timestep: changing tau of row 1 leaves rows 0 and 2 bit-identical
    tau2 = tau.copy(); tau2[1] += 0.5
    logits2, _, _ = G.run_denoise(shape, dtype, sw, tok, V, tau=tau2, d_ff=d_ff)
    np.testing.assert_array_equal(logits2[[0, 2]], logits[[0, 2]])
    assert np.any(logits2[1] != logits[1])


def test_shut_gates_reduce_the_stack_to_its_head(G):
    """W_cond = 0 and b_cond = 0 shut every gate: the logits are the head applied to the embeddings (a closed form)."""
    shape = I.MixerShape(2, 40, 128, 2, 128, 4, 4)
    V = 504
    sw, tau = _stack(shape, 2, V, 256, 64, 4, I.BF16)
    for l in sw["layers"]:
        l["w_cond"] = 0 * l["w_cond"]; l["b_cond"] = 0 * l["b_cond"]
    tok = I.make_tokens(2, 40, V - 1, V - 1, seed=4)
    e = np.asarray(sw["embed"], np.float64)[tok]
    head = e / np.sqrt(np.mean(e ** 2, -1, keepdims=True) + 1e-5) * np.asarray(sw["final_norm_w"], np.float64) @ np.asarray(sw["w_vocab"], np.float64).T
    logits, _, _ = G.run_denoise(shape, I.BF16, sw, tok, V, tau=tau, d_ff=256)
    assert G.rel_l2(logits, head) <= 1e-2


@pytest.mark.parametrize("dtype", [I.F32, I.BF16])
def test_conditioned_step_block_mode(G, dtype):
    """Prefix pass commits the state, the next block starts from it (Sec. 4.3), with the conditioned block in every layer."""
    d, N, H, V, layers, d_ff, d_c = 64, 16, 4, 120, 2, 128, 16
    full = I.MixerShape(2, 48, d, 2, N, 4, H)
    sw, tau = _stack(full, layers, V, d_ff, d_c, 5, dtype)
    tok = I.make_tokens(2, 48, V - 1, V - 1, seed=5)
    tol = 1e-4 if dtype == I.F32 else 1e-2
    pre = I.MixerShape(2, 32, d, 2, N, 4, H)
    kw = G.oracle_kwargs(pre)
    want_pre, st_o = O.denoise_step_cond(tok[:, :32], tau, sw, return_states=True, **kw)
    got_pre, _, st_g = G.run_denoise(pre, dtype, sw, tok[:, :32], V, want_states=True, tau=tau, d_ff=d_ff)
    assert G.rel_l2(got_pre, want_pre) <= tol
    for (so, co), (sg, cg) in zip(st_o, st_g):
        assert G.rel_l2(sg, so) <= tol and G.rel_l2(cg, co) <= tol
    blk = I.MixerShape(2, 16, d, 2, N, 4, H)
    st_in = [(s.astype(np.float32), (I.round_to_bf16(c.astype(np.float32)) if dtype == I.BF16 else c.astype(np.float32))) for s, c in st_o]
    want_blk, _ = O.denoise_step_cond(tok[:, 32:], tau, sw, states_in=st_in, return_states=True, **kw)
    got_blk, _, _ = G.run_denoise(blk, dtype, sw, tok[:, 32:], V, states_in=st_in, want_states=True, tau=tau, d_ff=d_ff)
    assert G.rel_l2(got_blk, want_blk) <= tol


def test_conditioned_step_argument_checks(G):
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(1, 8, 64, 2, 16, 4, 4)
    sw, tau = _stack(shape, 1, 50, 128, 8, 6, I.F32)
    tok = I.make_tokens(1, 8, 49, 49, seed=6)
    with pytest.raises(dm.DmError):
        G.run_denoise(shape, I.F32, sw, tok, 50, tau=tau, d_ff=0)          # d_ff must be positive
    before = dm.dm_kernel_launch_count()
    with pytest.raises(dm.DmError):
        G.run_denoise(I.MixerShape(1, 8, 66, 2, 16, 4, 3), I.F32, sw, tok, 50, tau=tau, d_ff=128)   # d_model not a multiple of 4
    assert dm.dm_kernel_launch_count() == before
