"""GPU parity of dm_generate (the K-step generation loop of Sec. 2 Eq. 3 / Sec. 4.3 around the reverse step) against the
same loop written with the CPU oracle's denoiser, reverse step and noise schedule.

The loop's decisions are index work and must be bit-exact: which positions stay masked after every step is fixed by the
uniforms and the float32 keep probabilities alone, a drawn token never changes again, the prompt is carried through, and
no mask is left at the end.  A drawn token is decided by floating-point sums, so each step is checked teacher-forced: the
oracle runs one reverse step from the library's own tokens before that step, and the library's draw must own its uniform
in the oracle's cumulative distribution widened by the measured logit error (the check of the single-step test)."""
import numpy as np
import pytest

from oracle import bimamba_oracle as O
from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu
EPS32 = float(np.float32(1e-3))            # the sampling eps as the float the C struct carries


@pytest.fixture(scope="module")
def G():
    from paper_2511_15927_b200 import build
    build.build()
    import tests.gpu_util as g
    return g


def _stack(dtype, shape, layers, V, cond, seed):
    sw = I.make_stack_weights(shape, layers, V, seed=seed, dtype=dtype, perturb=True)
    for k in ("embed", "w_vocab"):                            # a peaked distribution instead of near-uniform logits
        sw[k] = I.round_to_bf16(8.0 * np.asarray(sw[k], np.float32)) if dtype == I.BF16 else 8.0 * np.asarray(sw[k], np.float32)
    if cond:
        I.add_block_weights(sw, shape, 2 * shape.d_model, 32, seed=seed, dtype=dtype)
    return sw


@pytest.mark.parametrize("dtype,N,d,H,V,cond,K", [(I.F32, 16, 64, 4, 120, False, 4), (I.BF16, 128, 128, 4, 600, True, 6), (I.BF16, 16, 128, 4, 304, False, 1)])
def test_generation_loop_against_the_oracle_loop(G, dtype, N, d, H, V, cond, K):
    from tests.test_gpu_sampler import _check_draws
    B, L, layers = 2, 48, 2
    shape = I.MixerShape(B, L, d, 2, N, 4, H)
    vocab_real, mask_id = V - 7, V - 8
    sw = _stack(dtype, shape, layers, V, cond, seed=11 + K)
    r = np.random.default_rng(K)
    uk, uc = r.random((K + 1, B, L), dtype=np.float32), r.random((K + 1, B, L), dtype=np.float32)
    tau = np.stack([I.make_timestep_embedding(B, 32, seed=100 + k) for k in range(K + 1)]) if cond else None
    start = np.full((B, L), mask_id, np.int32)
    start[0, 5], start[1, 40] = 3, 9                                           # a prompt of two tokens
    out, trace = G.run_generate(shape, dtype, sw, start, V, uk, uc, K, mask_id, vocab_real, t_eps=EPS32, tau=tau, d_ff=2 * d)
    np.testing.assert_array_equal(trace[K], out)
    assert not np.any(out == mask_id) and out[0, 5] == 3 and out[1, 40] == 9
    # the mask pattern after every step, from the uniforms alone
    keeps = O.generation_keep_probs(K, EPS32)
    alive = start == mask_id
    for k in range(K + 1):
        alive = alive & (uk[k] < keeps[k])
        np.testing.assert_array_equal(trace[k] == mask_id, alive)
    # every step against the oracle's step from the same tokens
    kw = G.oracle_kwargs(shape)
    agree = total = 0
    for k in range(K + 1):
        before = start if k == 0 else trace[k - 1]
        ref_logits = O.denoise_step_cond(before, tau[k], sw, **kw) if cond else O.denoise_step(before, sw, **kw)
        want = O.reverse_step(before, ref_logits[..., :vocab_real], uk[k], uc[k], float(keeps[k]), mask_id)
        drawn = (before == mask_id) & (trace[k] != mask_id)
        np.testing.assert_array_equal(trace[k][~drawn], want[~drawn])           # carried over / still masked: exact
        gl, _, _ = G.run_denoise(shape, dtype, sw, before, V, want_argmax=False, tau=None if tau is None else tau[k], d_ff=2 * d)
        eps = np.abs(gl[..., :vocab_real] - ref_logits[..., :vocab_real]).max()
        assert eps <= (1e-4 if dtype == I.F32 else 1e-2) * np.abs(ref_logits).max()
        _check_draws(before, trace[k], ref_logits, uk[k], uc[k], float(keeps[k]), mask_id, vocab_real, slack=np.expm1(2 * eps) + 2e-5)
        agree += int((trace[k][drawn] == want[drawn]).sum()); total += int(drawn.sum())
    assert total == B * L - 2 and agree > total // 2                            # every masked position is drawn exactly once
    # the whole loop again without the trace: the result alone, through the two alternating token buffers
    out2, _ = G.run_generate(shape, dtype, sw, start, V, uk, uc, K, mask_id, vocab_real, t_eps=EPS32, tau=tau, d_ff=2 * d, want_trace=False)
    np.testing.assert_array_equal(out2, out)


def test_generation_argument_checks(G):
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(1, 8, 64, 2, 16, 4, 4)
    sw = I.make_stack_weights(shape, 1, 50, seed=9, dtype=I.F32)
    u = np.zeros((3, 1, 8), np.float32)
    tok = np.full((1, 8), 49, np.int32)
    before = dm.dm_kernel_launch_count()
    for steps, eps in ((0, 1e-3), (2, 0.0), (2, 1.0)):
        with pytest.raises(dm.DmError):
            G.run_generate(shape, I.F32, sw, tok, 50, u, u, steps, 49, 50, t_eps=eps)
    assert dm.dm_kernel_launch_count() == before
