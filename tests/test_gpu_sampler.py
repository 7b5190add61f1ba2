"""GPU parity of dm_denoise_sample_step (one reverse step of the masked diffusion, Sec. 2 Eq. 3) against the CPU oracle.
Index work (which positions are carried over, stay masked, are drawn) is compared bit-exactly; the drawn token is decided
by floating-point sums, so it is checked against the cumulative distribution of the library's own stored logits: the
token must own the interval that contains u_cat, up to rounding at the interval's ends."""
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


def _check_draws(tokens_in, tokens_out, logits, u_keep, u_cat, keep_prob, mask_id, vocab_real, slack):
    B, L = tokens_in.shape
    n_drawn = 0
    for b in range(B):
        for t in range(L):
            if tokens_in[b, t] != mask_id:
                assert tokens_out[b, t] == tokens_in[b, t]                     # carried over
            elif np.float32(u_keep[b, t]) < np.float32(keep_prob):
                assert tokens_out[b, t] == mask_id                             # stays masked
            else:
                n_drawn += 1
                v = int(tokens_out[b, t])
                assert 0 <= v < vocab_real and v != mask_id
                z = logits[b, t, :vocab_real].astype(np.float64).copy()
                z[mask_id] = -np.inf
                p = np.exp(z - z[np.isfinite(z)].max())
                cdf = np.cumsum(p) / p.sum()
                lo, hi = (cdf[v - 1] if v > 0 else 0.0), cdf[v]
                assert p[v] > 0 and lo - slack <= u_cat[b, t] <= hi + slack, (b, t, v, lo, hi, u_cat[b, t])
    return n_drawn


@pytest.mark.parametrize("dtype,N,d,H,V,vocab_real,cond", [(I.F32, 16, 64, 4, 200, 190, False), (I.BF16, 128, 128, 4, 1000, 950, False),
                                                          (I.BF16, 16, 128, 4, 3000, 2999, True)])
def test_reverse_step_against_oracle(G, dtype, N, d, H, V, vocab_real, cond):
    B, L, layers = 3, 90, 2
    shape = I.MixerShape(B, L, d, 2, N, 4, H)
    mask_id = vocab_real - 1
    sw = I.make_stack_weights(shape, layers, V, seed=7, dtype=dtype, perturb=True)
    for k in ("embed", "w_vocab"):                            # larger logits than N(0, 0.02) weights give: a peaked distribution
        sw[k] = I.round_to_bf16(8.0 * np.asarray(sw[k], np.float32)) if dtype == I.BF16 else 8.0 * np.asarray(sw[k], np.float32)
    tau, d_ff = None, 0
    if cond:
        d_ff = 2 * d
        I.add_block_weights(sw, shape, d_ff, 32, seed=7, dtype=dtype)
        tau = I.make_timestep_embedding(B, 32, seed=7)
    tok = I.make_tokens(B, L, mask_id, mask_id, seed=7)
    r = np.random.default_rng(7)
    u_keep, u_cat = r.random((B, L), dtype=np.float32), r.random((B, L), dtype=np.float32)
    keep_prob = 0.45
    out = G.run_sample_step(shape, dtype, sw, tok, V, u_keep, u_cat, keep_prob, mask_id, vocab_real, tau=tau, d_ff=d_ff)
    # the library's own logits for the same input (same kernels): the draw is checked against their distribution
    logits, _, _ = G.run_denoise(shape, dtype, sw, tok, V, want_argmax=False, tau=tau, d_ff=d_ff)
    n = _check_draws(tok, out, logits, u_keep, u_cat, keep_prob, mask_id, vocab_real, slack=2e-5 if dtype == I.F32 else 2e-4)
    assert 10 < n < B * L
    # and against the oracle end to end: same decisions everywhere; the drawn tokens agree except where u_cat sits next to
    # a boundary of the oracle's distribution (its logits differ from the stored ones by the stack's rounding)
    kw = G.oracle_kwargs(shape)
    ref_logits = O.denoise_step_cond(tok, tau, sw, **kw) if cond else O.denoise_step(tok, sw, **kw)
    want = O.reverse_step(tok, ref_logits[..., :vocab_real], u_keep, u_cat, keep_prob, mask_id)
    same_kind = (out == mask_id) == (want == mask_id)
    assert same_kind.all()
    drawn = (tok == mask_id) & (out != mask_id)
    np.testing.assert_array_equal(out[~drawn], want[~drawn])
    # If every logit is off by at most eps, every normalised probability changes by a factor within exp(+-2 eps), hence
    # every value of the cumulative distribution by at most exp(2 eps) - 1: the drawn token must own u_cat in the
    # oracle's distribution widened by that much.
    eps = np.abs(logits[..., :vocab_real] - ref_logits[..., :vocab_real]).max()
    assert eps <= (1e-4 if dtype == I.F32 else 1e-2) * np.abs(ref_logits).max()
    _check_draws(tok, out, ref_logits, u_keep, u_cat, keep_prob, mask_id, vocab_real, slack=np.expm1(2 * eps) + 2e-5)
    assert (out[drawn] == want[drawn]).mean() > 0.5           # and most draws coincide outright

def test_keep_everything_or_nothing_and_determinism(G):
    shape = I.MixerShape(2, 40, 64, 2, 16, 4, 4)
    V, mask_id = 120, 100
    sw = I.make_stack_weights(shape, 1, V, seed=8, dtype=I.F32)
    tok = I.make_tokens(2, 40, mask_id, mask_id, seed=8)
    r = np.random.default_rng(8)
    uk, uc = r.random((2, 40), dtype=np.float32), r.random((2, 40), dtype=np.float32)
    none = G.run_sample_step(shape, I.F32, sw, tok, V, uk, uc, 1.0, mask_id, 101)
    np.testing.assert_array_equal(none, tok)                                  # s = t: nothing changes
    full = G.run_sample_step(shape, I.F32, sw, tok, V, uk, uc, 0.0, mask_id, 101)
    assert np.all(full != mask_id) and np.all(full < 101) and np.all(full[tok != mask_id] == tok[tok != mask_id])
    np.testing.assert_array_equal(full, G.run_sample_step(shape, I.F32, sw, tok, V, uk, uc, 0.0, mask_id, 101))   # run to run
    # u_cat = 0 takes the first token with probability mass
    first = G.run_sample_step(shape, I.F32, sw, tok, V, uk, 0 * uc, 0.0, mask_id, 101)
    assert np.all(first[tok == mask_id] == 0)


def test_sample_step_argument_checks(G):
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(1, 8, 64, 2, 16, 4, 4)
    sw = I.make_stack_weights(shape, 1, 50, seed=9, dtype=I.F32)
    tok = I.make_tokens(1, 8, 49, 49, seed=9)
    u = np.zeros((1, 8), np.float32)
    before = dm.dm_kernel_launch_count()
    for bad in (dict(keep_prob=1.5), dict(mask_id=50), dict(vocab_real=51), dict(vocab_real=0)):
        kw = dict(keep_prob=0.5, mask_id=49, vocab_real=50); kw.update(bad)
        with pytest.raises(dm.DmError):
            G.run_sample_step(shape, I.F32, sw, tok, 50, u, u, kw["keep_prob"], kw["mask_id"], kw["vocab_real"])
    assert dm.dm_kernel_launch_count() == before
