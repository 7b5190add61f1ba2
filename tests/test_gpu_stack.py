"""GPU parity of dm_denoise_step (embedding -> layers with RMSNorm pre-norm and residual -> vocabulary
projection) against the CPU oracle, full-sequence and block mode."""
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


def _argmax_ok(amax, logits_gpu, logits_ref, tol):
    """The arg-max is decided on the GPU's own (stored-precision) logits: it must index a maximal stored logit,
    lowest index on ties, and agree with the oracle wherever the oracle's top-2 margin exceeds the tolerance."""
    B, L, V = logits_ref.shape
    g = logits_gpu.reshape(-1, V); r = logits_ref.reshape(-1, V); a = amax.reshape(-1)
    np.testing.assert_array_equal(a, np.argmax(g, axis=1))                # bit-exact on the same stored values
    srt = np.sort(r, axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 2 * tol
    assert clear.any()
    np.testing.assert_array_equal(a[clear], np.argmax(r, axis=1)[clear])


@pytest.mark.parametrize("dtype,N,d,H,layers,V", [(I.F32, 16, 64, 4, 3, 200), (I.BF16, 16, 128, 4, 2, 304), (I.BF16, 128, 128, 4, 2, 1000)])
def test_denoise_step_full_sequence(G, dtype, N, d, H, layers, V):
    shape = I.MixerShape(2, 50, d, 2, N, 4, H)
    sw = I.make_stack_weights(shape, layers, V, seed=1, dtype=dtype, perturb=True)
    tok = I.make_tokens(2, 50, V - 1, V - 1, seed=1)
    want = O.denoise_step(tok, sw, **G.oracle_kwargs(shape))
    logits, amax, _ = G.run_denoise(shape, dtype, sw, tok, V)
    rel = G.rel_l2(logits, want)
    tol = 1e-4 if dtype == I.F32 else 1e-2
    assert rel <= tol, rel
    _argmax_ok(amax, logits, want, tol * np.abs(want).max())
    # arg-max only (no logits buffer): same indices
    _, amax2, _ = G.run_denoise(shape, dtype, sw, tok, V, want_logits=False)
    np.testing.assert_array_equal(amax, amax2)


@pytest.mark.parametrize("dtype", [I.F32, I.BF16])
def test_denoise_step_block_mode(G, dtype):
    d, N, H, V, layers = 64, 16, 4, 120, 2
    sw = I.make_stack_weights(I.MixerShape(1, 1, d, 2, N, 4, H), layers, V, seed=2, dtype=dtype, perturb=True)
    tok = I.make_tokens(2, 48, V - 1, V - 1, seed=2)
    tol = 1e-4 if dtype == I.F32 else 1e-2
    # prefix pass commits the state; the next block starts from it
    pre = I.MixerShape(2, 32, d, 2, N, 4, H)
    kw = G.oracle_kwargs(pre)
    want_pre, st_o = O.denoise_step(tok[:, :32], sw, return_states=True, **kw)
    got_pre, _, st_g = G.run_denoise(pre, dtype, sw, tok[:, :32], V, want_states=True)
    assert G.rel_l2(got_pre, want_pre) <= tol
    for (so, co), (sg, cg) in zip(st_o, st_g):
        assert G.rel_l2(sg, so) <= tol and G.rel_l2(cg, co) <= tol
    blk = I.MixerShape(2, 16, d, 2, N, 4, H)
    typed = [(s.astype(np.float32), I.round_to_bf16(c.astype(np.float32)) if dtype == I.BF16 else c.astype(np.float32)) for s, c in st_o]
    want_blk = O.denoise_step(tok[:, 32:], sw, states_in=typed, **kw)
    got_blk, _, _ = G.run_denoise(blk, dtype, sw, tok[:, 32:], V, states_in=typed)
    assert G.rel_l2(got_blk, want_blk) <= tol


@pytest.mark.parametrize("dtype,N,H,tol_chain", [(I.F32, 16, 4, 2e-4), (I.BF16, 128, 4, 2e-2), (I.BF16, 128, 8, 2e-2)])
def test_block_decoding_chain_with_commits(G, dtype, N, H, tol_chain):
    """Block-autoregressive decoding as Sec. 4.3 states it, chained on the library's own states: a prefix committed by one
    block step from empty state, then three blocks of 32 tokens, each with two read-only denoising passes over partly masked
    tokens and a commit pass over the final tokens that writes the state the next block starts from (ping-pong buffers).
    Every pass's logits and every committed state are compared with the oracle running the same chain on its own states:
    per pass at the single-call tolerance (teacher-forced: the oracle starts the pass from the library's state) and end to
    end, where the two chains never exchange anything, at twice that."""
    d, V, layers, B, Gb = 128, 200, 2, 2, 32
    P = 2 * d // H
    sw = I.make_stack_weights(I.MixerShape(1, 1, d, 2, N, 4, H), layers, V, seed=5, dtype=dtype, perturb=True)
    mask_id = V - 1
    tol = 1e-4 if dtype == I.F32 else 1e-2
    r = np.random.default_rng(5)
    pre_len = 40
    final_tok = r.integers(0, mask_id, (B, pre_len + 3 * Gb)).astype(np.int32)            # the tokens every block ends up with
    kw = G.oracle_kwargs(I.MixerShape(B, Gb, d, 2, N, 4, H))
    typed = lambda st: [(s.astype(np.float32), I.round_to_bf16(c.astype(np.float32)) if dtype == I.BF16 else c.astype(np.float32)) for s, c in st]

    pre = I.MixerShape(B, pre_len, d, 2, N, 4, H)
    want, st_o = O.denoise_step(final_tok[:, :pre_len], sw, return_states=True, **kw)
    got, _, st_g = G.run_denoise(pre, dtype, sw, final_tok[:, :pre_len], V, want_states=True)
    assert G.rel_l2(got, want) <= tol
    blk = I.MixerShape(B, Gb, d, 2, N, 4, H)
    for bi in range(3):
        lo = pre_len + bi * Gb
        fin = final_tok[:, lo:lo + Gb]
        st_g_in, st_o_in = typed(st_g), typed(st_o)
        for p in range(2):                                    # read-only passes: part of the block still masked
            tok = fin.copy()
            tok[r.random((B, Gb)) < (0.7 - 0.4 * p)] = mask_id
            got, _, none = G.run_denoise(blk, dtype, sw, tok, V, states_in=st_g_in)
            assert none is None
            assert G.rel_l2(got, O.denoise_step(tok, sw, states_in=st_g_in, **kw)) <= tol, (bi, p)             # from the same state
            assert G.rel_l2(got, O.denoise_step(tok, sw, states_in=st_o_in, **kw)) <= tol_chain, (bi, p)       # chain against chain
        got, _, st_g = G.run_denoise(blk, dtype, sw, fin, V, states_in=st_g_in, want_states=True)               # commit pass
        want_tf, st_tf = O.denoise_step(fin, sw, states_in=st_g_in, return_states=True, **kw)
        want, st_o = O.denoise_step(fin, sw, states_in=st_o_in, return_states=True, **kw)
        assert G.rel_l2(got, want_tf) <= tol and G.rel_l2(got, want) <= tol_chain, bi
        for (sg, cg), (s1, c1), (s2, c2) in zip(st_g, st_tf, st_o):
            assert sg.shape == (B, H, P, N)
            assert G.rel_l2(sg, s1) <= tol and G.rel_l2(cg, c1) <= tol and G.rel_l2(sg, s2) <= tol_chain, bi
