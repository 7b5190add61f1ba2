"""GPU parity of the tensor-core chunked scan (bf16, d_state 128, headdim 64) against the CPU oracle:
lengths around the 128-token chunk, direction masks, flag variants, state in/out, determinism."""
import numpy as np
import pytest

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


def _shape(B, L, H=8, k=4):
    return I.MixerShape(B, L, 32 * H, 2, 128, k, H)        # d_inner = 64*H, headdim 64, d_in_proj multiple of 8


def _check(G, got, want):
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= BF16_REL, G.rel_l2(got, want)
    assert G.max_abs(got, want) <= BF16_ABS, G.max_abs(got, want)


@pytest.mark.parametrize("L", [64, 127, 128, 129, 255, 256, 257, 300, 1000])
def test_lengths_around_the_chunk(G, L):
    shape = _shape(2, L)
    wf, wr = I.make_mixer_weights(shape, L, I.BF16, perturb=True)
    x = I.make_activations(shape, L, I.BF16)
    got = G.run_forward(shape, I.BF16, wf, wr, x)
    _check(G, got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape)))


@pytest.mark.parametrize("flags", [7, 6, 5, 3, 0])
@pytest.mark.parametrize("k", [4, 2])
def test_flags_and_conv_width(G, flags, k):
    shape = _shape(1, 200, k=k)
    wf, wr = I.make_mixer_weights(shape, 3, I.BF16, perturb=True)
    x = I.make_activations(shape, 3, I.BF16)
    got = G.run_forward(shape, I.BF16, wf, wr, x, flags=flags)
    _check(G, got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape, flags)))


def test_directions_reversal_and_determinism(G):
    shape = _shape(2, 333)
    wf, wr = I.make_mixer_weights(shape, 4, I.BF16, perturb=True)
    x = I.make_activations(shape, 4, I.BF16)
    kw = G.oracle_kwargs(shape)
    f = G.run_forward(shape, I.BF16, wf, wr, x, dir_mask=1)
    r = G.run_forward(shape, I.BF16, wf, wr, x, dir_mask=2)
    _check(G, f, O.bimamba_forward(x, wf, wr, dir_mask=O.DIR_FWD, **kw))
    _check(G, r, O.bimamba_forward(x, wf, wr, dir_mask=O.DIR_REV, **kw))
    both = G.run_forward(shape, I.BF16, wf, wr, x)
    np.testing.assert_array_equal(both, G.run_forward(shape, I.BF16, wf, wr, x))          # run to run
    # reverse layer with W on u == flip(forward layer with W on flip(u)); chunk grids differ for ragged L
    f_on_flipped = G.run_forward(shape, I.BF16, wr, wr, np.ascontiguousarray(x[:, ::-1]), dir_mask=1)
    assert G.rel_l2(r, f_on_flipped[:, ::-1]) <= 5e-3
    x2 = x.copy(); x2[0, 150] += 1.0                                                       # causality
    df = G.run_forward(shape, I.BF16, wf, wr, x2, dir_mask=1) - f
    dr = G.run_forward(shape, I.BF16, wf, wr, x2, dir_mask=2) - r
    assert np.all(df[0, :150] == 0) and np.all(dr[0, 151:] == 0) and np.all(df[1] == 0) and np.all(dr[1] == 0)
    assert np.any(df[0, 150:] != 0) and np.any(dr[0, :151] != 0)


def test_state_in_and_out(G):
    """Long blocks run on the tensor-core path with an incoming SSM state and commit the outgoing one."""
    shape = _shape(2, 200)
    wf, wr = I.make_mixer_weights(shape, 5, I.BF16, perturb=True)
    x = I.make_activations(shape, 5, I.BF16)
    kw = G.oracle_kwargs(shape)
    ssm_in, _ = I.make_states(shape, 5, I.BF16)
    y_o, s_o, c_o = O.bimamba_block_step(x, wf, wr, ssm_state_in=ssm_in, **kw)
    y_g, s_g, c_g = G.run_block_step(shape, I.BF16, wf, wr, x, ssm_in, None)
    _check(G, y_g, y_o)
    _check(G, s_g, s_o)
    _check(G, c_g, c_o)
    # two 128-token blocks chained through the returned state == one 256-token pass (forward direction)
    s2 = _shape(1, 256)
    x2 = I.make_activations(s2, 6, I.BF16)
    whole, s_whole, _ = G.run_block_step(s2, I.BF16, wf, wr, x2, dir_mask=1)
    half = _shape(1, 128)
    y1, s1, c1 = G.run_block_step(half, I.BF16, wf, wr, np.ascontiguousarray(x2[:, :128]), dir_mask=1)
    y2, s2_, _ = G.run_block_step(half, I.BF16, wf, wr, np.ascontiguousarray(x2[:, 128:]), s1.astype(np.float32), c1.astype(np.float32), dir_mask=1)
    assert G.rel_l2(np.concatenate([y1, y2], axis=1), whole) <= 5e-3
    assert G.rel_l2(s2_, s_whole) <= 5e-3


@pytest.mark.parametrize("N,H", [(16, 8), (32, 8), (64, 8)])
def test_smaller_d_state_runs_zero_padded(G, N, H):
    """d_state below 128 takes the same kernel with B', C' and the state zero-padded: parity of the output, and the
    carried state in the model's own [B, H, P, d_state] layout, in and out."""
    shape = I.MixerShape(2, 300, 32 * H, 2, N, 4, H)
    assert shape.d_in_proj % 8 == 0                         # 16-byte rows: the tensor-core path takes the shape
    wf, wr = I.make_mixer_weights(shape, 20 + N, I.BF16, perturb=True)
    x = I.make_activations(shape, 20 + N, I.BF16)
    kw = G.oracle_kwargs(shape)
    _check(G, G.run_forward(shape, I.BF16, wf, wr, x), O.bimamba_forward(x, wf, wr, **kw))
    ssm_in, conv_in = I.make_states(shape, 20 + N, I.BF16)
    y_o, s_o, c_o = O.bimamba_block_step(x, wf, wr, ssm_state_in=ssm_in, conv_state_in=conv_in, **kw)
    y_g, s_g, c_g = G.run_block_step(shape, I.BF16, wf, wr, x, ssm_in, conv_in)
    assert s_g.shape == s_o.shape == (2, H, 64, N)
    _check(G, y_g, y_o)
    _check(G, s_g, s_o)
    _check(G, c_g, c_o)


@pytest.mark.parametrize("N", [128, 16])
def test_half_width_heads_run_with_padded_channels(G, N):
    """headdim 32 (the paper's 1.3B shape: 120 heads of 32, App. A.1) takes the same kernel: a CTA loads 64 channels, of
    which the second half (the next head's) is padding that never leaves it.  Parity of the output, the last head
    included, and of the carried state in the model's [B, H, 32, d_state] layout."""
    H = 8
    shape = I.MixerShape(2, 300, 128, 2, N, 4, H)           # d_inner 256 = 8 heads of 32
    assert shape.headdim == 32 and shape.d_in_proj % 8 == 0
    wf, wr = I.make_mixer_weights(shape, 40 + N, I.BF16, perturb=True)
    x = I.make_activations(shape, 40 + N, I.BF16)
    kw = G.oracle_kwargs(shape)
    for flags in (7, 6):                                    # with and without the gated norm (its sum of squares covers 32 channels)
        _check(G, G.run_forward(shape, I.BF16, wf, wr, x, flags=flags), O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape, flags)))
    ssm_in, conv_in = I.make_states(shape, 40 + N, I.BF16)
    y_o, s_o, c_o = O.bimamba_block_step(x, wf, wr, ssm_state_in=ssm_in, conv_state_in=conv_in, **kw)
    y_g, s_g, c_g = G.run_block_step(shape, I.BF16, wf, wr, x, ssm_in, conv_in)
    assert s_g.shape == s_o.shape == (2, H, 32, N)
    _check(G, y_g, y_o)
    _check(G, s_g, s_o)
    _check(G, c_g, c_o)


@pytest.mark.parametrize("seed", range(12))
def test_seeded_mix_of_shapes_and_options(G, seed):
    """A seeded draw over what the kernel takes -- length, batch, headdim 64 or 32, d_state, conv width, flags,
    direction mask, carried state or none -- against the oracle: combinations that the other tests visit one at a time."""
    r = np.random.default_rng(1000 + seed)
    P = int(r.choice([64, 32]))
    H = int(r.choice([2, 4, 8])) * (2 if P == 32 else 1)
    N = int(r.choice([128, 64, 32, 16]))
    while (2 * N + H) % 8:                                   # 16-byte rows of the in_proj output
        H += 2 if P == 32 else 1
    d_inner = P * H
    B, L, k = int(r.integers(1, 4)), int(r.integers(1, 700)), int(r.choice([4, 4, 3, 2]))
    flags = int(r.choice([7, 7, 6, 5, 3]))
    dir_mask = int(r.choice([3, 3, 1, 2]))
    shape = I.MixerShape(B, L, d_inner // 2, 2, N, k, H)
    assert shape.headdim == P and shape.d_in_proj % 8 == 0
    wf, wr = I.make_mixer_weights(shape, seed, I.BF16, perturb=True)
    x = I.make_activations(shape, seed, I.BF16)
    kw = G.oracle_kwargs(shape, flags)
    if r.random() < 0.5:
        ssm_in, conv_in = I.make_states(shape, seed, I.BF16)
        y_o, s_o, c_o = O.bimamba_block_step(x, wf, wr, ssm_state_in=ssm_in, conv_state_in=conv_in, dir_mask=dir_mask, **kw)
        want_state = bool(dir_mask & 1)
        y_g, s_g, c_g = G.run_block_step(shape, I.BF16, wf, wr, x, ssm_in, conv_in, want_state=want_state, flags=flags, dir_mask=dir_mask)
        _check(G, y_g, y_o)
        if want_state:
            _check(G, s_g, s_o)
            _check(G, c_g, c_o)
    else:
        _check(G, G.run_forward(shape, I.BF16, wf, wr, x, flags=flags, dir_mask=dir_mask),
               O.bimamba_forward(x, wf, wr, dir_mask=dir_mask, **kw))


@pytest.mark.parametrize("H,L", [(5, 300), (6, 300), (2, 129)])
def test_half_width_heads_single_and_paired(G, H, L):
    """Heads of 32 channels: an even head count puts two neighbouring heads into one CTA of the tensor-core scan (shared B', C' and
    S, one mask and one 32-wide product each), an odd one keeps one head per CTA with half of the tile as padding."""
    shape = I.MixerShape(2, L, 16 * H, 2, 128, 4, H)
    assert shape.headdim == 32
    wf, wr = I.make_mixer_weights(shape, 60 + H, I.BF16, perturb=True)
    x = I.make_activations(shape, 60 + H, I.BF16)
    got = G.run_forward(shape, I.BF16, wf, wr, x, chunk=128)
    _check(G, got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape)))
    # carried state in and out through the same kernel
    blk = I.MixerShape(2, L, 16 * H, 2, 128, 4, H)
    ssm_in, conv_in = I.make_states(blk, 61, I.BF16)
    y, s_out, c_out = G.run_block_step(blk, I.BF16, wf, wr, x, ssm_in, conv_in, chunk=128)
    y_o, s_o, c_o = O.bimamba_block_step(x, wf, wr, ssm_state_in=ssm_in, conv_state_in=conv_in, **G.oracle_kwargs(blk))
    _check(G, y, y_o)
    assert G.rel_l2(s_out, s_o) <= BF16_REL and G.rel_l2(c_out, c_o) <= BF16_REL
