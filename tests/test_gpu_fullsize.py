"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (dm_bimamba_forward, bf16,
d_model 2048, 64 heads x 64, d_state 128): batch rows of the B=8 / L=2048 workload and the whole L=8192 sequence
against the CPU oracle, the left-to-right layer over the whole L=16384 sequence, and at L=32768 -- where the oracle would take
minutes -- a property that holds at any
length: the left-to-right layer's outputs on a prefix do not depend on what follows it, and the right-to-left
layer's outputs on a suffix do not depend on what precedes it."""
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


def _check_rows(G, got, x, wf, wr, shape, rows):
    kw = G.oracle_kwargs(shape)
    for b in rows:
        want = O.bimamba_forward(x[b:b + 1], wf, wr, **kw)[0]
        assert np.all(np.isfinite(got[b]))
        assert G.rel_l2(got[b], want) <= BF16_REL, (b, G.rel_l2(got[b], want))
        assert G.max_abs(got[b], want) <= BF16_ABS, (b, G.max_abs(got[b], want))


def test_cfg1_sampled_batch_rows_against_the_oracle(G):
    shape, dtype = I.CONFIGS["cfg1"]
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    got = G.run_forward(shape, dtype, wf, wr, x)
    _check_rows(G, got, x, wf, wr, shape, rows=(0, 5))


def test_cfg3_8k_whole_sequence_against_the_oracle(G):
    shape, dtype = I.CONFIGS["cfg3_8k"]
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    got = G.run_forward(shape, dtype, wf, wr, x)
    _check_rows(G, got, x, wf, wr, shape, rows=(0,))


def test_cfg3_16k_left_to_right_layer_against_the_oracle(G):
    """The middle length of the scan-scaling sweep, element by element against the oracle: the whole 16 384-token sequence through
    the left-to-right layer alone (one direction keeps the oracle's token loop under half a minute; the right-to-left layer
    runs the same kernel with mirrored indices and is compared at 8192 above)."""
    shape, dtype = I.CONFIGS["cfg3_16k"]
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    got = G.run_forward(shape, dtype, wf, wr, x, dir_mask=1)
    want = O.bimamba_forward(x, wf, wr, dir_mask=O.DIR_FWD, **G.oracle_kwargs(shape))
    assert np.all(np.isfinite(got))
    assert G.rel_l2(got, want) <= BF16_REL, G.rel_l2(got, want)
    assert G.max_abs(got, want) <= BF16_ABS, G.max_abs(got, want)
    # the last 2048 tokens on their own: errors do not grow along the sequence
    assert G.rel_l2(got[:, -2048:], want[:, -2048:]) <= BF16_REL


def test_cfg3_32k_prefix_and_suffix_independence(G):
    shape, dtype = I.CONFIGS["cfg3_32k"]
    part = I.MixerShape(1, 8192, shape.d_model, shape.expand, shape.d_state, shape.d_conv, shape.n_heads)
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    fwd_full = G.run_forward(shape, dtype, wf, wr, x, dir_mask=1)
    fwd_part = G.run_forward(part, dtype, wf, wr, np.ascontiguousarray(x[:, :8192]), dir_mask=1)
    rev_full = G.run_forward(shape, dtype, wf, wr, x, dir_mask=2)
    rev_part = G.run_forward(part, dtype, wf, wr, np.ascontiguousarray(x[:, -8192:]), dir_mask=2)
    assert np.all(np.isfinite(fwd_full)) and np.all(np.isfinite(rev_full))
    # 8192 is a multiple of the 128-token chunk, so both runs do the same arithmetic on these rows
    np.testing.assert_array_equal(fwd_full[:, :8192], fwd_part)
    np.testing.assert_array_equal(rev_full[:, -8192:], rev_part)
    # and the two directions add up
    both = G.run_forward(shape, dtype, wf, wr, x)
    assert G.rel_l2(both, fwd_full + rev_full) <= 5e-3


def test_cfg2_layer_sampled_row_against_the_oracle(G):
    """d_state 16 (zero-padded to 128 on the tensor-core scan) at B=4, L=4096, d_model 1024."""
    shape, dtype = I.CONFIGS["cfg2_layer"]
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    got = G.run_forward(shape, dtype, wf, wr, x)
    _check_rows(G, got, x, wf, wr, shape, rows=(2,))


def test_cfg4_block_step_sampled_rows_against_the_oracle(G):
    """Block decoding at B=16, G=32, d_model 2048 from a carried state: outputs and the committed state of two rows."""
    shape, dtype = I.CONFIGS["cfg4_block"]
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    ssm_in, conv_in = I.make_states(shape, 0, dtype)
    y, ssm_out, conv_out = G.run_block_step(shape, dtype, wf, wr, x, ssm_in, conv_in)
    kw = G.oracle_kwargs(shape)
    for b in (0, 11):
        y_o, s_o, c_o = O.bimamba_block_step(x[b:b + 1], wf, wr, ssm_state_in=ssm_in[b:b + 1], conv_state_in=conv_in[b:b + 1], **kw)
        assert G.rel_l2(y[b], y_o[0]) <= BF16_REL and G.max_abs(y[b], y_o[0]) <= BF16_ABS, (b, G.rel_l2(y[b], y_o[0]))
        assert G.rel_l2(ssm_out[b], s_o[0]) <= BF16_REL, (b, G.rel_l2(ssm_out[b], s_o[0]))
        assert G.rel_l2(conv_out[b], c_o[0]) <= BF16_REL, (b, G.rel_l2(conv_out[b], c_o[0]))      # the block's last pre-conv rows, stored in bf16


def test_paper_shape_whole_sequence_against_the_oracle(G):
    """The paper's 1.3B mixer shape (App. A.1 / App. C: d = 1920, 120 heads of 32, d_state 128) at L = 1024: heads of 32
    channels on the tensor-core scan, every head against the oracle, the last one (whose tile reaches past the x columns)
    included."""
    shape, dtype = I.CONFIGS["paper_1p3b"]
    assert shape.headdim == 32 and shape.n_heads == 120
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    got = G.run_forward(shape, dtype, wf, wr, x)
    _check_rows(G, got, x, wf, wr, shape, rows=(0,))


def test_cfg3_64k_runs_and_is_deterministic(G):
    """The longest context of the paper's throughput sweep (Sec. 4.3): finite, run-to-run bit-identical, and the
    left-to-right layer's first 1024 outputs equal those of the 1024-token call (prefix independence at full length)."""
    shape, dtype = I.CONFIGS["cfg3_64k"]
    wf, wr = I.make_mixer_weights(shape, 0, dtype)
    x = I.make_activations(shape, 0, dtype)
    a = G.run_forward(shape, dtype, wf, wr, x, dir_mask=1)
    assert np.all(np.isfinite(a))
    np.testing.assert_array_equal(a, G.run_forward(shape, dtype, wf, wr, x, dir_mask=1))
    short = I.MixerShape(1, 1024, shape.d_model, shape.expand, shape.d_state, shape.d_conv, shape.n_heads)
    np.testing.assert_array_equal(a[:, :1024], G.run_forward(short, dtype, wf, wr, np.ascontiguousarray(x[:, :1024]), dir_mask=1))
