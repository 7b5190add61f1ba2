"""GPU parity of dm_bimamba_forward / dm_bimamba_block_step against the CPU oracle, through the C ABI.

Tolerances: fp32 I/O rel-L2 <= 1e-4 (fp32 products and sums in another order than the oracle's fp64); bf16 I/O with fp32 accumulation
rel-L2 <= 1e-2 and max-abs <= 5e-2; index work (state placement, carried conv rows) bit-exact.
"""
import numpy as np
import pytest

from oracle import bimamba_oracle as O
from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu

F32_REL = 1e-4
BF16_REL, BF16_ABS = 1e-2, 5e-2


@pytest.fixture(scope="module")
def G():
    from paper_2511_15927_b200 import build
    build.build()
    import tests.gpu_util as g
    return g


def _case(shape, dtype, seed=0, perturb=True):
    wf, wr = I.make_mixer_weights(shape, seed, dtype, perturb)
    x = I.make_activations(shape, seed, dtype)
    return wf, wr, x


def _check(got, want, dtype):
    from tests.gpu_util import max_abs, rel_l2
    assert np.all(np.isfinite(got))
    if dtype == I.F32:
        assert rel_l2(got, want) <= F32_REL, rel_l2(got, want)
    else:
        assert rel_l2(got, want) <= BF16_REL, rel_l2(got, want)
        assert max_abs(got, want) <= BF16_ABS, max_abs(got, want)


@pytest.mark.parametrize("flags", [7, 6, 1, 0])
def test_cfg0_fp32_parity(G, flags):
    shape, dtype = I.CONFIGS["cfg0"]
    wf, wr, x = _case(shape, dtype, seed=0, perturb=(flags != 7))
    got = G.run_forward(shape, dtype, wf, wr, x, flags=flags)
    want = O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape, flags))
    _check(got, want, dtype)


@pytest.mark.parametrize("L", [1, 2, 3, 5, 31, 33, 255, 257])
def test_ragged_lengths_fp32(G, L):
    shape = I.MixerShape(2, L, 64, 2, 16, 4, 4)
    wf, wr, x = _case(shape, I.F32, seed=L)
    got = G.run_forward(shape, I.F32, wf, wr, x)
    _check(got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape)), I.F32)


@pytest.mark.parametrize("dims", [(64, 2, 128, 4, 2), (96, 2, 64, 3, 6), (128, 1, 32, 2, 2), (64, 4, 256, 4, 4)])
def test_other_state_sizes_fp32(G, dims):
    d, expand, N, k, H = dims
    shape = I.MixerShape(2, 70, d, expand, N, k, H)
    wf, wr, x = _case(shape, I.F32, seed=11)
    got = G.run_forward(shape, I.F32, wf, wr, x)
    _check(got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape)), I.F32)


@pytest.mark.parametrize("dims", [(256, 128, 8, 300), (256, 16, 8, 260), (192, 128, 12, 130)])
def test_bf16_parity_small(G, dims):
    d, N, H, L = dims
    shape = I.MixerShape(2, L, d, 2, N, 4, H)
    wf, wr, x = _case(shape, I.BF16, seed=3)
    got = G.run_forward(shape, I.BF16, wf, wr, x)
    _check(got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape)), I.BF16)


@pytest.mark.parametrize("B,L,d,H", [(1, 1500, 1024, 32), (3, 400, 512, 16), (2, 60, 256, 8)])
def test_short_input_out_proj_paths_bf16(G, B, L, d, H):
    """Up to 2048 tokens the two out_proj run as one launch into fp32 partials that one pass scales and sums: 1500 tokens at d_model 1024
    fill the GPU with whole products (256 tiles), the two smaller cases cut each product in two along K (four partials)."""
    shape = I.MixerShape(B, L, d, 2, 128, 4, H)
    wf, wr, x = _case(shape, I.BF16, seed=9)
    got = G.run_forward(shape, I.BF16, wf, wr, x)
    _check(got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape)), I.BF16)
    # without the gated norm the partials are summed unscaled
    got0 = G.run_forward(shape, I.BF16, wf, wr, x, flags=dm_flags_no_norm())
    _check(got0, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape, flags=dm_flags_no_norm())), I.BF16)


def dm_flags_no_norm():
    from paper_2511_15927_b200 import binding as dm
    return dm.DM_FLAGS_DEFAULT & ~dm.DM_FLAG_GATED_RMSNORM


def test_direction_masks_and_reversal_invariant(G):
    shape = I.MixerShape(2, 77, 64, 2, 16, 4, 4)
    wf, wr, x = _case(shape, I.F32, seed=5)
    kw = G.oracle_kwargs(shape)
    f = G.run_forward(shape, I.F32, wf, wr, x, dir_mask=1)
    r = G.run_forward(shape, I.F32, wf, wr, x, dir_mask=2)
    both = G.run_forward(shape, I.F32, wf, wr, x, dir_mask=3)
    _check(f, O.bimamba_forward(x, wf, wr, dir_mask=O.DIR_FWD, **kw), I.F32)
    _check(r, O.bimamba_forward(x, wf, wr, dir_mask=O.DIR_REV, **kw), I.F32)
    np.testing.assert_allclose(both, f + r, rtol=1e-4, atol=1e-5)
    # the reverse layer with weights W on u equals flip(forward layer with W on flip(u))
    xf = np.ascontiguousarray(x[:, ::-1])
    f_on_flipped = G.run_forward(shape, I.F32, wr, wr, xf, dir_mask=1)
    np.testing.assert_allclose(r, f_on_flipped[:, ::-1], rtol=1e-5, atol=1e-6)


def test_causality_on_gpu(G):
    shape = I.MixerShape(1, 90, 64, 2, 16, 4, 4)
    wf, wr, x = _case(shape, I.F32, seed=6)
    x2 = x.copy(); x2[0, 40] += 1.0
    df = G.run_forward(shape, I.F32, wf, wr, x2, dir_mask=1) - G.run_forward(shape, I.F32, wf, wr, x, dir_mask=1)
    dr = G.run_forward(shape, I.F32, wf, wr, x2, dir_mask=2) - G.run_forward(shape, I.F32, wf, wr, x, dir_mask=2)
    assert np.all(df[0, :40] == 0) and np.any(df[0, 40:] != 0)
    assert np.all(dr[0, 41:] == 0) and np.any(dr[0, :41] != 0)


def test_chunk_size_invariance_fp32(G):
    """Sequential (exact) kernel: any chunk length gives the same result up to fp32 rounding order."""
    shape = I.MixerShape(1, 300, 128, 2, 16, 4, 4)
    wf, wr, x = _case(shape, I.F32, seed=7)
    want = O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape))
    outs = [G.run_forward(shape, I.F32, wf, wr, x, chunk=c) for c in (32, 64, 128, 256)]
    for o in outs:
        _check(o, want, I.F32)
        np.testing.assert_allclose(o, outs[0], rtol=1e-4, atol=1e-5)


@pytest.mark.parametrize("L", [300, 127, 128, 129, 257, 40])
@pytest.mark.parametrize("P", [64, 32])
def test_chunk_size_invariance_bf16(G, L, P):
    """Chunked bf16 path: chunk = 128 is the tensor-core kernel, chunk = 32 the CUDA-core kernel with a quarter of the
    chunk length (a different kernel with its own arithmetic: fp32 products, state in registers).  Both must match the
    oracle and each other on lengths around the chunk boundaries; other chunk values are refused."""
    from paper_2511_15927_b200 import binding as dm
    H = 4 if P == 64 else 8
    shape = I.MixerShape(2, L, 128, 2, 128, 4, H)
    wf, wr, x = _case(shape, I.BF16, seed=7 + L)
    want = O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape))
    o32 = G.run_forward(shape, I.BF16, wf, wr, x, chunk=32)
    o128 = G.run_forward(shape, I.BF16, wf, wr, x, chunk=128)
    _check(o32, want, I.BF16)
    _check(o128, want, I.BF16)
    assert G.rel_l2(o32, o128) <= BF16_REL and G.max_abs(o32, o128) <= BF16_ABS
    assert not np.array_equal(o32, o128)                      # two kernels, not one launched twice
    for bad in (64, 256, 16):
        with pytest.raises(dm.DmError) as e:
            G.run_forward(shape, I.BF16, wf, wr, x, chunk=bad)
        assert e.value.status == dm.DM_ERR_UNSUPPORTED


def test_run_to_run_determinism(G):
    shape = I.MixerShape(2, 200, 128, 2, 128, 4, 4)
    wf, wr, x = _case(shape, I.BF16, seed=8)
    a = G.run_forward(shape, I.BF16, wf, wr, x)
    b = G.run_forward(shape, I.BF16, wf, wr, x)
    np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("dtype,N,d,H", [(I.F32, 16, 64, 4), (I.BF16, 128, 128, 4)])
def test_block_step_parity_and_state_carry(G, dtype, N, d, H):
    full = I.MixerShape(2, 75, d, 2, N, 4, H)
    wf, wr, x = _case(full, dtype, seed=9)
    kw = G.oracle_kwargs(full)
    cuts = [(0, 32), (32, 33), (33, 35), (35, 75)]           # blocks of 32, 1, 2 and 40 tokens
    ssm_o = conv_o = ssm_g = conv_g = None
    for lo, hi in cuts:
        blk = I.MixerShape(2, hi - lo, d, 2, N, 4, H)
        xb = np.ascontiguousarray(x[:, lo:hi])
        # the oracle's incoming state, rounded to the storage types the library takes it in
        ssm_in = None if ssm_o is None else ssm_o.astype(np.float32)
        conv_in_typed = None if conv_o is None else (I.round_to_bf16(conv_o.astype(np.float32)) if dtype == I.BF16 else conv_o.astype(np.float32))
        y_o, ssm_o_new, conv_o_new = O.bimamba_block_step(xb, wf, wr, ssm_state_in=ssm_in, conv_state_in=conv_in_typed, **kw)
        y_g, ssm_g, conv_g = G.run_block_step(blk, dtype, wf, wr, xb, ssm_in, conv_in_typed)
        _check(y_g, y_o, dtype)
        _check(ssm_g, ssm_o_new, dtype)
        _check(conv_g, conv_o_new, dtype)
        if conv_in_typed is not None and hi - lo < 3:          # carried rows are moved, not recomputed: exact
            keep = 3 - (hi - lo)
            np.testing.assert_array_equal(conv_g[:, :keep], conv_in_typed[:, hi - lo:].astype(np.float64))
        ssm_o, conv_o = ssm_o_new, conv_o_new


def test_block_chain_equals_full_pass_on_gpu_and_snapshot_restore(G):
    """Left-to-right direction: block-by-block with the carried state == one pass over the prefix; a state
    copied to the host and back continues bit-identically."""
    d, N, H = 64, 16, 4
    full = I.MixerShape(1, 64, d, 2, N, 4, H)
    wf, wr, x = _case(full, I.F32, seed=10)
    whole = G.run_forward(full, I.F32, wf, wr, x, dir_mask=1)
    y_full, ssm_full, conv_full = G.run_block_step(full, I.F32, wf, wr, x, dir_mask=1)
    np.testing.assert_array_equal(y_full, whole)
    outs, ssm, conv = [], None, None
    for lo in range(0, 64, 16):
        blk = I.MixerShape(1, 16, d, 2, N, 4, H)
        y, ssm, conv = G.run_block_step(blk, I.F32, wf, wr, np.ascontiguousarray(x[:, lo:lo + 16]), ssm, conv, dir_mask=1)
        ssm = ssm.astype(np.float32).astype(np.float64)       # host round trip
        outs.append(y)
    np.testing.assert_allclose(np.concatenate(outs, axis=1), whole, rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(ssm, ssm_full, rtol=1e-4, atol=1e-7)
    np.testing.assert_array_equal(conv, conv_full)
    # reverse direction in block mode ignores the carried state
    blk = I.MixerShape(1, 16, d, 2, N, 4, H)
    xb = np.ascontiguousarray(x[:, 16:32])
    r1, _, _ = G.run_block_step(blk, I.F32, wf, wr, xb, ssm_full.astype(np.float32), conv_full, want_state=False, dir_mask=2)
    r2 = G.run_forward(blk, I.F32, wf, wr, xb, dir_mask=2)
    np.testing.assert_array_equal(r1, r2)


def test_unsupported_and_error_paths_do_not_launch(G):
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(1, 8, 64, 2, 16, 4, 4)
    cfg = G.cfg_of(shape, I.F32)
    before = dm.dm_kernel_launch_count()
    with pytest.raises(dm.DmError):
        dm.dm_bimamba_forward(cfg, (dm.dm_dir_weights(), dm.dm_dir_weights()), 0, 0, 0, 0)
    assert dm.dm_kernel_launch_count() == before
    dm.dm_check(0)


@pytest.mark.parametrize("B,pinned", [(1, True), (5, True), (20, True), (3, False)])
def test_host_buffer_entry_equals_device_entry(G, B, pinned):
    """The host-buffer call cuts the batch into pieces of whole rows and overlaps their copies with the compute;
    rows are independent, so its result is the device call's, bit for bit (uneven last piece included)."""
    shape = I.MixerShape(B, 2100, 128, 2, 128, 4, 4)          # pieces of 2 rows (3 rows at B = 20), the last one shorter
    wf, wr, x = _case(shape, I.BF16, seed=30 + B)
    want = G.run_forward(shape, I.BF16, wf, wr, x)
    for _ in range(2):                                        # second call reuses the library's copy streams
        np.testing.assert_array_equal(G.run_forward_host(shape, I.BF16, wf, wr, x, pinned), want)
