"""dm_bimamba_forward_static: the mixer for callers that cannot give the library device memory (no
cudaMalloc allowed where they run, or all memory already handed to their own pool).  It keeps its
intermediates in a fixed array inside the library instead of a caller workspace.

Checked here through the C ABI: two calls in a row (different inputs, so that anything left behind by the
first call would show in the second) must equal dm_bimamba_forward on the same inputs bit for bit -- both run
the same kernels in the same order, only the scratch address differs, so even a partly overlapping or
misplaced scratch region would show -- and stay inside the tolerance of the other parity tests; the second
call must leave the device's free memory unchanged (it allocates nothing); and a configuration too large for
the built-in array must be refused before any kernel is launched.  This file sorts last so that a run stopping at the first failure has already
run every other test; it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu
BF16_REL, BF16_ABS = 1e-2, 5e-2


@pytest.fixture(scope="module")
def G():
    from paper_2511_15927_b200 import build
    build.build()
    import tests.gpu_util as g
    return g


def _static_forward(G, shape, dtype, wf, wr, x):
    import torch
    from paper_2511_15927_b200 import binding as dm
    cfg = G.cfg_of(shape, dtype)
    dwf, dwr = G.dev_dir_weights(wf, dtype), G.dev_dir_weights(wr, dtype)
    xd = G.dev(x, dtype)
    yd = torch.full_like(xd, float("nan"))
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_bimamba_forward_static(cfg, (dm.make_dir_weights(dwf), dm.make_dir_weights(dwr)), xd.data_ptr(), yd.data_ptr(), st)
    dm.dm_check(st)
    return yd.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("dtype,N,H", [(I.BF16, 128, 8), (I.F32, 16, 16)])
def test_two_calls_match_the_workspace_entry_point(G, dtype, N, H):
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(2, 300, 256, 2, N, 4, H)
    assert dm.dm_bimamba_workspace_bytes(G.cfg_of(shape, dtype)) <= dm.DM_STATIC_WORKSPACE_BYTES
    wf, wr = I.make_mixer_weights(shape, 21, dtype, perturb=True)
    for seed in (21, 22):                                   # second call: new input over the first call's leftovers
        x = I.make_activations(shape, seed, dtype)
        want = G.run_forward(shape, dtype, wf, wr, x)
        got = _static_forward(G, shape, dtype, wf, wr, x)
        assert np.all(np.isfinite(got))
        assert G.rel_l2(got, want) <= (BF16_REL if dtype == I.BF16 else 1e-4), G.rel_l2(got, want)
        assert G.max_abs(got, want) <= BF16_ABS, G.max_abs(got, want)
        np.testing.assert_array_equal(got, want)            # same kernels, same inputs: identical bits


def test_second_call_allocates_nothing(G):
    """Device memory in use does not move across a call (after a first call has looked the array's address up)."""
    import torch
    from paper_2511_15927_b200 import binding as dm
    shape, dtype = I.MixerShape(2, 300, 256, 2, 128, 4, 8), I.BF16
    wf, wr = I.make_mixer_weights(shape, 23, dtype)
    cfg = G.cfg_of(shape, dtype)
    dwf, dwr = G.dev_dir_weights(wf, dtype), G.dev_dir_weights(wr, dtype)
    xd = G.dev(I.make_activations(shape, 23, dtype), dtype)
    yd = torch.empty_like(xd)
    st = torch.cuda.current_stream().cuda_stream
    cw = (dm.make_dir_weights(dwf), dm.make_dir_weights(dwr))
    dm.dm_bimamba_forward_static(cfg, cw, xd.data_ptr(), yd.data_ptr(), st)
    dm.dm_check(st)
    free0, _ = torch.cuda.mem_get_info()
    dm.dm_bimamba_forward_static(cfg, cw, xd.data_ptr(), yd.data_ptr(), st)
    dm.dm_check(st)
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)


def test_oversized_configuration_is_refused_without_a_launch(G):
    from paper_2511_15927_b200 import binding as dm
    shape, dtype = I.CONFIGS["cfg1"]
    cfg = G.cfg_of(shape, dtype)
    assert dm.dm_bimamba_workspace_bytes(cfg) > dm.DM_STATIC_WORKSPACE_BYTES
    fake = dm.dm_dir_weights(*([4096] * 8))
    before = dm.dm_kernel_launch_count()
    with pytest.raises(dm.DmError) as e:
        dm.dm_bimamba_forward_static(cfg, (fake, fake), 4096, 8192, 0)
    assert e.value.status == dm.DM_ERR_WORKSPACE and "built-in array" in str(e.value)
    assert dm.dm_kernel_launch_count() == before
