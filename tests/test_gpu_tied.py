"""The weight-tied variant (App. A.1 hyper-parameter "bidirectional weight tie"): both directions share in_proj and out_proj and
keep their own conv / step-size / decay / skip / norm parameters.  The oracle needs no new code for it -- tying is the same
bidirectional mixer called with the shared matrices in both directions' parameter sets -- while the library takes a
different route (one in_proj, the directions' gated outputs summed before one out_proj), so the comparison is a real one."""
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


def _tied(wf, wr):
    return dict(wr, w_in=wf["w_in"], w_out=wf["w_out"])


@pytest.mark.parametrize("dtype,N,H,L,flags", [(I.F32, 16, 4, 70, 7), (I.BF16, 128, 4, 300, 7), (I.BF16, 128, 8, 300, 6), (I.BF16, 128, 4, 32, 7),
                                               (I.BF16, 16, 4, 200, 7)])
def test_tied_projections_against_the_oracle(G, dtype, N, H, L, flags):
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(2, L, 128, 2, N, 4, H)
    wf, wr = I.make_mixer_weights(shape, 40 + L, dtype, perturb=True)
    x = I.make_activations(shape, 40 + L, dtype)
    want = O.bimamba_forward(x, wf, _tied(wf, wr), **G.oracle_kwargs(shape, flags))
    wr_gpu = dict(wr, w_in=None, w_out=None)                      # the second direction's projections are not read
    got = G.run_forward(shape, dtype, wf, wr_gpu, x, flags=flags | dm.DM_FLAG_TIED_PROJ)
    assert np.all(np.isfinite(got))
    if dtype == I.F32:
        assert G.rel_l2(got, want) <= 1e-4
    else:
        assert G.rel_l2(got, want) <= 1e-2 and G.max_abs(got, want) <= 5e-2
    # tying is not a no-op: the untied layer with its own second set of projections gives something else
    assert G.rel_l2(O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape, flags)), want) > 0.1
    # one direction alone (invariant tests use it): the shared projections with that direction's own scan parameters
    for mask, odir in ((1, O.DIR_FWD), (2, O.DIR_REV)):
        one = G.run_forward(shape, dtype, wf, wr_gpu, x, flags=flags | dm.DM_FLAG_TIED_PROJ, dir_mask=mask)
        ref = O.bimamba_forward(x, wf, _tied(wf, wr), dir_mask=odir, **G.oracle_kwargs(shape, flags))
        assert G.rel_l2(one, ref) <= (1e-4 if dtype == I.F32 else 1e-2)


def test_tied_block_step_with_carried_state(G):
    from paper_2511_15927_b200 import binding as dm
    shape, dtype = I.MixerShape(2, 32, 128, 2, 128, 4, 4), I.BF16
    wf, wr = I.make_mixer_weights(shape, 50, dtype, perturb=True)
    x = I.make_activations(shape, 50, dtype)
    ssm_in, conv_in = I.make_states(shape, 50, dtype)
    y_o, s_o, c_o = O.bimamba_block_step(x, wf, _tied(wf, wr), ssm_state_in=ssm_in, conv_state_in=conv_in, **G.oracle_kwargs(shape))
    y, s, c = G.run_block_step(shape, dtype, wf, dict(wr, w_in=None, w_out=None), x, ssm_in, conv_in, flags=dm.DM_FLAGS_DEFAULT | dm.DM_FLAG_TIED_PROJ)
    assert G.rel_l2(y, y_o) <= 1e-2 and G.rel_l2(s, s_o) <= 1e-2 and G.rel_l2(c, c_o) <= 1e-2
