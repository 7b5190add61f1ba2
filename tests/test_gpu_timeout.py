"""The failure path of the bounded device-side waits, exercised without faulting or hanging anything: a wait on a barrier that
nothing arrives at runs out after its (short) limit, the device status word receives DM_ERR_TIMEOUT, the CTA's other waiting
role is released through the abort flag, TMEM is freed, and the library stays usable afterwards."""
import numpy as np
import pytest

from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    from paper_2511_15927_b200 import build
    build.build()
    import tests.gpu_util as g
    return g


def test_a_wait_that_runs_out_is_reported_and_the_library_stays_usable(G):
    import torch
    from paper_2511_15927_b200 import binding as dm
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_check(st)                                             # clean slate
    out = torch.zeros(3, device="cuda", dtype=torch.int64)
    dm.dm_selftest_wait_timeout(1000, out.data_ptr(), st)       # 1 ms
    with pytest.raises(dm.DmError) as e:
        dm.dm_check(st)
    assert e.value.status == dm.DM_ERR_TIMEOUT
    gave_up, released, waited_ns = [int(v) for v in out.cpu()]
    assert gave_up == 1 and released == 1
    assert 0.9e6 <= waited_ns < 0.5e9                           # released about when the 1 ms ran out, long before its own 2 s limit
    dm.dm_check(st)                                             # the status is cleared by the read
    # the next call is unaffected (TMEM was given back: the tensor-core GEMM and scan allocate all 512 columns)
    shape = I.MixerShape(2, 300, 256, 2, 128, 4, 8)
    wf, wr = I.make_mixer_weights(shape, 3, I.BF16)
    x = I.make_activations(shape, 3, I.BF16)
    from oracle import bimamba_oracle as O
    got = G.run_forward(shape, I.BF16, wf, wr, x)
    assert G.rel_l2(got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape))) <= 1e-2


def test_the_scan_kernel_leaves_through_its_abort_path_when_its_prep_never_comes(G):
    """The tensor-core scan itself: with the prep role withheld, its load warps wait (bounded, 2 s) for flags nothing raises; the
    whole pipeline -- 28 warps in six roles per CTA -- has to unwind through the abort flag, wait for its loads in flight and free
    its TMEM.  The status comes back as DM_ERR_TIMEOUT, and the same call with the switch off is correct again."""
    import time
    import torch
    from oracle import bimamba_oracle as O
    from paper_2511_15927_b200 import binding as dm
    shape = I.MixerShape(1, 9 * 128 + 5, 128, 2, 128, 4, 4)    # 10 chunks, 8 scan CTAs: the configuration that fuses the prep work
    wf, wr = I.make_mixer_weights(shape, 4, I.BF16)
    x = I.make_activations(shape, 4, I.BF16)
    st = torch.cuda.current_stream().cuda_stream
    dm.dm_check(st)
    dm.dm_selftest_withhold_prep(True)
    try:
        t0 = time.time()
        with pytest.raises(dm.DmError) as e:
            G.run_forward(shape, I.BF16, wf, wr, x, chunk=128)
        waited = time.time() - t0
    finally:
        dm.dm_selftest_withhold_prep(False)
    assert e.value.status == dm.DM_ERR_TIMEOUT
    assert 1.5 < waited < 20.0                                  # the waits' own limit, not a hang
    dm.dm_check(st)
    got = G.run_forward(shape, I.BF16, wf, wr, x, chunk=128)
    assert G.rel_l2(got, O.bimamba_forward(x, wf, wr, **G.oracle_kwargs(shape))) <= 1e-2


def test_selftest_argument_checks(G):
    from paper_2511_15927_b200 import binding as dm
    before = dm.dm_kernel_launch_count()
    for limit, out in ((0, 4096), (2_000_000, 4096), (1000, 0)):
        with pytest.raises(dm.DmError):
            dm.dm_selftest_wait_timeout(limit, out, 0)
    assert dm.dm_kernel_launch_count() == before
