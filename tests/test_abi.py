"""The C-ABI library loads, exports every symbol the public header declares, and rejects bad arguments
before touching the GPU (none of these calls launches anything)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dm():
    from paper_2511_15927_b200 import build
    build.build()
    from paper_2511_15927_b200 import binding
    return binding


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if not fn.endswith(".h"):
            continue
        text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, fn)).read(), flags=re.S)
        names.update(re.findall(r"\b(dm_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported_and_bound(dm):
    declared = _declared_functions()
    assert {"dm_bimamba_forward", "dm_bimamba_block_step", "dm_denoise_step"} <= declared
    lib = C.CDLL(dm.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"
        assert hasattr(dm, name), f"{name} has no Python binding of the same name"
    assert set(dm.EXPORTS) == declared


def test_status_strings(dm):
    assert dm.dm_status_string(0) == "ok"
    texts = {dm.dm_status_string(s) for s in range(-5, 1)}
    assert len(texts) == 6 and "unknown status" not in texts
    assert dm.dm_status_string(-99) == "unknown status"


def _cfg(dm, **kw):
    base = dict(batch=1, seqlen=256, d_model=128, expand=2, d_state=16, d_conv=4, n_heads=8, dtype=dm.DM_F32)
    base.update(kw)
    return dm.make_mixer_cfg(**base)


def test_workspace_query_and_shape_checks(dm):
    n = dm.dm_bimamba_workspace_bytes(_cfg(dm))
    # zx 2*256*552*4 + g 2*256*256*4 + ssq 2*256*8*4 + rstd 2*256*4 + ytmp 256*128*4, each rounded up to 256 bytes
    assert n >= 2 * 256 * 552 * 4 + 2 * 256 * 256 * 4 + 2 * 256 * 8 * 4 + 2 * 256 * 4 + 256 * 128 * 4
    assert n % 256 == 0
    assert dm.dm_bimamba_workspace_bytes(_cfg(dm, seqlen=512)) > n
    for bad, status in [(dict(batch=0), dm.DM_ERR_INVALID_ARG), (dict(seqlen=-3), dm.DM_ERR_INVALID_ARG),
                        (dict(n_heads=7), dm.DM_ERR_INVALID_ARG), (dict(dtype=5), dm.DM_ERR_INVALID_ARG),
                        (dict(dir_mask=0), dm.DM_ERR_INVALID_ARG), (dict(flags=64), dm.DM_ERR_INVALID_ARG),
                        (dict(n_groups=2), dm.DM_ERR_UNSUPPORTED), (dict(d_conv=7), dm.DM_ERR_UNSUPPORTED),
                        (dict(d_state=24), dm.DM_ERR_UNSUPPORTED), (dict(n_heads=2), dm.DM_ERR_UNSUPPORTED)]:
        with pytest.raises(dm.DmError) as e:
            dm.dm_bimamba_workspace_bytes(_cfg(dm, **bad))
        assert e.value.status == status, bad
        assert dm.dm_last_error_message()


def test_calls_reject_bad_arguments_before_any_launch(dm):
    cfg = _cfg(dm)
    before = dm.dm_kernel_launch_count()
    w = (dm.dm_dir_weights(), dm.dm_dir_weights())
    with pytest.raises(dm.DmError) as e:
        dm.dm_bimamba_forward(cfg, w, 0, 0, 0, 0)
    assert e.value.status == dm.DM_ERR_INVALID_ARG
    fake = dm.dm_dir_weights(*([4096] * 8))
    with pytest.raises(dm.DmError) as e:                      # x == y
        dm.dm_bimamba_forward(cfg, (fake, fake), 4096, 4096, 4096, 1 << 30)
    assert e.value.status == dm.DM_ERR_INVALID_ARG
    with pytest.raises(dm.DmError) as e:                      # workspace too small
        dm.dm_bimamba_forward(cfg, (fake, fake), 4096, 8192, 4096, 1024)
    assert e.value.status == dm.DM_ERR_WORKSPACE and "too small" in str(e.value)
    with pytest.raises(dm.DmError) as e:                      # workspace misaligned
        dm.dm_bimamba_forward(cfg, (fake, fake), 4096, 8192, 4096 + 16, 1 << 30)
    assert e.value.status == dm.DM_ERR_WORKSPACE
    with pytest.raises(dm.DmError) as e:                      # misaligned x
        dm.dm_bimamba_forward(cfg, (fake, fake), 4100, 8192, 4096, 1 << 30)
    assert e.value.status == dm.DM_ERR_INVALID_ARG
    with pytest.raises(dm.DmError) as e:                      # state in == state out
        dm.dm_bimamba_block_step(cfg, (fake, fake), 4096, 8192, 0, 8192, 0, 12288, 4096, 1 << 30)
    assert e.value.status == dm.DM_ERR_INVALID_ARG
    scfg = dm.dm_stack_cfg(cfg, 2, 1000, 1e-5)
    assert dm.dm_denoise_workspace_bytes(scfg) > dm.dm_bimamba_workspace_bytes(cfg)
    with pytest.raises(dm.DmError) as e:
        dm.dm_denoise_step(scfg, dm.dm_stack_weights(), 4096, 0, 0, None, 4096, 1 << 30)
    assert e.value.status == dm.DM_ERR_INVALID_ARG
    assert dm.dm_kernel_launch_count() == before
