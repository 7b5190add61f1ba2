"""GPU parity of the dense projection (dm_linear) against the oracle's in_proj / out_proj rows: sizes that
span several 128 x 256 tiles with ragged tails in every dimension, the row-scale and addend epilogue, and
in-place accumulation into an fp32 output."""
import numpy as np
import pytest
import torch

from oracle import bimamba_oracle as O
from paper_2511_15927_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dm():
    from paper_2511_15927_b200 import build
    build.build()
    from paper_2511_15927_b200 import binding
    return binding


def _rand(shape, seed, dtype, scale=1.0):
    a = (scale * np.random.default_rng(seed).standard_normal(shape)).astype(np.float32)
    return I.round_to_bf16(a) if dtype == I.BF16 else a


@pytest.mark.parametrize("dtype", [I.BF16, I.F32])
@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (300, 520, 200), (129, 257, 72), (1000, 1288, 256), (2048, 2048, 1024), (77, 100, 64),
                                   (512, 50304 // 16, 128),
                                   # few rows, many columns: two rounds of 128 x 256 tiles or one of 256 x 256 -- the tall tile (ragged rows and columns)
                                   (300, 13000, 192), (512, 17024, 256), (130, 18000, 64)])
def test_linear_parity(dm, dtype, M, N, K):
    from paper_2511_15927_b200.torch_io import dev, dm_dtype, tdtype
    x = _rand((M, K), 1, dtype); w = _rand((N, K), 2, dtype, 0.05)
    xd, wd = dev(x, dtype), dev(w, dtype)
    want = O.in_proj(x, w)
    for y_dtype in ([I.BF16, I.F32] if dtype == I.BF16 else [I.F32]):
        yd = torch.empty((M, N), device="cuda", dtype=tdtype(y_dtype))
        dm.dm_linear(dm_dtype(dtype), xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), dm_dtype(y_dtype), M, K, N, 0, 0,
                     torch.cuda.current_stream().cuda_stream)
        dm.dm_check(0)
        got = yd.float().cpu().numpy().astype(np.float64)
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert rel <= (3e-3 if y_dtype == I.BF16 else 1e-5), rel       # bf16 output rounding alone is ~2e-3
        if y_dtype == I.F32:
            np.testing.assert_allclose(got, want, rtol=0, atol=2e-5 * np.sqrt(K) * 0.05 * 4 + 1e-6)


@pytest.mark.parametrize("dtype", [I.BF16, I.F32])
@pytest.mark.parametrize("shape", [(333, 300, 136), (300, 13000, 136)])
def test_linear_epilogue_scale_addend_inplace(dm, dtype, shape):
    from paper_2511_15927_b200.torch_io import dev, dm_dtype
    M, N, K = shape                                         # the second shape takes the tall tile on the tensor-core path
    x = _rand((M, K), 3, dtype); w = _rand((N, K), 4, dtype, 0.05)
    sc = np.random.default_rng(5).uniform(0.5, 2.0, M).astype(np.float32)
    add = np.random.default_rng(6).standard_normal((M, N)).astype(np.float32)
    xd, wd, scd = dev(x, dtype), dev(w, dtype), dev(sc)
    yd = dev(add.copy())                                    # accumulate in place: y <- sc * (x W^T) + y
    dm.dm_linear(dm_dtype(dtype), xd.data_ptr(), wd.data_ptr(), yd.data_ptr(), dm.DM_F32, M, K, N, scd.data_ptr(), yd.data_ptr(),
                 torch.cuda.current_stream().cuda_stream)
    dm.dm_check(0)
    want = sc[:, None].astype(np.float64) * O.out_proj(x, w) + add
    np.testing.assert_allclose(yd.cpu().numpy().astype(np.float64), want, rtol=1e-5, atol=1e-5)
