"""The seeded input generators: determinism, stream independence, bf16 rounding, value ranges."""
import numpy as np

from paper_2511_15927_b200 import inputs as I


def test_streams_are_deterministic_and_independent():
    s = I.MixerShape(2, 16, 32, 2, 16, 4, 4)
    a = I.make_mixer_weights(s, seed=3)
    b = I.make_mixer_weights(s, seed=3)
    for k in a[0]:
        np.testing.assert_array_equal(a[0][k], b[0][k])
        assert a[0][k].dtype == np.float32
    assert not np.array_equal(a[0]["w_in"], a[1]["w_in"])              # untied directions
    assert not np.array_equal(a[0]["w_in"], I.make_mixer_weights(s, seed=4)[0]["w_in"])
    assert a[0]["w_in"].shape == (s.d_in_proj, s.d_model) and a[0]["w_out"].shape == (s.d_model, s.d_inner)
    assert a[0]["conv_w"].shape == (s.conv_ch, 4) and s.conv_ch == 64 + 32 and s.d_in_proj == 128 + 32 + 4


def test_value_ranges_follow_the_recipe():
    s = I.MixerShape(1, 8, 256, 2, 16, 4, 64)
    w = I.make_dir_weights(s, seed=0)
    assert np.all((np.exp(w["A_log"]) >= 1.0) & (np.exp(w["A_log"]) <= 16.0))
    dt = np.log1p(np.exp(w["dt_bias"].astype(np.float64)))
    assert np.all((dt > 0.999e-3) & (dt < 1.001e-1))
    assert abs(float(np.std(w["w_in"])) - 0.02) < 1e-3
    assert np.all(np.abs(w["conv_w"]) <= 0.5)
    x = I.make_activations(s, seed=0)
    assert abs(float(np.std(x)) - 1.0) < 0.05


def test_bf16_rounding_is_nearest_even_and_idempotent():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -3.14159, 1e-30, 65504.0], np.float32)
    r = I.round_to_bf16(v)
    np.testing.assert_array_equal(r[:4], np.array([1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6], np.float32))  # ties to even
    np.testing.assert_array_equal(I.round_to_bf16(r), r)
    assert np.all(np.abs(r - v) <= np.abs(v) * 2.0 ** -8)
    import torch
    t = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(r, t)
    np.testing.assert_array_equal(I.bf16_bits(v), torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def test_tokens_masking():
    tok = I.make_tokens(4, 512, 50257, 50257, seed=0)
    assert tok.dtype == np.int32 and tok.min() >= 0 and tok.max() <= 50257
    frac = (tok == 50257).mean(axis=1)
    assert np.all(frac >= 0) and len(set(np.round(frac, 2))) > 1        # one masking level per row
