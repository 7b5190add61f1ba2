"""Pins for the CPU oracle: each test ties a piece of it to something other than itself --
the paper's printed numbers, an explicitly materialised sum, a closed form, a textbook routine,
a structural invariant -- so that a dropped term, a wrong sign or index or a transposed operand
fails at least one of them."""
import os

import numpy as np
import pytest
from scipy import signal, special

from oracle import bimamba_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


# ------------------------------------------------------------------ printed numbers (App. C)

def test_shapes_and_flops_match_printed_table():
    g = _golden("appC_mamba_layer_flops.txt")
    dd = O.derived_dims(1920, 2, 128, 120, 1)
    assert dd["d_in_proj"] == g["d_in_proj"] and dd["conv_ch"] == g["conv_ch"]
    assert dd["d_inner"] == 3840 and dd["headdim"] == 32
    fl = O.flops_per_token(1920, 2, 128, 4, 120, 1, d_ff=3840, d_c=128)
    for key, name in [("in_proj", "in_proj_M"), ("scan", "scan_M"), ("out_proj", "out_proj_M"),
                      ("one_direction", "one_direction_M"), ("mixer", "mixer_M"), ("mlp", "mlp_M"),
                      ("adaln", "adaln_M"), ("layer", "layer_M")]:
        assert round(fl[key] / 1e6, 2) == pytest.approx(g[name], abs=0.0101), key
    assert round(fl["conv"] / 1e6, 3) == g["conv_M"]
    model = 24 * fl["layer"] + g["shared_head_M"] * 1e6
    assert round(model / 1e9, 3) == pytest.approx(g["model_G"], abs=0.0011)


def test_param_count_needs_two_untied_directions():
    g = _golden("appC_mamba_layer_flops.txt")
    n = O.param_count(1920, 2, 128, 4, 120, 24, 50258)
    assert abs(n / 1e6 - g["params_M"]) < 0.001 * g["params_M"]     # the paper prints 4 digits
    # a tied (single in/out projection) layer would be far off
    dd = O.derived_dims(1920, 2, 128, 120)
    tied = n - 24 * (1920 * dd["d_in_proj"] + dd["d_inner"] * 1920)
    assert abs(tied / 1e6 - g["params_M"]) > 400


# ------------------------------------------------------------------ scalar functions

def test_softplus_and_silu_against_library():
    v = np.concatenate([np.linspace(-40, 40, 401), [-745.0, 0.0, 700.0]])
    np.testing.assert_allclose(O.softplus(v), np.logaddexp(0.0, v), rtol=1e-14, atol=0)
    np.testing.assert_allclose(O.silu(v), v * special.expit(v), rtol=1e-14, atol=1e-300)
    assert O.softplus(-745.0) > 0 and O.softplus(700.0) == 700.0


def test_discretise_values():
    delta, a = O.discretise(np.array([[0.0, 3.0]]), np.array([0.0, -3.0]), np.log(np.array([2.0, 5.0])))
    np.testing.assert_allclose(delta, [[np.log(2.0), np.log(2.0)]], rtol=1e-15)
    np.testing.assert_allclose(a, [[2.0 ** -2.0, 2.0 ** -5.0]], rtol=1e-14)      # exp(-A*ln2) = 2^-A
    assert np.all((a > 0) & (a < 1))


# ------------------------------------------------------------------ conv

def test_conv_impulse_returns_taps_in_order():
    k, ch, L = 4, 3, 9
    w = rng.standard_normal((ch, k))
    x = np.zeros((L, ch)); x[2] = 1.0
    out, _ = O.causal_conv_silu(x, w, None)
    pre = np.zeros((L, ch))
    for j in range(k):                       # an impulse at row 2 shows tap k-1 at row 2, tap k-2 at row 3, ...
        pre[2 + j] = w[:, k - 1 - j]
    np.testing.assert_allclose(out, O.silu(pre), rtol=1e-14, atol=1e-15)


def test_conv_equals_textbook_fir_filter():
    k, ch, L = 4, 5, 37
    w = rng.standard_normal((ch, k)); b = rng.standard_normal(ch)
    x = rng.standard_normal((L, ch))
    out, state = O.causal_conv_silu(x, w, b)
    for c in range(ch):
        fir = signal.lfilter(w[c, ::-1], [1.0], x[:, c]) + b[c]      # y[t] = sum_m w[k-1-m] x[t-m]
        np.testing.assert_allclose(out[:, c], fir * special.expit(fir), rtol=1e-12, atol=1e-13)
        full = np.correlate(np.concatenate([np.zeros(k - 1), x[:, c]]), w[c], mode="valid") + b[c]
        np.testing.assert_allclose(out[:, c], full * special.expit(full), rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(state, x[-(k - 1):])


def test_conv_state_carry_and_short_blocks():
    k, ch = 4, 6
    w = rng.standard_normal((ch, k)); b = rng.standard_normal(ch)
    x = rng.standard_normal((11, ch))
    whole, st_whole = O.causal_conv_silu(x, w, b)
    outs, st = [], None
    for lo, hi in [(0, 1), (1, 3), (3, 4), (4, 9), (9, 11)]:       # pieces shorter than k-1 too
        o, st = O.causal_conv_silu(x[lo:hi], w, b, st)
        outs.append(o)
    np.testing.assert_allclose(np.concatenate(outs), whole, rtol=1e-14, atol=1e-15)
    np.testing.assert_array_equal(st, st_whole)
    _, st1 = O.causal_conv_silu(x[:1], w, b)                        # one row: two zero rows then the row
    np.testing.assert_array_equal(st1, np.concatenate([np.zeros((2, ch)), x[:1]]))


# ------------------------------------------------------------------ recurrence

def _tiny_scan_inputs(L=7, H=2, P=3, N=4, G=1):
    x = rng.standard_normal((L, H, P))
    delta = rng.uniform(0.05, 1.0, (L, H))
    a = rng.uniform(0.2, 0.99, (L, H))
    Bm = rng.standard_normal((L, G, N)); Cm = rng.standard_normal((L, G, N))
    D = rng.standard_normal(H)
    return x, delta, a, Bm, Cm, D


def test_recurrence_equals_materialised_sum():
    """h_t = sum_{s<=t} (prod_{r=s+1..t} a_r) Delta_s x_s (outer) B_s, built term by term."""
    L, H, P, N = 7, 2, 3, 4
    x, delta, a, Bm, Cm, D = _tiny_scan_inputs(L, H, P, N)
    y, h_last = O.ssm_recurrence(x, delta, a, Bm, Cm, D)
    for t in range(L):
        for h in range(H):
            hs = np.zeros((P, N))
            for s in range(t + 1):
                decay = 1.0
                for r in range(s + 1, t + 1):
                    decay *= a[r, h]
                for p in range(P):
                    for n in range(N):
                        hs[p, n] += decay * delta[s, h] * x[s, h, p] * Bm[s, 0, n]
            yt = hs @ Cm[t, 0] + D[h] * x[t, h]
            np.testing.assert_allclose(y[t, h], yt, rtol=1e-12, atol=1e-13)
            if t == L - 1:
                np.testing.assert_allclose(h_last[h], hs, rtol=1e-12, atol=1e-13)


def test_recurrence_equals_masked_quadratic_form():
    """y = (M o (C B^T)) (Delta o x) + D x with M_ts = prod_{r=s+1..t} a_r for t >= s, else 0."""
    L, H, P, N = 12, 3, 2, 5
    x, delta, a, Bm, Cm, D = _tiny_scan_inputs(L, H, P, N)
    y, _ = O.ssm_recurrence(x, delta, a, Bm, Cm, D)
    S = Cm[:, 0] @ Bm[:, 0].T
    for h in range(H):
        M = np.zeros((L, L))
        for t in range(L):
            for s in range(t + 1):
                M[t, s] = np.prod(a[s + 1:t + 1, h])
        yq = (M * S) @ (delta[:, h, None] * x[:, h]) + D[h] * x[:, h]
        np.testing.assert_allclose(y[:, h], yq, rtol=1e-12, atol=1e-13)


def test_recurrence_initial_state_term():
    """With x = 0 the state only decays: h_t = (prod a) h0 and y_t = h_t C_t."""
    L, H, P, N = 6, 2, 3, 4
    _, delta, a, Bm, Cm, D = _tiny_scan_inputs(L, H, P, N)
    h0 = rng.standard_normal((H, P, N))
    y, h_last = O.ssm_recurrence(np.zeros((L, H, P)), delta, a, Bm, Cm, D, h0)
    cum = np.cumprod(a, axis=0)
    for t in range(L):
        np.testing.assert_allclose(y[t], np.einsum("hpn,n->hp", cum[t][:, None, None] * h0, Cm[t, 0]), rtol=1e-12)
    np.testing.assert_allclose(h_last, cum[-1][:, None, None] * h0, rtol=1e-12)


def test_closed_form_geometric_series():
    L, dlt, av = 20, 0.3, 0.8
    x = np.ones((L, 1, 1)); B = np.ones((L, 1, 1)); C = np.ones((L, 1, 1))
    y, h = O.ssm_recurrence(x, np.full((L, 1), dlt), np.full((L, 1), av), B, C, None)
    t = np.arange(L)
    np.testing.assert_allclose(y[:, 0, 0], dlt * (1 - av ** (t + 1)) / (1 - av), rtol=1e-13)


def test_no_decay_is_running_sum_and_full_decay_is_memoryless():
    L, H, P, N = 15, 2, 3, 4
    x, delta, _, Bm, Cm, D = _tiny_scan_inputs(L, H, P, N)
    y1, _ = O.ssm_recurrence(x, delta, np.ones((L, H)), Bm, Cm, None)
    for h in range(H):
        for p in range(P):
            run = np.cumsum((delta[:, h] * x[:, h, p])[:, None] * Bm[:, 0], axis=0)      # [L, N]
            np.testing.assert_allclose(y1[:, h, p], np.sum(run * Cm[:, 0], axis=1), rtol=1e-12, atol=1e-13)
    y0, _ = O.ssm_recurrence(x, delta, np.zeros((L, H)), Bm, Cm, D)
    cb = np.sum(Cm[:, 0] * Bm[:, 0], axis=1)
    np.testing.assert_allclose(y0, (delta * cb[:, None])[:, :, None] * x + D[None, :, None] * x, rtol=1e-12, atol=1e-13)


def test_single_token():
    x, delta, a, Bm, Cm, D = _tiny_scan_inputs(1, 2, 3, 4)
    y, h = O.ssm_recurrence(x, delta, a, Bm, Cm, D)
    np.testing.assert_allclose(h, (delta[0][:, None] * x[0])[:, :, None] * Bm[0, 0][None, None, :], rtol=1e-14)
    np.testing.assert_allclose(y[0], np.dot(Bm[0, 0], Cm[0, 0]) * delta[0][:, None] * x[0] + D[:, None] * x[0], rtol=1e-13)


def test_groups_share_B_and_C():
    L, H, P, N, G = 6, 4, 2, 3, 2
    x, delta, a, Bm, Cm, D = _tiny_scan_inputs(L, H, P, N, G)
    y, _ = O.ssm_recurrence(x, delta, a, Bm, Cm, D)
    for h in range(H):
        g = h // (H // G)
        yh, _ = O.ssm_recurrence(x[:, h:h + 1], delta[:, h:h + 1], a[:, h:h + 1], Bm[:, g:g + 1], Cm[:, g:g + 1], D[h:h + 1])
        np.testing.assert_allclose(y[:, h], yh[:, 0], rtol=1e-13)


def test_scan_is_linear_in_x():
    x, delta, a, Bm, Cm, D = _tiny_scan_inputs(9, 2, 3, 4)
    x2 = rng.standard_normal(x.shape)
    f = lambda v: O.ssm_recurrence(v, delta, a, Bm, Cm, D)[0]
    np.testing.assert_allclose(f(2.0 * x - 3.0 * x2), 2.0 * f(x) - 3.0 * f(x2), rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ gate / norm

def test_gate_and_gated_norm():
    y = rng.standard_normal((5, 16)); z = rng.standard_normal((5, 16)); w = rng.uniform(0.5, 1.5, 16)
    g0 = O.gate(y, z, None, gated_norm=False)
    np.testing.assert_allclose(g0, y * z * special.expit(z), rtol=1e-14)
    g1 = O.gate(y, z, None, eps=0.0, gated_norm=True)
    np.testing.assert_allclose(np.sqrt(np.mean(g1 ** 2, axis=-1)), 1.0, rtol=1e-13)       # unit RMS
    np.testing.assert_allclose(O.gate(7.0 * y, z, w, eps=0.0), O.gate(y, z, w, eps=0.0), rtol=1e-12)   # scale free
    np.testing.assert_allclose(O.gate(y, z, w, eps=0.0), g1 * w, rtol=1e-13)
    ge = O.gate(y, z, w, eps=0.5)
    np.testing.assert_allclose(ge, g0 / np.sqrt(np.mean(g0 ** 2, -1, keepdims=True) + 0.5) * w, rtol=1e-13)


# ------------------------------------------------------------------ a whole direction, by scalar loops

def _tiny_weights(d=6, expand=2, N=3, H=4, k=4, G=1, seed=5):
    r = np.random.default_rng(seed)
    dd = O.derived_dims(d, expand, N, H, G)
    return {
        "w_in": r.standard_normal((dd["d_in_proj"], d)) * 0.5,
        "conv_w": r.standard_normal((dd["conv_ch"], k)) * 0.5,
        "conv_b": r.standard_normal(dd["conv_ch"]) * 0.5,
        "dt_bias": r.standard_normal(H),
        "A_log": np.log(r.uniform(1, 4, H)),
        "D": r.standard_normal(H),
        "norm_w": r.uniform(0.5, 1.5, dd["d_inner"]),
        "w_out": r.standard_normal((d, dd["d_inner"])) * 0.5,
    }, dd


KW = dict(expand=2, d_state=3, n_heads=4, n_groups=1)


def _direction_by_scalar_loops(u, w, dd, N, H, k, reverse, gated_norm=True, eps=1e-5):
    """Independent scalar statement: for the reverse direction the conv looks at right neighbours and
    the recurrence runs t = L-1 .. 0 (no flipping anywhere)."""
    import math
    L, d = u.shape
    di, P, cc = dd["d_inner"], dd["headdim"], dd["conv_ch"]
    proj = [[sum(w["w_in"][o, i] * u[t, i] for i in range(d)) for o in range(dd["d_in_proj"])] for t in range(L)]
    step = -1 if reverse else 1
    act = [[0.0] * cc for _ in range(L)]
    for t in range(L):
        for c in range(cc):
            v = w["conv_b"][c]
            for j in range(k):
                src = t - step * (k - 1 - j)           # fwd: t-(k-1-j); rev: t+(k-1-j)
                if 0 <= src < L:
                    v += w["conv_w"][c, j] * proj[src][di + c]
            act[t][c] = v / (1.0 + math.exp(-v))
    out = np.zeros((L, d))
    hst = np.zeros((H, P, N))
    order = range(L - 1, -1, -1) if reverse else range(L)
    for t in order:
        gvec = np.zeros(di)
        for h in range(H):
            raw = proj[t][di + cc + h] + w["dt_bias"][h]
            dl = max(raw, 0.0) + math.log1p(math.exp(-abs(raw)))
            dec = math.exp(-dl * math.exp(w["A_log"][h]))
            for p in range(P):
                xv = act[t][h * P + p]
                acc = 0.0
                for n in range(N):
                    hst[h, p, n] = dec * hst[h, p, n] + dl * xv * act[t][di + n]
                    acc += hst[h, p, n] * act[t][di + N + n]
                zv = proj[t][h * P + p]
                gvec[h * P + p] = (acc + w["D"][h] * xv) * zv / (1.0 + math.exp(-zv))
        if gated_norm:
            gvec = gvec / math.sqrt(float(np.mean(gvec ** 2)) + eps) * w["norm_w"]
        out[t] = w["w_out"] @ gvec
    return out


@pytest.mark.parametrize("gated_norm", [True, False])
def test_bimamba_forward_equals_scalar_definition(gated_norm):
    w_f, dd = _tiny_weights(seed=5)
    w_r, _ = _tiny_weights(seed=6)
    x = rng.standard_normal((2, 9, 6))
    full = O.bimamba_forward(x, w_f, w_r, gated_norm=gated_norm, **KW)
    for b in range(2):
        f = _direction_by_scalar_loops(x[b], w_f, dd, 3, 4, 4, False, gated_norm)
        r = _direction_by_scalar_loops(x[b], w_r, dd, 3, 4, 4, True, gated_norm)
        np.testing.assert_allclose(full[b], f + r, rtol=1e-10, atol=1e-11)
        np.testing.assert_allclose(O.bimamba_forward(x[b:b + 1], w_f, w_r, dir_mask=O.DIR_REV, gated_norm=gated_norm, **KW)[0],
                                   r, rtol=1e-10, atol=1e-11)


# ------------------------------------------------------------------ invariants of the mixer

def test_reversal_invariant():
    w_f, _ = _tiny_weights(seed=7)
    x = rng.standard_normal((1, 13, 6))
    rev = O.bimamba_forward(x, w_f, w_f, dir_mask=O.DIR_REV, **KW)
    fwd_on_flipped = O.bimamba_forward(x[:, ::-1], w_f, w_f, dir_mask=O.DIR_FWD, **KW)
    np.testing.assert_allclose(rev, fwd_on_flipped[:, ::-1], rtol=1e-13, atol=1e-14)


def test_causality_of_each_direction():
    w_f, _ = _tiny_weights(seed=8)
    w_r, _ = _tiny_weights(seed=9)
    x = rng.standard_normal((1, 12, 6)); tau = 5
    x2 = x.copy(); x2[0, tau] += 1.0
    df = O.bimamba_forward(x2, w_f, w_r, dir_mask=O.DIR_FWD, **KW) - O.bimamba_forward(x, w_f, w_r, dir_mask=O.DIR_FWD, **KW)
    dr = O.bimamba_forward(x2, w_f, w_r, dir_mask=O.DIR_REV, **KW) - O.bimamba_forward(x, w_f, w_r, dir_mask=O.DIR_REV, **KW)
    assert np.all(df[0, :tau] == 0) and np.any(df[0, tau] != 0) and np.any(df[0, tau + 1:] != 0)
    assert np.all(dr[0, tau + 1:] == 0) and np.any(dr[0, tau] != 0) and np.any(dr[0, :tau] != 0)


def test_batch_rows_are_independent_and_sum_of_directions():
    w_f, _ = _tiny_weights(seed=10)
    w_r, _ = _tiny_weights(seed=11)
    x = rng.standard_normal((3, 8, 6))
    full = O.bimamba_forward(x, w_f, w_r, **KW)
    np.testing.assert_allclose(full[1:2], O.bimamba_forward(x[1:2], w_f, w_r, **KW), rtol=1e-14)
    parts = O.bimamba_forward(x, w_f, w_r, dir_mask=O.DIR_FWD, **KW) + O.bimamba_forward(x, w_f, w_r, dir_mask=O.DIR_REV, **KW)
    np.testing.assert_allclose(full, parts, rtol=1e-13, atol=1e-14)


def test_heads_interact_only_through_the_norm():
    w_f, dd = _tiny_weights(seed=12)
    u = rng.standard_normal((7, 6))
    _, _, _, parts = O.mamba2_direction(u, w_f, gated_norm=False, return_parts=True, **KW)
    w2 = {k: v.copy() for k, v in w_f.items()}
    w2["A_log"][2] += 1.0; w2["D"][2] -= 0.5; w2["dt_bias"][2] += 0.3
    _, _, _, parts2 = O.mamba2_direction(u, w2, gated_norm=False, return_parts=True, **KW)
    P = dd["headdim"]
    same = np.ones(dd["d_inner"], bool); same[2 * P:3 * P] = False
    np.testing.assert_array_equal(parts["g"][:, same], parts2["g"][:, same])
    assert np.any(parts["g"][:, ~same] != parts2["g"][:, ~same])


def test_block_step_invariant():
    """Block-by-block state carry == one pass over the committed prefix (left-to-right layer)."""
    w_f, dd = _tiny_weights(seed=13)
    w_r, _ = _tiny_weights(seed=14)
    x = rng.standard_normal((2, 14, 6))
    whole = O.bimamba_forward(x, w_f, w_r, dir_mask=O.DIR_FWD, **KW)
    _, ssm_whole, conv_whole = O.bimamba_block_step(x, w_f, w_r, dir_mask=O.DIR_FWD, **KW)
    ssm = conv = None
    outs = []
    for lo, hi in [(0, 4), (4, 5), (5, 7), (7, 14)]:
        o, ssm, conv = O.bimamba_block_step(x[:, lo:hi], w_f, w_r, ssm_state_in=ssm, conv_state_in=conv,
                                            dir_mask=O.DIR_FWD, **KW)
        outs.append(o)
    np.testing.assert_allclose(np.concatenate(outs, axis=1), whole, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(ssm, ssm_whole, rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(conv, conv_whole)
    assert ssm.shape == (2, 4, dd["headdim"], 3) and conv.shape == (2, 3, dd["conv_ch"])


def test_block_step_reverse_sees_only_the_block():
    w_f, _ = _tiny_weights(seed=15)
    w_r, _ = _tiny_weights(seed=16)
    x = rng.standard_normal((1, 10, 6))
    ssm = rng.standard_normal((1, 4, 3, 3)); conv = rng.standard_normal((1, 3, 18))
    blk = x[:, 6:]
    y, _, _ = O.bimamba_block_step(blk, w_f, w_r, ssm_state_in=ssm, conv_state_in=conv, dir_mask=O.DIR_REV, **KW)
    np.testing.assert_allclose(y, O.bimamba_forward(blk, w_f, w_r, dir_mask=O.DIR_REV, **KW), rtol=1e-14)
    both, _, _ = O.bimamba_block_step(blk, w_f, w_r, ssm_state_in=ssm, conv_state_in=conv, **KW)
    f_only, _, _ = O.bimamba_block_step(blk, w_f, w_r, ssm_state_in=ssm, conv_state_in=conv, dir_mask=O.DIR_FWD, **KW)
    np.testing.assert_allclose(both, f_only + y, rtol=1e-13, atol=1e-14)


# ------------------------------------------------------------------ stack

def _tiny_stack(n_layers=2, V=11, d=6, seed=20):
    r = np.random.default_rng(seed)
    layers = []
    for i in range(n_layers):
        f, _ = _tiny_weights(seed=seed + 2 * i + 1)
        b, _ = _tiny_weights(seed=seed + 2 * i + 2)
        layers.append({"norm_w": r.uniform(0.5, 1.5, d), "fwd": f, "rev": b})
    return {"embed": r.standard_normal((V, d)), "w_vocab": r.standard_normal((V, d)),
            "final_norm_w": r.uniform(0.5, 1.5, d), "layers": layers}


def test_rmsnorm():
    r = rng.standard_normal((4, 8)); w = rng.uniform(0.5, 1.5, 8)
    n = O.rmsnorm(r, w, eps=0.0)
    np.testing.assert_allclose(n, r / np.linalg.norm(r, axis=-1, keepdims=True) * np.sqrt(8) * w, rtol=1e-13)


def test_stack_structure():
    sw = _tiny_stack()
    tok = rng.integers(0, 11, (2, 7))
    logits, hidden = O.denoise_step(tok, sw, return_hidden=True, **KW)
    assert logits.shape == (2, 7, 11)
    np.testing.assert_array_equal(hidden[0], sw["embed"][tok])
    for i, layer in enumerate(sw["layers"]):                      # r_{l+1} - r_l is the mixer of the normed input
        m = O.bimamba_forward(O.rmsnorm(hidden[i], layer["norm_w"]), layer["fwd"], layer["rev"], **KW)
        np.testing.assert_allclose(hidden[i + 1] - hidden[i], m, rtol=1e-10, atol=1e-12)
    # with silent mixers the stack is a table lookup followed by the head
    mute = {**sw, "layers": [{**l, "fwd": {**l["fwd"], "w_out": 0 * l["fwd"]["w_out"]},
                              "rev": {**l["rev"], "w_out": 0 * l["rev"]["w_out"]}} for l in sw["layers"]]}
    e = sw["embed"][tok]
    head = e / np.sqrt(np.mean(e ** 2, -1, keepdims=True) + 1e-5) * sw["final_norm_w"] @ sw["w_vocab"].T
    np.testing.assert_allclose(O.denoise_step(tok, mute, **KW), head, rtol=1e-12)


def test_stack_block_mode_matches_prefix_pass_for_forward_direction():
    sw = _tiny_stack()
    tok = rng.integers(0, 11, (1, 9))
    kw = dict(KW, dir_mask=O.DIR_FWD)
    whole = O.denoise_step(tok, sw, **kw)
    _, st = O.denoise_step(tok[:, :5], sw, return_states=True, **kw)
    tail, st2 = O.denoise_step(tok[:, 5:], sw, states_in=st, return_states=True, **kw)
    np.testing.assert_allclose(tail, whole[:, 5:], rtol=1e-10, atol=1e-12)
    assert len(st2) == 2 and st2[0][0].shape == (1, 4, 3, 3)


# ------------------------------------------------------------------ timestep-conditioned block (App. A.1)

def _tiny_cond_stack(n_layers=2, d=6, d_ff=12, d_c=5, seed=40):
    sw = _tiny_stack(n_layers, d=d, seed=seed)
    r = np.random.default_rng(seed + 100)
    for layer in sw["layers"]:
        layer.update(w_cond=r.standard_normal((6 * d, d_c)), b_cond=r.standard_normal(6 * d),
                     w_up=r.standard_normal((d_ff, d)), b_up=r.standard_normal(d_ff),
                     w_down=r.standard_normal((d, d_ff)), b_down=r.standard_normal(d))
    return sw, r.standard_normal((2, d_c))


def test_layernorm_standardises_and_adaln_is_affine_in_its_modulation():
    x = rng.standard_normal((2, 5, 9)) * 3 + 7
    n = O.layernorm_plain(x, eps=0.0)
    np.testing.assert_allclose(n.mean(-1), 0, atol=1e-13)
    np.testing.assert_allclose((n ** 2).mean(-1), 1, rtol=1e-12)
    np.testing.assert_allclose(O.layernorm_plain(4.0 * x - 11.0, eps=0.0), n, rtol=1e-10, atol=1e-12)   # shift and scale invariant
    for bb in range(2):                                           # the textbook z-score, element by element
        for t in range(5):
            row = x[bb, t]
            mu = sum(row) / 9
            sd = (sum((v - mu) ** 2 for v in row) / 9 + 1e-5) ** 0.5
            np.testing.assert_allclose(O.layernorm_plain(x)[bb, t], [(v - mu) / sd for v in row], rtol=1e-12)
    g, b = rng.standard_normal((2, 9)), rng.standard_normal((2, 9))
    np.testing.assert_allclose(O.adaln(x, np.ones((2, 9)), np.zeros((2, 9)), 0.0), n, rtol=1e-13)
    np.testing.assert_allclose(O.adaln(x, g, b, 0.0), g[:, None] * n + b[:, None], rtol=1e-13)
    assert np.all(O.adaln(x, g, b)[0, :, 0] != O.adaln(x, g, b)[1, :, 0])      # one modulation per sequence


def test_gelu_against_the_exact_form_and_its_symmetry():
    v = np.linspace(-8, 8, 1601)
    exact = 0.5 * v * (1 + special.erf(v / np.sqrt(2)))
    assert np.max(np.abs(O.gelu_tanh(v) - exact)) < 5e-4          # the tanh form's known distance from the erf form
    np.testing.assert_allclose(O.gelu_tanh(v) - O.gelu_tanh(-v), v, atol=1e-14)   # gelu(x) - gelu(-x) = x
    assert O.gelu_tanh(0.0) == 0.0 and abs(O.gelu_tanh(30.0) - 30.0) < 1e-12 and abs(O.gelu_tanh(-30.0)) < 1e-12


def test_modulation_and_mlp_by_loops():
    sw, tau = _tiny_cond_stack()
    L0 = sw["layers"][0]
    parts = O.modulation(tau, L0["w_cond"], L0["b_cond"])
    assert len(parts) == 6 and all(p.shape == (2, 6) for p in parts)
    for k in range(6):
        for bb in range(2):
            for j in range(6):
                want = L0["b_cond"][k * 6 + j] + sum(L0["w_cond"][k * 6 + j, c] * tau[bb, c] for c in range(5))
                assert parts[k][bb, j] == pytest.approx(want, rel=1e-12, abs=1e-13)
    np.testing.assert_allclose(np.concatenate(O.modulation(0 * tau, L0["w_cond"], L0["b_cond"]), 1), np.tile(L0["b_cond"], (2, 1)))
    u = rng.standard_normal((2, 3, 6))
    got = O.mlp(u, L0["w_up"], L0["w_down"], L0["b_up"], L0["b_down"])
    for bb in range(2):
        for t in range(3):
            hid = [O.gelu_tanh(L0["b_up"][f] + sum(L0["w_up"][f, c] * u[bb, t, c] for c in range(6))) for f in range(12)]
            for j in range(6):
                assert got[bb, t, j] == pytest.approx(L0["b_down"][j] + sum(L0["w_down"][j, f] * hid[f] for f in range(12)), rel=1e-11)
    # FLOP rows "MLP" and "AdaLN" of App. C from the weight shapes a 1.3B layer would have (2mn per linear layer)
    g = _golden("appC_mamba_layer_flops.txt")
    d, d_ff, d_c = 1920, 3840, 128
    assert round((2 * d_ff * d + 2 * d * d_ff) / 1e6, 2) == g["mlp_M"] and round(2 * (6 * d) * d_c / 1e6, 2) == g["adaln_M"]


def test_diffusion_block_structure():
    sw, tau = _tiny_cond_stack()
    L0 = sw["layers"][0]
    x = rng.standard_normal((2, 7, 6))
    d = 6
    def with_bias(vec):                                           # modulation independent of tau: W_cond = 0, bias = vec
        return {**L0, "w_cond": 0 * L0["w_cond"], "b_cond": np.asarray(vec, float)}
    one, zero = np.ones(d), np.zeros(d)
    # both gates shut: the block is the identity
    np.testing.assert_array_equal(O.diffusion_block(x, tau, with_bias(np.r_[zero, one, zero, zero, one, zero]), **KW), x)
    # gamma = 1, beta = 0, gates = 1: the two equations as printed
    y = O.diffusion_block(x, tau, with_bias(np.r_[zero, one, one, zero, one, one]), **KW)
    ym = x + O.bimamba_forward(O.layernorm_plain(x), L0["fwd"], L0["rev"], **KW)
    want = ym + O.mlp(O.layernorm_plain(ym), L0["w_up"], L0["w_down"], L0["b_up"], L0["b_down"])
    np.testing.assert_allclose(y, want, rtol=1e-11, atol=1e-12)
    # MLP gate shut: what remains is linear in the mixer gate
    y1 = O.diffusion_block(x, tau, with_bias(np.r_[zero, one, one, zero, one, zero]), **KW)
    y3 = O.diffusion_block(x, tau, with_bias(np.r_[zero, one, 3 * one, zero, one, zero]), **KW)
    np.testing.assert_allclose(y3 - x, 3 * (y1 - x), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(y1, ym, rtol=1e-11, atol=1e-12)
    # the general case, assembled from the pinned parts
    b1, s1, g1, b2, s2, g2 = O.modulation(tau, L0["w_cond"], L0["b_cond"])
    ym = x + g1[:, None] * O.bimamba_forward(O.adaln(x, s1, b1), L0["fwd"], L0["rev"], **KW)
    want = ym + g2[:, None] * O.mlp(O.adaln(ym, s2, b2), L0["w_up"], L0["w_down"], L0["b_up"], L0["b_down"])
    np.testing.assert_allclose(O.diffusion_block(x, tau, L0, **KW), want, rtol=1e-11, atol=1e-12)
    # sequences do not interact and each sees its own timestep
    tau2 = tau.copy(); tau2[1] += 1.0
    ya, yb = O.diffusion_block(x, tau, L0, **KW), O.diffusion_block(x, tau2, L0, **KW)
    np.testing.assert_array_equal(ya[0], yb[0]); assert np.any(ya[1] != yb[1])


def test_conditioned_stack_and_its_block_mode():
    sw, tau = _tiny_cond_stack()
    tok = rng.integers(0, 11, (2, 8))
    logits = O.denoise_step_cond(tok, tau, sw, **KW)
    r = sw["embed"][tok]
    for layer in sw["layers"]:
        r = O.diffusion_block(r, tau, layer, **KW)
    np.testing.assert_allclose(logits, O.rmsnorm(r, sw["final_norm_w"]) @ sw["w_vocab"].T, rtol=1e-12)
    # all gates shut: a table lookup followed by the head
    shut = {**sw, "layers": [{**l, "w_cond": 0 * l["w_cond"], "b_cond": 0 * l["b_cond"]} for l in sw["layers"]]}
    e = sw["embed"][tok]
    head = e / np.sqrt(np.mean(e ** 2, -1, keepdims=True) + 1e-5) * sw["final_norm_w"] @ sw["w_vocab"].T
    np.testing.assert_allclose(O.denoise_step_cond(tok, tau, shut, **KW), head, rtol=1e-12)
    # block mode, left-to-right direction only: two blocks through the carried state == one pass (Sec. 4.3);
    # the AdaLN statistics are per token, so they do not couple the blocks
    kw = dict(KW, dir_mask=O.DIR_FWD)
    whole = O.denoise_step_cond(tok, tau, sw, **kw)
    l1, st = O.denoise_step_cond(tok[:, :5], tau, sw, return_states=True, **kw)
    l2, _ = O.denoise_step_cond(tok[:, 5:], tau, sw, states_in=st, return_states=True, **kw)
    np.testing.assert_allclose(np.concatenate([l1, l2], 1), whole, rtol=1e-9, atol=1e-11)


# ------------------------------------------------------------------ reverse step (Sec. 2, Eq. 3)

def test_reverse_step_cases_and_probabilities():
    V, mask = 7, 6
    z = rng.standard_normal(V) * 2
    # the three cases of Eq. 3 as a probability vector
    q = O.reverse_step_probabilities(z, False, 3, 0.4, mask)
    assert q[3] == 1.0 and q.sum() == 1.0
    q = O.reverse_step_probabilities(z, True, mask, 0.4, mask)
    soft = np.exp(z[:mask]) / np.exp(z[:mask]).sum()                      # softmax over the real tokens only
    np.testing.assert_allclose(q[:mask], 0.6 * soft, rtol=1e-12)
    assert q[mask] == pytest.approx(0.4) and q.sum() == pytest.approx(1.0)
    # the draw realises those probabilities: sweep both uniforms over a fine grid (a deterministic integral)
    n = 400
    uk, uc = np.meshgrid((np.arange(n) + 0.5) / n, (np.arange(n) + 0.5) / n, indexing="ij")
    tok = np.full((1, n * n), mask)
    logits = np.broadcast_to(z, (1, n * n, V))
    out = O.reverse_step(tok, logits, uk.reshape(1, -1), uc.reshape(1, -1), 0.4, mask)
    freq = np.bincount(out.ravel(), minlength=V) / (n * n)
    np.testing.assert_allclose(freq, q, atol=2.0 / n)
    # unmasked tokens are carried over whatever the uniforms say; the mask token is never drawn
    tok2 = np.array([[0, mask, 5, mask]])
    lg = rng.standard_normal((1, 4, V))
    o2 = O.reverse_step(tok2, lg, np.array([[0.0, 0.9, 0.0, 0.1]]), np.array([[0.5, 0.5, 0.5, 0.5]]), 0.4, mask)
    assert o2[0, 0] == 0 and o2[0, 2] == 5 and o2[0, 3] == mask and o2[0, 1] != mask
    # extremes of the inverse CDF: u -> 0 picks the first token with probability, u -> 1 the last one
    lg3 = np.zeros((1, 2, V)); lg3[0, :, 0] = -np.inf
    o3 = O.reverse_step(np.full((1, 2), mask), lg3, np.ones((1, 2)) * 0.99, np.array([[0.0, 1.0 - 1e-12]]), 0.4, mask)
    assert o3[0, 0] == 1 and o3[0, 1] == mask - 1
    # keep_prob 0 unmasks everything, keep_prob 1 nothing
    full = O.reverse_step(np.full((1, 50), mask), rng.standard_normal((1, 50, V)), rng.random((1, 50)), rng.random((1, 50)), 0.0, mask)
    assert np.all(full != mask)
    none = O.reverse_step(np.full((1, 50), mask), rng.standard_normal((1, 50, V)), rng.random((1, 50)), rng.random((1, 50)), 1.0, mask)
    assert np.all(none == mask)


def test_noise_schedule_endpoints_and_expected_unmasking():
    t = O.noise_schedule(8)
    assert t[0] == 1.0 and t[-1] == pytest.approx(1e-3) and np.all(np.diff(t) < 0)
    np.testing.assert_allclose(np.diff(t), np.diff(t)[0])                  # uniform spacing: K = L / p steps of equal size (Sec. 4.3)
    # the chance that a token is still masked after k steps telescopes to t_k (Eq. 1's marginal: masked w.p. t)
    np.testing.assert_allclose(np.cumprod(t[1:] / t[:-1]), t[1:], rtol=1e-12)


# ------------------------------------------------------------------ attention mixer of the hybrid (Sec. 3.3)

def test_attention_mixer_by_loops_and_its_invariances():
    B, L, d, H = 2, 6, 8, 2
    dh = d // H
    x = rng.standard_normal((B, L, d)); wqkv = rng.standard_normal((3 * d, d)) * 0.5; wo = rng.standard_normal((d, d)) * 0.5
    got = O.attention_mixer(x, wqkv, wo, H)
    # scalar loops, straight from the definition
    want = np.zeros((B, L, d))
    for b in range(B):
        q = [[sum(wqkv[j, c] * x[b, t, c] for c in range(d)) for j in range(d)] for t in range(L)]
        k = [[sum(wqkv[d + j, c] * x[b, t, c] for c in range(d)) for j in range(d)] for t in range(L)]
        v = [[sum(wqkv[2 * d + j, c] * x[b, t, c] for c in range(d)) for j in range(d)] for t in range(L)]
        for t in range(L):
            cat = [0.0] * d
            for h in range(H):
                sc = [sum(q[t][h * dh + e] * k[u][h * dh + e] for e in range(dh)) / dh ** 0.5 for u in range(L)]
                m = max(sc); ex = [np.exp(a - m) for a in sc]; z = sum(ex)
                for e in range(dh):
                    cat[h * dh + e] = sum(ex[u] / z * v[u][h * dh + e] for u in range(L))
            for j in range(d):
                want[b, t, j] = sum(wo[j, c] * cat[c] for c in range(d))
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)
    # no position encoding and no causal mask: permuting the tokens permutes the outputs
    perm = rng.permutation(L)
    np.testing.assert_allclose(O.attention_mixer(x[:, perm], wqkv, wo, H), got[:, perm], rtol=1e-11, atol=1e-12)
    # zero queries: uniform attention, every token receives the mean value vector
    w0 = wqkv.copy(); w0[:d] = 0
    vbar = (x @ w0[2 * d:].T).mean(axis=1, keepdims=True)
    np.testing.assert_allclose(O.attention_mixer(x, w0, wo, H), np.broadcast_to(vbar @ wo.T, (B, L, d)), rtol=1e-11, atol=1e-12)
    # sequences do not interact; a single token attends to itself: out = W_o V x
    np.testing.assert_allclose(O.attention_mixer(x[:1], wqkv, wo, H), got[:1], rtol=1e-12)
    one = x[:, :1]
    np.testing.assert_allclose(O.attention_mixer(one, wqkv, wo, H), one @ wqkv[2 * d:].T @ wo.T, rtol=1e-11)
    # the parameter-free part costs 4 L d FLOPs per token and the projections 8 d^2 (App. C, Transformer-layer table)
    assert 2 * (3 * d) * d + 2 * d * d == 8 * d * d


def test_hybrid_stack_places_attention_every_period_layers():
    d, H_attn = 6, 2
    sw, tau = _tiny_cond_stack(n_layers=6, d=d)
    r = np.random.default_rng(77)
    for l in sw["layers"]:
        l["w_qkv"] = r.standard_normal((3 * d, d)) * 0.3; l["w_o"] = r.standard_normal((d, d)) * 0.3
    tok = rng.integers(0, 11, (2, 5))
    # period 0: no attention anywhere = the plain stacks
    np.testing.assert_allclose(O.denoise_step_hybrid(tok, sw, attn_period=0, attn_heads=H_attn, **KW), O.denoise_step(tok, sw, **KW), rtol=1e-12)
    np.testing.assert_allclose(O.denoise_step_hybrid(tok, sw, attn_period=0, attn_heads=H_attn, tau=tau, **KW),
                               O.denoise_step_cond(tok, tau, sw, **KW), rtol=1e-12)
    # period 5 on 6 layers: layers 0 and 5 are attention (1 attention + 4 Mamba, repeated); rebuilt layer by layer
    x = sw["embed"][tok]
    for i, l in enumerate(sw["layers"]):
        u = O.rmsnorm(x, l["norm_w"])
        x = x + (O.attention_mixer(u, l["w_qkv"], l["w_o"], H_attn) if i in (0, 5) else O.bimamba_forward(u, l["fwd"], l["rev"], **KW))
    np.testing.assert_allclose(O.denoise_step_hybrid(tok, sw, attn_period=5, attn_heads=H_attn, **KW),
                               O.rmsnorm(x, sw["final_norm_w"]) @ sw["w_vocab"].T, rtol=1e-11)
    # Mamba weights of an attention layer are not used, and vice versa
    sw2 = {**sw, "layers": [dict(l) for l in sw["layers"]]}
    sw2["layers"][0]["fwd"] = {**sw2["layers"][0]["fwd"], "w_out": 0 * sw2["layers"][0]["fwd"]["w_out"]}
    sw2["layers"][1]["w_o"] = 0 * sw2["layers"][1]["w_o"]
    np.testing.assert_array_equal(O.denoise_step_hybrid(tok, sw2, attn_period=5, attn_heads=H_attn, tau=tau, **KW),
                                  O.denoise_step_hybrid(tok, sw, attn_period=5, attn_heads=H_attn, tau=tau, **KW))


def test_attention_block_step_with_a_key_value_cache():
    B, d, H = 2, 8, 2
    x = rng.standard_normal((B, 9, d)); wqkv = rng.standard_normal((3 * d, d)) * 0.5; wo = rng.standard_normal((d, d)) * 0.5
    # an empty cache: the block alone
    y, k, v = O.attention_block_step(x, wqkv, wo, H)
    np.testing.assert_allclose(y, O.attention_mixer(x, wqkv, wo, H), rtol=1e-12)
    np.testing.assert_allclose(k, x @ wqkv[d:2 * d].T, rtol=1e-12); np.testing.assert_allclose(v, x @ wqkv[2 * d:].T, rtol=1e-12)
    # prefix of 5 tokens cached, block of 4: the block's rows of full attention over all 9 tokens (the prefix rows of that
    # full pass differ, since a committed prefix never saw the block -- only the block's rows are compared)
    _, k5, v5 = O.attention_block_step(x[:, :5], wqkv, wo, H)
    y_blk, k9, v9 = O.attention_block_step(x[:, 5:], wqkv, wo, H, k5, v5)
    np.testing.assert_allclose(y_blk, O.attention_mixer(x, wqkv, wo, H)[:, 5:], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(k9, k, rtol=1e-12); np.testing.assert_allclose(v9, v, rtol=1e-12)
    # the cache is read, not recomputed: scaling the cached values scales their contribution
    y_zero, _, _ = O.attention_block_step(x[:, 5:], wqkv, wo, H, k5, 0 * v5)
    assert np.abs(y_zero - y_blk).max() > 1e-3


def test_hybrid_stack_block_mode_left_to_right_equals_one_pass_on_the_block_rows():
    """Left-to-right Mamba direction only: two blocks through the carried states and key/value caches give, on the second
    block's rows, the logits of ... a pass in which the first block never saw the second: rebuilt layer by layer."""
    d, H_attn = 6, 2
    sw, _ = _tiny_cond_stack(n_layers=3, d=d)
    r = np.random.default_rng(78)
    for l in sw["layers"]:
        l["w_qkv"] = r.standard_normal((3 * d, d)) * 0.3; l["w_o"] = r.standard_normal((d, d)) * 0.3
    tok = rng.integers(0, 11, (2, 9))
    kw = dict(KW, dir_mask=O.DIR_FWD)
    l1, st = O.denoise_step_hybrid(tok[:, :5], sw, attn_period=2, attn_heads=H_attn, return_states=True, **kw)
    l2, st2 = O.denoise_step_hybrid(tok[:, 5:], sw, attn_period=2, attn_heads=H_attn, states_in=st, return_states=True, **kw)
    assert len(st) == 3 and st[0][0].shape == (2, 5, d) and st2[0][0].shape == (2, 9, d) and st[1][0].ndim == 4
    # layer by layer: the prefix rows evolve alone; the block rows see the prefix through the Mamba state (exactly, for the
    # left-to-right direction) and through the cached keys and values
    xa, xb = sw["embed"][tok[:, :5]], sw["embed"][tok[:, 5:]]
    for i, l in enumerate(sw["layers"]):
        ua, ub = O.rmsnorm(xa, l["norm_w"]), O.rmsnorm(xb, l["norm_w"])
        if i % 2 == 0:
            ya, ka, va = O.attention_block_step(ua, l["w_qkv"], l["w_o"], H_attn)
            yb, _, _ = O.attention_block_step(ub, l["w_qkv"], l["w_o"], H_attn, ka, va)
        else:
            full = O.bimamba_forward(np.concatenate([ua, ub], 1), l["fwd"], l["rev"], **kw)     # causal: the prefix rows do not see the block
            ya, yb = full[:, :5], full[:, 5:]
        xa, xb = xa + ya, xb + yb
    np.testing.assert_allclose(l1, O.rmsnorm(xa, sw["final_norm_w"]) @ sw["w_vocab"].T, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(l2, O.rmsnorm(xb, sw["final_norm_w"]) @ sw["w_vocab"].T, rtol=1e-9, atol=1e-11)


# ------------------------------------------------------------------------------------------------
# The generation loop (Sec. 2 Eq. 3 applied K = L / p times, Sec. 4.3): pins that do not re-run the loop's own code
# ------------------------------------------------------------------------------------------------
def test_generation_survivors_follow_the_uniforms_in_closed_form():
    """Which positions are still masked after step k depends on the uniforms alone: position j survives steps 0..k iff
    u_keep[i, j] < s_i / t_i for every i <= k (and nothing survives the clean-up pass).  The survivor sets computed from
    that closed form -- without the denoiser -- must be the mask pattern of every entry of the loop's trace."""
    K, V, mask_id = 5, 40, 39
    sw, kw = _tiny_stack(n_layers=1, V=V, seed=31), KW
    r = np.random.default_rng(3)
    uk, uc = r.random((K + 1, 2, 12), dtype=np.float32), r.random((K + 1, 2, 12), dtype=np.float32)
    start = np.full((2, 12), mask_id, np.int32)
    start[0, 3], start[1, 7] = 5, 11                                   # a two-token prompt
    out, trace = O.generate(start, sw, uk, uc, K, mask_id, V, return_trace=True, **kw)
    t = O.noise_schedule(K)
    alive = start == mask_id
    for k in range(K):
        alive = alive & (uk[k] < np.float32(t[k + 1] / t[k]))
        np.testing.assert_array_equal(trace[k] == mask_id, alive)
    assert not np.any(trace[K] == mask_id) and np.array_equal(trace[K], out)
    assert out[0, 3] == 5 and out[1, 7] == 11                          # the prompt is carried through every step
    for k in range(1, K + 1):                                          # once drawn, a token never changes again
        fixed = trace[k - 1] != mask_id
        np.testing.assert_array_equal(trace[k][fixed], trace[k - 1][fixed])


def test_generation_keep_probabilities_telescope_to_the_noise_levels():
    """prod_{i <= k} s_i / t_i = t_{k+1} / t_0: the chance of still being masked after step k is the noise level itself
    (the marginal of the forward process, Eq. 1); the list ends with the clean-up pass's 0."""
    for K in (1, 4, 64):
        kp = O.generation_keep_probs(K, 1e-3)
        assert len(kp) == K + 1 and kp[-1] == 0.0
        t = 1.0 - (1.0 - 1e-3) * np.arange(K + 1) / K                  # App. A.1: from 1 to the sampling eps
        np.testing.assert_allclose(np.cumprod(np.asarray(kp[:-1], np.float64)), t[1:], rtol=1e-6)
        assert all(0.0 < p < 1.0 for p in kp[:-1])


def test_generation_with_one_step_is_two_reverse_steps():
    """K = 1: one scheduled step (keep probability eps / 1) and the clean-up pass -- written out with reverse_step."""
    V, mask_id = 40, 39
    sw, kw = _tiny_stack(n_layers=1, V=V, seed=32), KW
    r = np.random.default_rng(4)
    uk, uc = r.random((2, 2, 12), dtype=np.float32), r.random((2, 2, 12), dtype=np.float32)
    uk[0, 0, :3] = 0.0                                                 # below eps: these three stay masked in the scheduled step
    start = np.full((2, 12), mask_id, np.int32)
    x1 = O.reverse_step(start, O.denoise_step(start, sw, **kw), uk[0], uc[0], 1e-3, mask_id)
    assert np.all(x1[0, :3] == mask_id) and np.all(x1[1] != mask_id)
    x2 = O.reverse_step(x1, O.denoise_step(x1, sw, **kw), uk[1], uc[1], 0.0, mask_id)
    np.testing.assert_array_equal(O.generate(start, sw, uk, uc, 1, mask_id, V, **kw), x2)
