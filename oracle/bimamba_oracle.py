"""CPU oracle for the bidirectional Mamba-2 mixer of DiffuMamba's denoising step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of what the hot path
computes.  Only the tests, the smoke check and the benchmark's `cpu_baseline` / reference arm may
import it; the product (the CUDA library and its Python binding) never does, and this file imports
nothing from the product.

Everything is written token by token, in the order the paper states its model:

  * Sec. 3.2 / App. A.1: a BiMamba block is two independent Mamba layers, one run left-to-right and
    one right-to-left, fused by addition (Eq. "Mamba(x_i) = h_i-> + h_i<-").
  * App. C (per-token FLOPs table): one direction is in_proj (d -> D_in), a short depthwise Conv1d
    over conv_ch channels, the SSM scan with d_state states per channel, and out_proj (d_inner -> d).
    D_in combines gate, input, B, C and the per-head step size.
  * Sec. 4.3 (block-autoregressive inference): the left-to-right state is cached and carried from one
    committed block to the next; the right-to-left pass only sees the active block.
  * App. A.1: the stack is Embed -> N blocks (pre-norm, residual) -> OutputProj.

The paper does not print the discretisation of the Mamba-2 layer it uses; the reading taken here
(the usual Mamba-2 one: scalar decay per head, a = exp(Delta * A), input scaled by Delta, B and C
shared by the heads of a group, depthwise conv then SiLU on [x, B, C], gate by SiLU(z), optional
RMS normalisation of the gated output) is listed point by point in the design notes.

Parity status: every function below is pinned by tests (explicit sums, closed forms, textbook
routines, the paper's printed shape / FLOP numbers) except three choices the paper leaves open and
nothing printed can confirm -- the gated RMS norm inside each direction (both settings are
implemented and tested), when the carried state is committed, and the stack's plain RMSNorm
pre-norm without the MLP sublayer.  For those three: parity unpinned (by the paper); they follow
the stated readings.

The timestep-conditioned block of App. A.1 (AdaLN before the mixer and before the MLP, Eq. "AdaLN" and
the two equations after it) is `diffusion_block` / `denoise_step_cond`.  Its arithmetic is pinned
(standardisation, identities, brute force, the FLOP rows "MLP" and "AdaLN" of App. C); what the paper
leaves open there -- the third modulation vector per sublayer that App. C's 6*d count implies and the
equation does not show (read as a gate on the sublayer's output), the MLP's activation (GELU, tanh
form) and the epsilon of the normalisation -- is parity unpinned (by the paper) as well.

The generation loop `generate` (K reverse steps of Eq. 3 along `noise_schedule`, then one pass with keep probability 0) has
its arithmetic pinned (the survivor sets follow from the uniforms in closed form, the keep probabilities telescope to the
noise levels).  That the tokens still masked at the last noise level are drawn in one extra pass is this build's reading of
a point the paper leaves open: parity unpinned (by the paper).  The weight-tied variant needs no function of its own (it is
`bimamba_forward` called with the shared matrices in both directions' parameter sets); which parameters the paper's
"bidirectional weight tie" would cover is not stated: parity unpinned (by the paper).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------------------------
# Shapes and the per-token cost table (App. C)
# --------------------------------------------------------------------------------------------

def derived_dims(d_model: int, expand: int, d_state: int, n_heads: int, n_groups: int = 1) -> dict:
    """Widths of one direction (App. C: d_inner = expand*d; conv_ch covers x, B and C; D_in adds the
    gate and one step size per head)."""
    d_inner = expand * d_model
    if d_inner % n_heads or n_heads % n_groups:
        raise ValueError("d_inner must divide into heads, heads into groups")
    return {
        "d_inner": d_inner,
        "headdim": d_inner // n_heads,
        "conv_ch": d_inner + 2 * n_groups * d_state,
        "d_in_proj": 2 * d_inner + 2 * n_groups * d_state + n_heads,
    }


def flops_per_token(d_model: int, expand: int, d_state: int, d_conv: int, n_heads: int,
                    n_groups: int = 1, d_ff: int | None = None, d_c: int = 128) -> dict:
    """Forward FLOPs per token of one bidirectional Mamba-2 layer, with App. C's counting rules:
    2mn per linear layer, 2*d_inner*d_state for the scan, conv_ch*d_conv for the conv, twice for the
    two directions; MLP 4*d*d_ff; AdaLN 2*6d*d_c."""
    dd = derived_dims(d_model, expand, d_state, n_heads, n_groups)
    d_ff = 2 * d_model if d_ff is None else d_ff
    one = {
        "in_proj": 2 * d_model * dd["d_in_proj"],
        "conv": dd["conv_ch"] * d_conv,
        "scan": 2 * dd["d_inner"] * d_state,
        "out_proj": 2 * dd["d_inner"] * d_model,
    }
    one_dir = sum(one.values())
    out = dict(one)
    out["one_direction"] = one_dir
    out["mixer"] = 2 * one_dir
    out["mlp"] = 4 * d_model * d_ff
    out["adaln"] = 2 * 6 * d_model * d_c
    out["layer"] = out["mixer"] + out["mlp"] + out["adaln"]
    return out


def param_count(d_model: int, expand: int, d_state: int, d_conv: int, n_heads: int, n_layers: int,
                vocab: int, n_groups: int = 1, d_ff: int | None = None, d_c: int = 128) -> int:
    """Weights of the whole denoiser with two untied directions per layer (App. A.1 "bidirectional
    weight tie: False"), MLP and AdaLN modulation per layer, untied embedding and unembedding."""
    dd = derived_dims(d_model, expand, d_state, n_heads, n_groups)
    d_ff = 2 * d_model if d_ff is None else d_ff
    one_dir = (d_model * dd["d_in_proj"] + dd["conv_ch"] * d_conv + dd["conv_ch"]
               + 3 * n_heads + dd["d_inner"] + dd["d_inner"] * d_model)
    mlp = 2 * d_model * d_ff + d_ff + d_model
    adaln = 6 * d_model * d_c + 6 * d_model
    return n_layers * (2 * one_dir + mlp + adaln) + 2 * vocab * d_model + d_model


# --------------------------------------------------------------------------------------------
# Scalar functions
# --------------------------------------------------------------------------------------------

def softplus(v):
    v = np.asarray(v, dtype=F64)
    return np.maximum(v, 0.0) + np.log1p(np.exp(-np.abs(v)))


def silu(v):
    v = np.asarray(v, dtype=F64)
    with np.errstate(over="ignore"):          # exp(-v) = inf for very negative v gives the limit -0
        return v / (1.0 + np.exp(-v))


# --------------------------------------------------------------------------------------------
# One direction, step by step (App. C table rows, in order)
# --------------------------------------------------------------------------------------------

def in_proj(u, w_in):
    """Row "in_proj": zxBCdt[t] = W_in u[t], W_in [D_in, d], no bias."""
    return np.asarray(u, F64) @ np.asarray(w_in, F64).T


def split_zxbcdt(zxbcdt, d_inner: int, d_state: int, n_heads: int, n_groups: int = 1):
    """Column order [ z | x | B | C | dt ]; returns z, xBC (x, B, C still joined), dt."""
    conv_ch = d_inner + 2 * n_groups * d_state
    z = zxbcdt[..., :d_inner]
    xbc = zxbcdt[..., d_inner:d_inner + conv_ch]
    dt = zxbcdt[..., d_inner + conv_ch:]
    assert dt.shape[-1] == n_heads
    return z, xbc, dt


def causal_conv_silu(xbc, conv_w, conv_b=None, conv_state=None):
    """Row "Conv1d": depthwise filter of width k over each channel, looking only at the current and
    the k-1 previous rows, then SiLU.  Tap k-1 multiplies the current row.  Rows before the start are
    zero, or the carried conv_state [k-1, conv_ch] (the k-1 rows that preceded this call).
    Returns (activated [L, conv_ch], new conv_state = last k-1 pre-conv rows seen)."""
    xbc = np.asarray(xbc, F64)
    conv_w = np.asarray(conv_w, F64)
    L, ch = xbc.shape
    k = conv_w.shape[1]
    hist = np.zeros((k - 1, ch), F64) if conv_state is None else np.asarray(conv_state, F64)
    assert hist.shape == (k - 1, ch)
    padded = np.concatenate([hist, xbc], axis=0)          # row i of xbc is padded[i + k - 1]
    out = np.empty((L, ch), F64)
    for t in range(L):
        v = np.zeros(ch, F64) if conv_b is None else np.asarray(conv_b, F64).copy()
        for j in range(k):
            v += conv_w[:, j] * padded[t + j]              # padded[t + j] = xbc[t - (k-1) + j]
        out[t] = silu(v)
    return out, padded[L:L + k - 1].copy()


def discretise(dt_raw, dt_bias, A_log):
    """Step size and decay per token and head: Delta = softplus(dt + bias), A = -exp(A_log) < 0,
    a = exp(Delta * A) in (0, 1)."""
    delta = softplus(np.asarray(dt_raw, F64) + np.asarray(dt_bias, F64))
    A = -np.exp(np.asarray(A_log, F64))
    return delta, np.exp(delta * A)


def ssm_recurrence(x, delta, a, Bm, Cm, D=None, h0=None):
    """Row "SSM scan" (Sec. 3.2, first recurrence): for t = 0..L-1

        h_t = a_t * h_{t-1} + Delta_t * x_t (outer) B_t        h: [H, P, N]
        y_t = h_t C_t + D * x_t                                 (state after the update)

    x [L,H,P]; delta, a [L,H]; Bm, Cm [L,G,N] with heads h*G//H sharing a group; D [H] or None;
    h0 [H,P,N] or None (zeros).  Returns y [L,H,P] and the final state."""
    x = np.asarray(x, F64)
    L, H, P = x.shape
    G, N = Bm.shape[1], Bm.shape[2]
    rep = H // G
    h = np.zeros((H, P, N), F64) if h0 is None else np.array(h0, F64)
    y = np.empty((L, H, P), F64)
    for t in range(L):
        Bt = np.repeat(np.asarray(Bm[t], F64), rep, axis=0)     # [H, N]
        Ct = np.repeat(np.asarray(Cm[t], F64), rep, axis=0)
        h = a[t][:, None, None] * h + (delta[t][:, None] * x[t])[:, :, None] * Bt[:, None, :]
        y[t] = np.einsum("hpn,hn->hp", h, Ct)
        if D is not None:
            y[t] += np.asarray(D, F64)[:, None] * x[t]
    return y, h


def gate(y, z, norm_w=None, eps: float = 1e-5, gated_norm: bool = True):
    """g = y * SiLU(z); with gated_norm, g <- g / sqrt(mean_c g^2 + eps) * norm_w over the d_inner
    channels of each token (Sec. 3.2 "normalized ... before" the output projection)."""
    g = np.asarray(y, F64) * silu(z)
    if gated_norm:
        ms = np.mean(g * g, axis=-1, keepdims=True)
        g = g / np.sqrt(ms + eps)
        if norm_w is not None:
            g = g * np.asarray(norm_w, F64)
    return g


def out_proj(g, w_out):
    """Row "out_proj": out[t] = W_out g[t], W_out [d, d_inner], no bias."""
    return np.asarray(g, F64) @ np.asarray(w_out, F64).T


def mamba2_direction(u, w: dict, *, expand: int, d_state: int, n_heads: int, n_groups: int = 1,
                     gated_norm: bool = True, conv_bias: bool = True, d_skip: bool = True,
                     norm_eps: float = 1e-5, ssm_state=None, conv_state=None, return_parts: bool = False):
    """One left-to-right Mamba-2 layer over u [L, d].  Returns (out [L,d], ssm_state_out [H,P,N],
    conv_state_out [k-1, conv_ch])."""
    u = np.asarray(u, F64)
    L, d = u.shape
    dd = derived_dims(d, expand, d_state, n_heads, n_groups)
    d_inner, P = dd["d_inner"], dd["headdim"]
    zxbcdt = in_proj(u, w["w_in"])
    z, xbc, dt = split_zxbcdt(zxbcdt, d_inner, d_state, n_heads, n_groups)
    xbc_act, conv_out = causal_conv_silu(xbc, w["conv_w"], w["conv_b"] if conv_bias else None, conv_state)
    xs = xbc_act[:, :d_inner].reshape(L, n_heads, P)
    Bm = xbc_act[:, d_inner:d_inner + n_groups * d_state].reshape(L, n_groups, d_state)
    Cm = xbc_act[:, d_inner + n_groups * d_state:].reshape(L, n_groups, d_state)
    delta, a = discretise(dt, w["dt_bias"], w["A_log"])
    y, h_last = ssm_recurrence(xs, delta, a, Bm, Cm, w["D"] if d_skip else None, ssm_state)
    g = gate(y.reshape(L, d_inner), z, w.get("norm_w"), norm_eps, gated_norm)
    out = out_proj(g, w["w_out"])
    if return_parts:
        return out, h_last, conv_out, {"zxbcdt": zxbcdt, "xbc_act": xbc_act, "delta": delta, "a": a,
                                       "y": y.reshape(L, d_inner), "g": g}
    return out, h_last, conv_out


# --------------------------------------------------------------------------------------------
# The bidirectional mixer (Sec. 3.2) and its block-cache form (Sec. 4.3)
# --------------------------------------------------------------------------------------------

DIR_FWD, DIR_REV, DIR_BOTH = 1, 2, 3


def bimamba_forward(x, w_fwd: dict, w_rev: dict, *, dir_mask: int = DIR_BOTH, **kw):
    """Mamba(x) = h-> + h<- for x [B, L, d].  The right-to-left layer is the same operator applied
    to the sequence in reverse order (second recurrence of Sec. 3.2: i = L..1, anti-causal conv):
    flip, run, flip back.  dir_mask selects one direction only (for invariants)."""
    x = np.asarray(x, F64)
    out = np.zeros_like(x)
    for b in range(x.shape[0]):
        if dir_mask & DIR_FWD:
            out[b] += mamba2_direction(x[b], w_fwd, **kw)[0]
        if dir_mask & DIR_REV:
            out[b] += mamba2_direction(x[b][::-1], w_rev, **kw)[0][::-1]
    return out


def bimamba_block_step(x_blk, w_fwd: dict, w_rev: dict, *, ssm_state_in=None, conv_state_in=None,
                       dir_mask: int = DIR_BOTH, **kw):
    """One pass over the active block x_blk [B, G, d] (Sec. 4.3): the left-to-right layer starts from
    the carried (ssm, conv) state of the committed prefix; the right-to-left layer starts from zero
    and sees the block only.  Returns (y_blk, ssm_state_out [B,H,P,N], conv_state_out [B,k-1,conv_ch]):
    the left-to-right state after the block's last token."""
    x_blk = np.asarray(x_blk, F64)
    out = np.zeros_like(x_blk)
    ssm_out, conv_out = [], []
    for b in range(x_blk.shape[0]):
        s_in = None if ssm_state_in is None else ssm_state_in[b]
        c_in = None if conv_state_in is None else conv_state_in[b]
        o, s, c = mamba2_direction(x_blk[b], w_fwd, ssm_state=s_in, conv_state=c_in, **kw)
        ssm_out.append(s)
        conv_out.append(c)
        if dir_mask & DIR_FWD:
            out[b] += o
        if dir_mask & DIR_REV:
            out[b] += mamba2_direction(x_blk[b][::-1], w_rev, **kw)[0][::-1]
    return out, np.stack(ssm_out), np.stack(conv_out)


# --------------------------------------------------------------------------------------------
# The layer stack (App. A.1: Embed -> blocks -> OutputProj), mixer sublayer with RMSNorm pre-norm
# --------------------------------------------------------------------------------------------

def rmsnorm(r, w, eps: float = 1e-5):
    r = np.asarray(r, F64)
    return r / np.sqrt(np.mean(r * r, axis=-1, keepdims=True) + eps) * np.asarray(w, F64)


def denoise_step(tokens, sw: dict, *, rms_eps: float = 1e-5, states_in=None, return_states: bool = False,
                 return_hidden: bool = False, **kw):
    """logits[b,t,:] = W_vocab RMSNorm(r_N[b,t]); r_0 = E[tokens]; r_{l+1} = r_l + BiMamba_l(RMSNorm(r_l)).
    With states_in (one (ssm, conv) pair per layer, or None entries) every layer runs as a block step.
    Returns logits [B, L, V] (and the per-layer states after the block when return_states)."""
    tokens = np.asarray(tokens)
    r = np.asarray(sw["embed"], F64)[tokens]                   # [B, L, d]
    states_out = []
    hidden = [r.copy()]
    for i, layer in enumerate(sw["layers"]):
        u = rmsnorm(r, layer["norm_w"], rms_eps)
        if states_in is None and not return_states:
            m = bimamba_forward(u, layer["fwd"], layer["rev"], **kw)
        else:
            s_in, c_in = (None, None) if states_in is None or states_in[i] is None else states_in[i]
            m, s_out, c_out = bimamba_block_step(u, layer["fwd"], layer["rev"], ssm_state_in=s_in,
                                                 conv_state_in=c_in, **kw)
            states_out.append((s_out, c_out))
        r = r + m
        hidden.append(r.copy())
    logits = rmsnorm(r, sw["final_norm_w"], rms_eps) @ np.asarray(sw["w_vocab"], F64).T
    res = (logits,)
    if return_states:
        res += (states_out,)
    if return_hidden:
        res += (hidden,)
    return res[0] if len(res) == 1 else res


# --------------------------------------------------------------------------------------------
# Timestep-conditioned block (App. A.1): AdaLN -> mixer -> residual, AdaLN -> MLP -> residual
# --------------------------------------------------------------------------------------------
def layernorm_plain(x, eps: float = 1e-5):
    """(x - mu(x)) / sigma(x) over the channel axis (App. A.1, Eq. "AdaLN"): population variance,
    epsilon under the root, no learned affine."""
    x = np.asarray(x, F64)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps)


def adaln(x, gamma, beta, eps: float = 1e-5):
    """AdaLN(x; tau) = gamma_t * (x - mu) / sigma + beta_t (App. A.1); gamma, beta: [B, d], one pair per
    sequence (the timestep is per sequence), x: [B, L, d]."""
    return np.asarray(gamma, F64)[:, None, :] * layernorm_plain(x, eps) + np.asarray(beta, F64)[:, None, :]


def gelu_tanh(v):
    v = np.asarray(v, F64)
    return 0.5 * v * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (v + 0.044715 * v ** 3)))


def modulation(tau, w_cond, b_cond=None):
    """W_cond tau_t (+ bias): [B, d_c] -> six vectors of d channels per sequence (App. C counts
    2 * 6d * d_c FLOPs per layer).  Order: (beta, gamma, gate) of the mixer sublayer, then of the MLP
    sublayer."""
    tau = np.asarray(tau, F64)
    m = tau @ np.asarray(w_cond, F64).T
    if b_cond is not None:
        m = m + np.asarray(b_cond, F64)
    d = m.shape[1] // 6
    return tuple(m[:, i * d:(i + 1) * d] for i in range(6))


def mlp(u, w_up, w_down, b_up=None, b_down=None):
    """Two linear layers, d -> d_ff -> d (App. C: 4 * d * d_ff FLOPs), GELU between them."""
    hmid = np.asarray(u, F64) @ np.asarray(w_up, F64).T
    if b_up is not None:
        hmid = hmid + np.asarray(b_up, F64)
    out = gelu_tanh(hmid) @ np.asarray(w_down, F64).T
    if b_down is not None:
        out = out + np.asarray(b_down, F64)
    return out


def diffusion_block(x, tau, layer: dict, *, ln_eps: float = 1e-5, ssm_state_in=None, conv_state_in=None,
                    return_state: bool = False, **kw):
    """y_mixer = x + g1 * Mamba(AdaLN(x; tau)),  y_mlp = y_mixer + g2 * MLP(AdaLN(y_mixer; tau))  (App. A.1;
    g1 = g2 = 1 gives the equations exactly as printed)."""
    x = np.asarray(x, F64)
    b1, s1, g1, b2, s2, g2 = modulation(tau, layer["w_cond"], layer.get("b_cond"))
    u = adaln(x, s1, b1, ln_eps)
    if return_state or ssm_state_in is not None or conv_state_in is not None:
        m, s_out, c_out = bimamba_block_step(u, layer["fwd"], layer["rev"], ssm_state_in=ssm_state_in,
                                             conv_state_in=conv_state_in, **kw)
    else:
        m, s_out, c_out = bimamba_forward(u, layer["fwd"], layer["rev"], **kw), None, None
    y = x + g1[:, None, :] * m
    y = y + g2[:, None, :] * mlp(adaln(y, s2, b2, ln_eps), layer["w_up"], layer["w_down"], layer.get("b_up"), layer.get("b_down"))
    return (y, s_out, c_out) if return_state else y


def denoise_step_cond(tokens, tau, sw: dict, *, rms_eps: float = 1e-5, ln_eps: float = 1e-5, states_in=None,
                      return_states: bool = False, **kw):
    """z = OutputProj(B_N(... B_1(E(x_t), tau_t) ...))  (App. A.1), OutputProj = final RMSNorm + unembedding
    (App. C).  tau: [B, d_c], the timestep embedding of each sequence."""
    r = np.asarray(sw["embed"], F64)[np.asarray(tokens)]
    states_out = []
    for i, layer in enumerate(sw["layers"]):
        if states_in is None and not return_states:
            r = diffusion_block(r, tau, layer, ln_eps=ln_eps, **kw)
        else:
            s_in, c_in = (None, None) if states_in is None or states_in[i] is None else states_in[i]
            r, s_out, c_out = diffusion_block(r, tau, layer, ln_eps=ln_eps, ssm_state_in=s_in, conv_state_in=c_in,
                                              return_state=True, **kw)
            states_out.append((s_out, c_out))
    logits = rmsnorm(r, sw["final_norm_w"], rms_eps) @ np.asarray(sw["w_vocab"], F64).T
    return (logits, states_out) if return_states else logits


# --------------------------------------------------------------------------------------------
# Reverse step of the masked diffusion (Sec. 2, Eq. 3): from noise level t to s < t
# --------------------------------------------------------------------------------------------
def reverse_step_probabilities(logits_row, is_masked: bool, token: int, keep_prob: float, mask_id: int):
    """q_{s|t}(. | x_t) of one position as a vector over the vocabulary (Eq. 3), keep_prob = s / t:
    an unmasked token stays with probability 1; a masked one stays masked with probability s/t and
    otherwise becomes token v with probability (1 - s/t) * q_{0|t}(v), where q_{0|t} is the softmax of
    the logits with the mask token excluded (the substitution parameterisation of App. A.1: the
    model never predicts [MASK])."""
    z = np.asarray(logits_row, F64)
    q = np.zeros_like(z)
    if not is_masked:
        q[token] = 1.0
        return q
    zz = z.copy()
    zz[mask_id] = -np.inf
    p = np.exp(zz - zz[np.isfinite(zz)].max())
    p /= p.sum()
    q = (1.0 - keep_prob) * p
    q[mask_id] = keep_prob
    return q


def reverse_step(tokens, logits, u_keep, u_cat, keep_prob: float, mask_id: int):
    """One draw from Eq. 3 for every position, driven by two uniforms per position (inputs, so that the
    draw is a function): a masked position stays masked iff u_keep < s/t; otherwise its token is the
    inverse-CDF sample of q_{0|t} at u_cat: the first v (mask excluded) whose cumulative probability
    reaches u_cat.  tokens [B, L] int, logits [B, L, V], u_* [B, L] in [0, 1)."""
    tokens = np.asarray(tokens)
    out = tokens.copy()
    B, L = tokens.shape
    for b in range(B):
        for t in range(L):
            if tokens[b, t] != mask_id:
                continue                                   # case 1: carried over
            if np.float32(u_keep[b, t]) < np.float32(keep_prob):
                continue                                   # case 2: stays masked
            z = np.asarray(logits[b, t], F64).copy()
            z[mask_id] = -np.inf
            p = np.exp(z - z[np.isfinite(z)].max())
            cdf = np.cumsum(p)
            target = np.float64(u_cat[b, t]) * cdf[-1]
            v = int(np.searchsorted(cdf, target, side="right"))     # first v with cdf[v] > target
            v = min(v, len(cdf) - 1)
            while p[v] == 0.0:                             # u_cat == 0 with zero-probability leading entries
                v += 1
            out[b, t] = v
    return out


def noise_schedule(K: int, eps: float = 1e-3):
    """Noise levels of a K-step generation, t_0 = 1 > ... > t_K = eps (App. A.1: sampling eps 1e-3), uniformly
    spaced; step k goes from t_k to s = t_{k+1} and keeps a masked token masked with probability s / t_k
    (the last step, to eps, still leaves s / t of the masked tokens to a final clean-up pass with keep 0)."""
    t = 1.0 - (1.0 - eps) * np.arange(K + 1) / K
    return t


# --------------------------------------------------------------------------------------------
# The K-step generation loop around the reverse step (Sec. 2 Eq. 3, Sec. 4.3: K = L / p denoising steps)
# --------------------------------------------------------------------------------------------
def generation_keep_probs(K: int, eps: float = 1e-3):
    """keep probability s / t of each of the K scheduled steps (t_k -> t_{k+1} of noise_schedule), as the
    float32 values the decision `u_keep < s/t` is taken with, followed by 0 for the final clean-up pass
    that unmasks whatever is still masked at noise level eps."""
    t = noise_schedule(K, eps)
    return [np.float32(t[k + 1] / t[k]) for k in range(K)] + [np.float32(0.0)]


def generate(tokens, sw: dict, u_keep, u_cat, K: int, mask_id: int, vocab_real: int, *, eps: float = 1e-3, tau=None,
             return_trace: bool = False, **kw):
    """K reverse steps of Eq. 3 along noise_schedule(K, eps) plus the clean-up pass: step k runs the denoiser on
    the current tokens (denoise_step, or denoise_step_cond with tau[k] when tau [K+1, B, d_c] is given), then
    reverse_step with keep probability generation_keep_probs(K)[k] and the uniforms u_keep[k], u_cat[k]
    ([K+1, B, L] each).  Returns the final tokens (and the tokens after every step when return_trace)."""
    x = np.asarray(tokens).copy()
    trace = []
    for k, keep in enumerate(generation_keep_probs(K, eps)):
        logits = denoise_step(x, sw, **kw) if tau is None else denoise_step_cond(x, tau[k], sw, **kw)
        x = reverse_step(x, logits[..., :vocab_real], u_keep[k], u_cat[k], float(keep), mask_id)
        trace.append(x.copy())
    return (x, trace) if return_trace else x


# --------------------------------------------------------------------------------------------
# Bidirectional multi-head attention mixer of the hybrid variant (Sec. 3.3, App. C Transformer-layer table)
# --------------------------------------------------------------------------------------------
def attention_mixer(x, w_qkv, w_o, n_heads: int):
    """The hybrid's attention mixer: full (non-causal) multi-head self-attention over each sequence, no position
    encoding.  App. C counts it as QKV and output projections (8 d^2 FLOPs) plus QK^T and Attn.V (4 L d).
    x [B, L, d]; w_qkv [3 d, d] with rows [Q | K | V], each split into n_heads blocks of d / n_heads;
    w_o [d, d].  out = concat_h softmax(Q_h K_h^T / sqrt(d_h)) V_h  W_o^T."""
    x = np.asarray(x, F64)
    B, L, d = x.shape
    dh = d // n_heads
    qkv = x @ np.asarray(w_qkv, F64).T
    q, k, v = qkv[..., :d], qkv[..., d:2 * d], qkv[..., 2 * d:]
    out = np.zeros((B, L, d), F64)
    for b in range(B):
        for h in range(n_heads):
            sl = slice(h * dh, (h + 1) * dh)
            s = q[b, :, sl] @ k[b, :, sl].T / np.sqrt(dh)
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p /= p.sum(axis=1, keepdims=True)
            out[b, :, sl] = p @ v[b, :, sl]
    return out @ np.asarray(w_o, F64).T


def denoise_step_hybrid(tokens, sw: dict, *, attn_period: int, attn_heads: int, tau=None, rms_eps: float = 1e-5,
                        ln_eps: float = 1e-5, states_in=None, return_states: bool = False, **kw):
    """The hybrid stack (Sec. 3.3, App. A.3): the mixer of layer i is the attention mixer when i is a multiple of
    attn_period (one attention mixer followed by attn_period - 1 bidirectional Mamba mixers; the paper uses 5), the
    bidirectional Mamba mixer otherwise.  tau None: RMSNorm pre-norm + mixer + residual per layer; tau given: the
    timestep-conditioned block around either mixer.  Attention layers carry "w_qkv" and "w_o".
    Block mode (states_in given or return_states): every layer runs as a block step from its entry of states_in --
    (ssm, conv) for a Mamba layer, (k_cache, v_cache) for an attention layer, None for an empty prefix -- and the
    states after the block are returned in the same form."""
    block_mode = states_in is not None or return_states
    r = np.asarray(sw["embed"], F64)[np.asarray(tokens)]
    states_out = []
    for i, layer in enumerate(sw["layers"]):
        is_attn = attn_period > 0 and i % attn_period == 0
        st = None if states_in is None else states_in[i]

        def mix(u, layer=layer, is_attn=is_attn, st=st):
            if is_attn:
                if not block_mode:
                    return attention_mixer(u, layer["w_qkv"], layer["w_o"], attn_heads)
                kc, vc = (None, None) if st is None else st
                y, k_all, v_all = attention_block_step(u, layer["w_qkv"], layer["w_o"], attn_heads, kc, vc)
                states_out.append((k_all, v_all))
                return y
            if not block_mode:
                return bimamba_forward(u, layer["fwd"], layer["rev"], **kw)
            s_in, c_in = (None, None) if st is None else st
            y, s_out, c_out = bimamba_block_step(u, layer["fwd"], layer["rev"], ssm_state_in=s_in, conv_state_in=c_in, **kw)
            states_out.append((s_out, c_out))
            return y

        if tau is None:
            r = r + mix(rmsnorm(r, layer["norm_w"], rms_eps))
        else:
            b1, s1, g1, b2, s2, g2 = modulation(tau, layer["w_cond"], layer.get("b_cond"))
            y = r + g1[:, None, :] * mix(adaln(r, s1, b1, ln_eps))
            r = y + g2[:, None, :] * mlp(adaln(y, s2, b2, ln_eps), layer["w_up"], layer["w_down"], layer.get("b_up"), layer.get("b_down"))
    logits = rmsnorm(r, sw["final_norm_w"], rms_eps) @ np.asarray(sw["w_vocab"], F64).T
    return (logits, states_out) if return_states else logits


def attention_block_step(x_blk, w_qkv, w_o, n_heads: int, k_cache=None, v_cache=None):
    """The attention mixer in block-autoregressive decoding (Sec. 4.3: the cache of a denoised block is kept and reused):
    the block's queries attend to the cached keys and values of the committed prefix and, without a mask, to the block
    itself.  k_cache, v_cache: [B, Lc, d] (None = empty prefix).  Returns (y_blk, k_all, v_all) with the block's keys and
    values appended, i.e. the cache a commit of this block would leave."""
    x = np.asarray(x_blk, F64)
    B, G, d = x.shape
    dh = d // n_heads
    qkv = x @ np.asarray(w_qkv, F64).T
    q, k, v = qkv[..., :d], qkv[..., d:2 * d], qkv[..., 2 * d:]
    if k_cache is not None:
        k = np.concatenate([np.asarray(k_cache, F64), k], axis=1)
        v = np.concatenate([np.asarray(v_cache, F64), v], axis=1)
    out = np.zeros((B, G, d), F64)
    for b in range(B):
        for h in range(n_heads):
            sl = slice(h * dh, (h + 1) * dh)
            s = q[b, :, sl] @ k[b, :, sl].T / np.sqrt(dh)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[b, :, sl] = p @ v[b, :, sl]
    return out @ np.asarray(w_o, F64).T, k, v
