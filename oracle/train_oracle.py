"""CPU oracle for MTLA's training path (Section 4.2): the dense parallel forward and its
backward.  TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU leg may
import it, the product path never does.  Plain fp64 numpy, sharing no code with the CUDA library.

Forward, for one sequence X [T][d], in the paper's order (Eq. 14-16, the stride-aware mask, and
the RoPE shortcut of Section 4.3):

    C   = LayerNorm(X W_r)                                      Eq. 8
    W   = Sigmoid(Linear(PE) x Linear(C)) in R^{T x T}          Eq. 15-16, PE = pe_j repeated s times
    C'  = (W o chunk mask) C                                    Eq. 14: every chunk's running sums
    K   = C' W_K,  V = C' W_V                                   Eq. 9-10 on C'
    E_h = (Q_h K_h^T + Q^R_h K^R^T) / sqrt(d_h) + M             Eq. 17 with the un-compressed K^R,
                                                                M the stride-aware causal mask
    Y   = concat_h(softmax(E_h) V_h) W_O                        Eq. 11

It is the same arithmetic as mtla_oracle.forward_dense (which the pins tie to the incremental
form); this file keeps the intermediates and adds the reverse pass: given dL/dY it returns dL/dX
and the gradient of every parameter, each step the transpose of the forward step above (softmax,
masked products, sigmoid gate, LayerNorm, rotations by the negative angle).

Parity pins (tests/test_train_oracle_pins.py): the forward against mtla_oracle.forward_dense;
every gradient against central finite differences of mtla_oracle.forward_dense (a function this
file does not define) along random directions; at s = 1 the hyper-network receives exactly zero
gradient; sequences of a batch do not mix; planted mistakes (a dropped term of the LayerNorm
backward, a forgotten chunk mask, the rotation not inverted) must fail the finite-difference pin.
Readings: those of mtla_oracle.py, nothing new.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from oracle import mtla_oracle as O

PARAM_NAMES = ("w_q", "w_qr", "w_r", "w_kr", "ln_gamma", "ln_beta", "w_k", "w_v", "w_o",
               "hyp_c_w", "hyp_c_b", "hyp_pe_w", "hyp_pe_b")


@dataclass
class Saved:
    """Intermediates of one sequence's forward pass that the backward pass reads."""
    xs: np.ndarray
    xhat: np.ndarray        # normalised latent before gain and bias [T][r]
    rstd: np.ndarray        # [T][1]
    c: np.ndarray           # [T][r]
    pe: np.ndarray          # [T][r] positional embedding of each row's chunk (None at s = 1)
    g: np.ndarray           # Linear(PE)  [T][d_w]
    h: np.ndarray           # Linear(C)   [T][d_w]
    w_gate: np.ndarray      # Sigmoid(g h^T) [T][T] before the chunk mask
    chunk: np.ndarray       # chunk mask [T][T] (0 / 1)
    c_prime: np.ndarray     # [T][r]
    q: np.ndarray           # [T][n_h d_h]
    q_rope: np.ndarray      # rotated [T][n_h d_R]
    k_rope: np.ndarray      # rotated [T][d_R]
    keys: np.ndarray        # [T][n_h d_h]
    values: np.ndarray
    probs: list             # per head [T][T]
    concat: np.ndarray      # [T][n_h d_h]


def chunk_mask(t_len: int, s: int) -> np.ndarray:
    """1 where row m and column n fall in the same chunk and n <= m (Section 4.2)."""
    idx = np.arange(t_len)
    same = (idx[:, None] // s) == (idx[None, :] // s)
    return (same & (idx[None, :] <= idx[:, None])).astype(np.float64)


def rotate_rows(v: np.ndarray, theta: float, sign: float = 1.0) -> np.ndarray:
    """Row i of v (last axis = RoPE dims) rotated by sign * the angles of position i."""
    return np.stack([O.rope(row, sign * i, theta) for i, row in enumerate(v)])


def forward(p: O.Params, xs: np.ndarray):
    """Dense training forward of one sequence; returns (Y [T][d], Saved)."""
    xs = np.asarray(xs, dtype=np.float64)
    t_len = xs.shape[0]
    nh, dh, dr = p.n_heads, p.head_dim, p.rope_dim
    c_raw = xs @ p.w_r
    mu = c_raw.mean(axis=-1, keepdims=True)
    var = ((c_raw - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + p.ln_eps)
    xhat = (c_raw - mu) * rstd
    c = xhat * p.ln_gamma + p.ln_beta
    chunk = chunk_mask(t_len, p.stride)
    gated = not (p.stride == 1 and not p.gate_at_stride_one)
    if gated:
        pe = np.stack([O.sinusoid_pe(m // p.stride + 1, p.latent_rank) for m in range(t_len)])   # Eq. 15
        g = pe @ p.hyp_pe_w + p.hyp_pe_b
        h = c @ p.hyp_c_w + p.hyp_c_b
        w_gate = 1.0 / (1.0 + np.exp(-(g @ h.T)))                                               # Eq. 16
    else:
        pe = g = h = None
        w_gate = np.ones((t_len, t_len))
    c_prime = (w_gate * chunk) @ c                                                              # Eq. 14
    q = xs @ p.w_q
    q_rope = rotate_rows((xs @ p.w_qr).reshape(t_len, nh, dr), p.rope_theta).reshape(t_len, nh * dr)
    k_rope = rotate_rows(xs @ p.w_kr, p.rope_theta)
    keys, values = c_prime @ p.w_k, c_prime @ p.w_v
    allowed = O.stride_aware_mask(t_len, p.stride)
    probs, heads = [], []
    for hd in range(nh):
        e = (q[:, hd * dh:(hd + 1) * dh] @ keys[:, hd * dh:(hd + 1) * dh].T
             + q_rope[:, hd * dr:(hd + 1) * dr] @ k_rope.T) / np.sqrt(dh)
        pr = O.softmax(np.where(allowed, e, -np.inf))
        probs.append(pr)
        heads.append(pr @ values[:, hd * dh:(hd + 1) * dh])
    concat = np.concatenate(heads, axis=1)
    y = concat @ p.w_o
    return y, Saved(xs, xhat, rstd, c, pe, g, h, w_gate, chunk, c_prime, q, q_rope, k_rope, keys,
                    values, probs, concat)


def backward(p: O.Params, sv: Saved, dy: np.ndarray):
    """Reverse pass of `forward` for one sequence: returns (dX [T][d], {parameter: gradient})."""
    dy = np.asarray(dy, dtype=np.float64)
    t_len = sv.xs.shape[0]
    nh, dh, dr = p.n_heads, p.head_dim, p.rope_dim
    grads = {}
    grads["w_o"] = sv.concat.T @ dy
    dconcat = dy @ p.w_o.T
    dq = np.zeros_like(sv.q)
    dq_rope = np.zeros_like(sv.q_rope)
    dk_rope = np.zeros_like(sv.k_rope)
    dkeys = np.zeros_like(sv.keys)
    dvalues = np.zeros_like(sv.values)
    for hd in range(nh):
        a, b = hd * dh, (hd + 1) * dh
        ar, br = hd * dr, (hd + 1) * dr
        pr = sv.probs[hd]
        do = dconcat[:, a:b]
        dvalues[:, a:b] = pr.T @ do
        dp = do @ sv.values[:, a:b].T
        de = pr * (dp - (dp * pr).sum(axis=-1, keepdims=True)) / np.sqrt(dh)     # softmax, then the scale
        dq[:, a:b] = de @ sv.keys[:, a:b]
        dkeys[:, a:b] = de.T @ sv.q[:, a:b]
        dq_rope[:, ar:br] = de @ sv.k_rope
        dk_rope += de.T @ sv.q_rope[:, ar:br]
    grads["w_k"] = sv.c_prime.T @ dkeys
    grads["w_v"] = sv.c_prime.T @ dvalues
    dc_prime = dkeys @ p.w_k.T + dvalues @ p.w_v.T
    # C' = (W o chunk) C
    dc = (sv.w_gate * sv.chunk).T @ dc_prime
    if sv.g is not None:
        dz = (dc_prime @ sv.c.T) * sv.chunk * sv.w_gate * (1.0 - sv.w_gate)       # through the sigmoid
        dg = dz @ sv.h
        dh_lin = dz.T @ sv.g
        grads["hyp_pe_w"] = sv.pe.T @ dg
        grads["hyp_pe_b"] = dg.sum(axis=0)
        grads["hyp_c_w"] = sv.c.T @ dh_lin
        grads["hyp_c_b"] = dh_lin.sum(axis=0)
        dc = dc + dh_lin @ p.hyp_c_w.T
    else:
        for name in ("hyp_pe_w", "hyp_pe_b", "hyp_c_w", "hyp_c_b"):
            grads[name] = np.zeros_like(getattr(p, name))
    # LayerNorm
    grads["ln_gamma"] = (dc * sv.xhat).sum(axis=0)
    grads["ln_beta"] = dc.sum(axis=0)
    dxhat = dc * p.ln_gamma
    dc_raw = (dxhat - dxhat.mean(axis=-1, keepdims=True)
              - sv.xhat * (dxhat * sv.xhat).mean(axis=-1, keepdims=True)) * sv.rstd
    grads["w_r"] = sv.xs.T @ dc_raw
    dx = dc_raw @ p.w_r.T
    # Rotations are orthogonal: the gradient of the un-rotated projection is the rotated-back one.
    dqr_raw = rotate_rows(dq_rope.reshape(t_len, nh, dr), p.rope_theta, -1.0).reshape(t_len, nh * dr)
    dkr_raw = rotate_rows(dk_rope, p.rope_theta, -1.0)
    grads["w_qr"] = sv.xs.T @ dqr_raw
    grads["w_kr"] = sv.xs.T @ dkr_raw
    grads["w_q"] = sv.xs.T @ dq
    dx = dx + dqr_raw @ p.w_qr.T + dkr_raw @ p.w_kr.T + dq @ p.w_q.T
    return dx, grads


def forward_backward_batch(p: O.Params, xs: np.ndarray, dy: np.ndarray):
    """A batch X [B][T][d] with dL/dY [B][T][d]: sequences are independent in the forward pass,
    so dX is per sequence and the parameter gradients are the sums over the batch.
    Returns (Y, dX, grads)."""
    ys, dxs, total = [], [], None
    for x, d in zip(xs, dy):
        y, sv = forward(p, x)
        dx, grads = backward(p, sv, d)
        ys.append(y)
        dxs.append(dx)
        total = grads if total is None else {k: total[k] + grads[k] for k in grads}
    return np.stack(ys), np.stack(dxs), total
