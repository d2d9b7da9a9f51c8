"""CPU oracle for Multi-head Temporal Latent Attention (MTLA): TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy statement of what the paper's attention module computes,
written from the paper's Section 4 and sharing no code with the CUDA library.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it; the product
path never does.

Three independent formulations live here so that they can be checked against each other:

  Form I    incremental decoding, one token at a time (Section 4.1, Eq. 13, and the cache
            update rules of Sections 4.1 and 4.3), attention in the un-absorbed form
            (Eq. 9-11) with the decoupled-RoPE score term of Eq. 17;
  Form II   the dense parallel form of Section 4.2 (Eq. 14-16): T x T merge-weight matrix
            with chunk mask, stride-aware causal mask, un-compressed RoPE keys;
  Form III  plain multi-head latent attention (Eq. 5-6 with decoupled RoPE), which MTLA
            must equal at s = 1.

Readings of points the paper leaves open (each is a documented convention):
  * Eq. 13's product of the two Linear outputs is an inner product over the hyper-network
    width, giving one scalar weight per token (Eq. 16 writes the same quantity as a matrix
    product).  No extra scaling.
  * A new slot opens when (i - 1) mod s == 0 for the 1-based token index i, so that the
    cache holds ceil(i / s) slots (Section 4).
  * The stride-aware mask uses 1-based row/column indices (Section 4.2).
  * pe_j is the sinusoidal embedding of dimension r at the 1-based slot number j.
  * LayerNorm is affine, biased variance, eps inside the square root.
  * RoPE keys come from the token itself: k^R_i = RoPE_i(x_i W_KR), one head shared by
    all query heads; RoPE rotates adjacent pairs (2k, 2k+1) by pos * theta^(-2k/d_R),
    pos = i - 1.
  * The score scale is 1/sqrt(d_h) as printed in Eq. 17.
  * At s = 1 nothing is merged: the hyper-network is skipped and w = 1.

Parity pins: tests/test_oracle_pins.py checks Form I against Form II, Form I(s=1)
against Form III, the paper's worked merge example, closed forms (uniform attention,
single slot, zero hyper-network => w = 1/2), slot counts and RoPE shift invariance;
reorder_states against hypotheses decoded one by one from their full token histories.
Parity unpinned (free conventions the paper does not fix, shared with the CUDA path):
the sinusoid's exact form, LayerNorm eps, the RoPE pairing, bias presence.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass
class Params:
    """Dimensions (paper's notation) and fp64 weights, row-major [in][out]."""
    d_model: int
    n_heads: int
    head_dim: int
    latent_rank: int
    rope_dim: int
    hyper_dim: int
    stride: int
    w_q: np.ndarray        # [d][n_h*d_h]            Eq. 7
    w_qr: np.ndarray       # [d][n_h*d_R]            Section 4.3
    w_r: np.ndarray        # [d][r]                  Eq. 8
    w_kr: np.ndarray       # [d][d_R]                Section 4.3
    ln_gamma: np.ndarray   # [r]
    ln_beta: np.ndarray    # [r]
    w_k: np.ndarray        # [r][n_h*d_h]            Eq. 9
    w_v: np.ndarray        # [r][n_h*d_h]            Eq. 10
    w_o: np.ndarray        # [n_h*d_h][d]            Eq. 11
    hyp_c_w: np.ndarray    # [r][d_w]                Eq. 13, Linear(c_i)
    hyp_c_b: np.ndarray    # [d_w]
    hyp_pe_w: np.ndarray   # [r][d_w]                Eq. 13, Linear(pe_j)
    hyp_pe_b: np.ndarray   # [d_w]
    ln_eps: float = 1e-5
    rope_theta: float = 10000.0
    gate_at_stride_one: bool = False   # True: apply Eq. 13 even at s = 1 (secondary identity)


@dataclass
class State:
    """Per-sequence decoding state: the compressed caches and the token count."""
    c_hat: list = field(default_factory=list)    # slots, each [r]      (Section 4.1)
    kr_hat: list = field(default_factory=list)   # slots, each [d_R]    (Section 4.3)
    tokens: int = 0

    @property
    def n_slots(self) -> int:
        return len(self.c_hat)


def params_from_tensors(dims: dict, weights: dict, **kw) -> Params:
    """Build Params from a dict of array-likes (anything np.asarray(.., float64) accepts)."""
    arrays = {k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}
    return Params(**dims, **arrays, **kw)


# ----------------------------------------------------------------------------- pieces

def layer_norm(c_raw: np.ndarray, p: Params) -> np.ndarray:
    """LayerNorm over the latent dimension (Section 4, after Eq. 8)."""
    mu = c_raw.mean(axis=-1, keepdims=True)
    var = ((c_raw - mu) ** 2).mean(axis=-1, keepdims=True)
    return (c_raw - mu) / np.sqrt(var + p.ln_eps) * p.ln_gamma + p.ln_beta


def sinusoid_pe(j: int, dim: int) -> np.ndarray:
    """Sinusoidal positional embedding of slot number j (1-based), Eq. 13's pe_j."""
    k = np.arange(dim // 2, dtype=np.float64)
    angle = j / (10000.0 ** (2.0 * k / dim))
    pe = np.zeros(dim, dtype=np.float64)
    pe[0::2] = np.sin(angle)
    pe[1::2] = np.cos(angle)
    return pe


def rope(v: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotate adjacent pairs of the last axis by the position-dependent angles (Section 4.3)."""
    dim = v.shape[-1]
    k = np.arange(dim // 2, dtype=np.float64)
    angle = pos * theta ** (-2.0 * k / dim)
    cos, sin = np.cos(angle), np.sin(angle)
    out = np.empty_like(v)
    out[..., 0::2] = v[..., 0::2] * cos - v[..., 1::2] * sin
    out[..., 1::2] = v[..., 0::2] * sin + v[..., 1::2] * cos
    return out


def merge_weight(c: np.ndarray, j: int, p: Params) -> float:
    """w_i = Sigmoid(<Linear(c_i), Linear(pe_j)>), Eq. 13 (j = ceil(i/s), 1-based)."""
    if p.stride == 1 and not p.gate_at_stride_one:
        return 1.0
    h = c @ p.hyp_c_w + p.hyp_c_b
    g = sinusoid_pe(j, p.latent_rank) @ p.hyp_pe_w + p.hyp_pe_b
    return float(1.0 / (1.0 + np.exp(-np.dot(h, g))))


def softmax(e: np.ndarray) -> np.ndarray:
    z = np.exp(e - e.max(axis=-1, keepdims=True))
    return z / z.sum(axis=-1, keepdims=True)


def attend(p: Params, q: np.ndarray, q_rope: np.ndarray, c_hat: np.ndarray,
           kr_hat: np.ndarray) -> np.ndarray:
    """One query against n cached slots: Eq. 9-11 with the RoPE term of Eq. 17.

    q [n_h*d_h], q_rope [n_h*d_R] (already rotated), c_hat [n][r], kr_hat [n][d_R].
    Returns y [d].
    """
    nh, dh, dr = p.n_heads, p.head_dim, p.rope_dim
    keys = c_hat @ p.w_k                         # [n][n_h*d_h]   Eq. 9
    values = c_hat @ p.w_v                       # [n][n_h*d_h]   Eq. 10
    heads = []
    for h in range(nh):
        k_h = keys[:, h * dh:(h + 1) * dh]
        v_h = values[:, h * dh:(h + 1) * dh]
        e = (k_h @ q[h * dh:(h + 1) * dh] + kr_hat @ q_rope[h * dr:(h + 1) * dr]) / np.sqrt(dh)
        heads.append(softmax(e) @ v_h)
    return np.concatenate(heads) @ p.w_o         # Eq. 11


# ----------------------------------------------------------------------------- Form I

def decode_step(p: Params, st: State, x: np.ndarray, want_output: bool = True):
    """Consume token x [d] for one sequence, update its cache, return y [d] (Section 4.1).

    want_output=False performs only the cache update (used to reach a sampled step of a
    long sequence without paying for the attention of every earlier step).
    """
    x = np.asarray(x, dtype=np.float64)
    i = st.tokens + 1                            # the paper's 1-based token index
    j = -(-i // p.stride)                        # ceil(i / s)
    c = layer_norm(x @ p.w_r, p)                 # Eq. 8 + LayerNorm
    w = merge_weight(c, j, p)                    # Eq. 13
    k_rope = rope(x @ p.w_kr, i - 1, p.rope_theta)
    if (i - 1) % p.stride == 0:                  # a chunk starts: Concat
        st.c_hat.append(w * c)
        st.kr_hat.append(k_rope)
    else:                                        # fold into the open slot; keep the latest key
        st.c_hat[j - 1] = st.c_hat[j - 1] + w * c
        st.kr_hat[j - 1] = k_rope
    st.tokens = i
    if not want_output:
        return None
    q = x @ p.w_q                                # Eq. 7
    q_rope = rope((x @ p.w_qr).reshape(p.n_heads, p.rope_dim), i - 1, p.rope_theta).reshape(-1)
    return attend(p, q, q_rope, np.stack(st.c_hat), np.stack(st.kr_hat))


def decode_sequence(p: Params, xs: np.ndarray, st: State | None = None, rows=None):
    """Run Form I over xs [T][d]; returns (Y, final State).

    Y holds one output per token, or only those of the 0-based token indices in `rows`
    (in increasing order) when given.
    """
    st = State() if st is None else st
    wanted = None if rows is None else set(int(m) for m in rows)
    ys = []
    for m, x in enumerate(np.asarray(xs, dtype=np.float64)):
        y = decode_step(p, st, x, want_output=wanted is None or m in wanted)
        if y is not None:
            ys.append(y)
    return (np.stack(ys) if ys else np.zeros((0, p.d_model))), st


def reorder_states(states: list, parents) -> list:
    """Beam-search re-parenting: hypothesis b of the new beam continues old hypothesis
    parents[b].  The paper decodes with beam search; its cache rules (Sections 4.1, 4.3) are
    per sequence, so a forked hypothesis simply starts from a copy of its parent's caches and
    token count.  Every returned State owns its arrays: siblings never share storage."""
    return [State(c_hat=[v.copy() for v in states[q].c_hat],
                  kr_hat=[v.copy() for v in states[q].kr_hat], tokens=states[q].tokens)
            for q in (int(v) for v in parents)]


def state_from_cache(cache: np.ndarray, tokens: int, p: Params) -> State:
    """State holding an externally supplied cache [n_slots][r + d_R] after `tokens` tokens."""
    cache = np.asarray(cache, dtype=np.float64)
    assert cache.shape == (-(-tokens // p.stride), p.latent_rank + p.rope_dim)
    return State(c_hat=[row[: p.latent_rank].copy() for row in cache],
                 kr_hat=[row[p.latent_rank:].copy() for row in cache], tokens=tokens)


def cache_array(st: State) -> np.ndarray:
    """The cache as one array [n_slots][r + d_R] (latent then RoPE key per slot)."""
    return np.concatenate([np.stack(st.c_hat), np.stack(st.kr_hat)], axis=1)


# ----------------------------------------------------------------------------- Form II

def merge_matrix(p: Params, c: np.ndarray) -> np.ndarray:
    """Chunk-masked T x T merge weights of Eq. 16: row m, column n (0-based here)."""
    t_len = c.shape[0]
    slot_of = np.arange(t_len) // p.stride                      # ceil(m/s) - 1 for 1-based m
    if p.stride == 1 and not p.gate_at_stride_one:
        w = np.ones((t_len, t_len))
    else:
        pe = np.stack([sinusoid_pe(j + 1, p.latent_rank) for j in slot_of])   # Eq. 15
        g = pe @ p.hyp_pe_w + p.hyp_pe_b
        h = c @ p.hyp_c_w + p.hyp_c_b
        w = 1.0 / (1.0 + np.exp(-(g @ h.T)))                    # Eq. 16
    same_chunk = slot_of[:, None] == slot_of[None, :]
    not_future = np.arange(t_len)[None, :] <= np.arange(t_len)[:, None]
    return np.where(same_chunk & not_future, w, 0.0)


def stride_aware_mask(t_len: int, s: int) -> np.ndarray:
    """Boolean T x T: True where attention is allowed (Section 4.2), 1-based m, n."""
    m = np.arange(1, t_len + 1)[:, None]
    n = np.arange(1, t_len + 1)[None, :]
    return (n == m) | ((n < m) & (n % s == 0))


def forward_dense(p: Params, xs: np.ndarray, rows=None) -> np.ndarray:
    """Form II over a whole sequence xs [T][d]; returns Y [T][d] (or only `rows`)."""
    xs = np.asarray(xs, dtype=np.float64)
    t_len = xs.shape[0]
    nh, dh, dr = p.n_heads, p.head_dim, p.rope_dim
    c = layer_norm(xs @ p.w_r, p)
    c_prime = merge_matrix(p, c) @ c                            # Eq. 14: running chunk sums
    k_rope = np.stack([rope(v, i, p.rope_theta) for i, v in enumerate(xs @ p.w_kr)])
    q = xs @ p.w_q
    q_rope = np.stack([rope(v.reshape(nh, dr), i, p.rope_theta).reshape(-1)
                       for i, v in enumerate(xs @ p.w_qr)])
    keys, values = c_prime @ p.w_k, c_prime @ p.w_v
    allowed = stride_aware_mask(t_len, p.stride)
    rows = range(t_len) if rows is None else rows
    out = []
    for m in rows:
        heads = []
        for h in range(nh):
            e = (keys[:, h * dh:(h + 1) * dh] @ q[m, h * dh:(h + 1) * dh]
                 + k_rope @ q_rope[m, h * dr:(h + 1) * dr]) / np.sqrt(dh)
            e = np.where(allowed[m], e, -np.inf)
            heads.append(softmax(e) @ values[:, h * dh:(h + 1) * dh])
        out.append(np.concatenate(heads) @ p.w_o)
    return np.stack(out)


# ----------------------------------------------------------------------------- Form III

def mla_forward(p: Params, xs: np.ndarray) -> np.ndarray:
    """Plain causal multi-head latent attention with decoupled RoPE (Eq. 5-6)."""
    xs = np.asarray(xs, dtype=np.float64)
    t_len = xs.shape[0]
    nh, dh, dr = p.n_heads, p.head_dim, p.rope_dim
    c = layer_norm(xs @ p.w_r, p)                               # Eq. 5
    keys, values = c @ p.w_k, c @ p.w_v                         # Eq. 6
    q = xs @ p.w_q
    pos = np.arange(t_len)
    ys = np.zeros((t_len, p.d_model))
    k_rope = np.stack([rope(v, i, p.rope_theta) for i, v in zip(pos, xs @ p.w_kr)])
    q_rope_all = xs @ p.w_qr
    causal = pos[None, :] <= pos[:, None]
    concat = np.zeros((t_len, nh * dh))
    for h in range(nh):
        qr_h = np.stack([rope(q_rope_all[i, h * dr:(h + 1) * dr], i, p.rope_theta) for i in pos])
        e = (q[:, h * dh:(h + 1) * dh] @ keys[:, h * dh:(h + 1) * dh].T + qr_h @ k_rope.T)
        e = np.where(causal, e / np.sqrt(dh), -np.inf)
        concat[:, h * dh:(h + 1) * dh] = softmax(e) @ values[:, h * dh:(h + 1) * dh]
    ys[:] = concat @ p.w_o
    return ys


# ----------------------------------------------------------------------------- accounting

def cache_slots(tokens: int, stride: int) -> int:
    """Slots held after `tokens` tokens: ceil(T / s) (Section 4)."""
    return -(-tokens // stride)


def cache_elements(tokens: int, p: Params, batch: int = 1) -> int:
    """Cache elements in use: one latent (r) and one RoPE key (d_R) per slot."""
    return batch * cache_slots(tokens, p.stride) * (p.latent_rank + p.rope_dim)
