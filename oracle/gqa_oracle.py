"""CPU oracle for the comparison attentions of the paper's Section 3: multi-head (MHA),
multi-query (MQA) and grouped-query (GQA) attention with a key-value cache.  TEST
INFRASTRUCTURE ONLY: the tests and the benchmark's CPU leg import it, the product path never
does, and it shares no code with the CUDA library (nor with the MTLA oracle).

Plain fp64 numpy, two formulations that are checked against each other:

  incremental   one token at a time over cached keys and values (Section 3, "Key-Value Cache in
                Auto-regressive Inference"): q_i from x_i, softmax(q_i K^T / sqrt(d_h)) V;
  dense         all T rows at once with a causal mask.

One definition covers the three methods: g groups of heads, each group sharing one key head and
one value head (Section 3: MHA is g = n_h, MQA is g = 1).  Query head h belongs to group
h // (n_h / g).  Positions enter through standard rotary embedding of queries and keys (the
paper's appendix: "Standard RoPE is used in MHA").

Readings of points the paper leaves open:
  * RoPE rotates adjacent pairs (2k, 2k+1) of each head by pos * theta^(-2k/d_h), pos = i - 1
    for the 1-based token i, theta = 10000 - the same convention as the MTLA oracle's
    decoupled RoPE, so that the comparison differs only in what the paper says differs.
  * The score scale is 1/sqrt(d_h) per head (the background section writes sqrt(d) for a single
    head of width d).
  * The token attends to itself and everything before it: its key and value are appended
    before the scores are formed, like MTLA's own slot update.
  * No biases, no dropout.

Parity pins (tests/test_gqa_oracle_pins.py): incremental against dense; dense against torch's
scaled_dot_product_attention with a causal mask (a library routine); MQA / MHA special cases
written out by hand; RoPE's relative-position property; the paper's cache-size statements
(2 n_h d_h, 2 d_h, 2 g d_h elements per token; MLA's 4.5 d_h = GQA with 2.25 groups).
Parity unpinned: the RoPE pairing and base (free conventions shared with the CUDA path).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass
class GQAParams:
    d_model: int
    n_heads: int          # n_h
    n_groups: int         # g: key / value heads (n_h: MHA, 1: MQA)
    head_dim: int         # d_h
    w_q: np.ndarray       # [d][n_h * d_h]
    w_k: np.ndarray       # [d][g * d_h]
    w_v: np.ndarray       # [d][g * d_h]
    w_o: np.ndarray       # [n_h * d_h][d]
    rope_theta: float = 10000.0


@dataclass
class GQAState:
    """Per-sequence cache: one [g][d_h] key array and one value array per token."""
    keys: list = field(default_factory=list)
    values: list = field(default_factory=list)

    @property
    def tokens(self) -> int:
        return len(self.keys)


def params_from_tensors(dims: dict, weights: dict, **kw) -> GQAParams:
    return GQAParams(**dims, **{k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}, **kw)


def rotate(v: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Standard rotary embedding of the last axis at position pos."""
    half = v.shape[-1] // 2
    freq = theta ** (-np.arange(half, dtype=np.float64) / half)
    c, s = np.cos(pos * freq), np.sin(pos * freq)
    even, odd = v[..., 0::2], v[..., 1::2]
    out = np.empty_like(v, dtype=np.float64)
    out[..., 0::2] = even * c - odd * s
    out[..., 1::2] = odd * c + even * s
    return out


def _softmax(e: np.ndarray) -> np.ndarray:
    z = np.exp(e - e.max(axis=-1, keepdims=True))
    return z / z.sum(axis=-1, keepdims=True)


def decode_step(p: GQAParams, st: GQAState, x: np.ndarray, want_output: bool = True):
    """Consume token x [d]: append its key and value, return y [d] (or None)."""
    x = np.asarray(x, dtype=np.float64)
    pos = st.tokens
    st.keys.append(rotate((x @ p.w_k).reshape(p.n_groups, p.head_dim), pos, p.rope_theta))
    st.values.append((x @ p.w_v).reshape(p.n_groups, p.head_dim))
    if not want_output:
        return None
    q = rotate((x @ p.w_q).reshape(p.n_heads, p.head_dim), pos, p.rope_theta)
    keys, values = np.stack(st.keys), np.stack(st.values)          # [T][g][d_h]
    per_group = p.n_heads // p.n_groups
    heads = []
    for h in range(p.n_heads):
        grp = h // per_group
        e = keys[:, grp, :] @ q[h] / np.sqrt(p.head_dim)
        heads.append(_softmax(e) @ values[:, grp, :])
    return np.concatenate(heads) @ p.w_o


def decode_sequence(p: GQAParams, xs: np.ndarray, st: GQAState | None = None, rows=None):
    st = GQAState() if st is None else st
    wanted = None if rows is None else set(int(m) for m in rows)
    ys = []
    for m, x in enumerate(np.asarray(xs, dtype=np.float64)):
        y = decode_step(p, st, x, want_output=wanted is None or m in wanted)
        if y is not None:
            ys.append(y)
    return (np.stack(ys) if ys else np.zeros((0, p.d_model))), st


def forward_dense(p: GQAParams, xs: np.ndarray) -> np.ndarray:
    """All rows at once under a causal mask (row m sees columns n <= m)."""
    xs = np.asarray(xs, dtype=np.float64)
    t_len = xs.shape[0]
    q = (xs @ p.w_q).reshape(t_len, p.n_heads, p.head_dim)
    k = (xs @ p.w_k).reshape(t_len, p.n_groups, p.head_dim)
    v = (xs @ p.w_v).reshape(t_len, p.n_groups, p.head_dim)
    for m in range(t_len):
        q[m] = rotate(q[m], m, p.rope_theta)
        k[m] = rotate(k[m], m, p.rope_theta)
    mask = np.where(np.tril(np.ones((t_len, t_len), dtype=bool)), 0.0, -np.inf)
    per_group = p.n_heads // p.n_groups
    out = np.empty((t_len, p.n_heads * p.head_dim))
    for h in range(p.n_heads):
        grp = h // per_group
        e = q[:, h, :] @ k[:, grp, :].T / np.sqrt(p.head_dim) + mask
        out[:, h * p.head_dim:(h + 1) * p.head_dim] = _softmax(e) @ v[:, grp, :]
    return out @ p.w_o


def state_from_cache(cache: np.ndarray) -> GQAState:
    """State from a stored cache [g][T][2 d_h] (value then key per row, the library's layout)."""
    cache = np.asarray(cache, dtype=np.float64)
    dh = cache.shape[2] // 2
    return GQAState(keys=[cache[:, t, dh:].copy() for t in range(cache.shape[1])],
                    values=[cache[:, t, :dh].copy() for t in range(cache.shape[1])])


def cache_array(st: GQAState) -> np.ndarray:
    """The cache as [g][T][2 d_h], value then key per row."""
    return np.concatenate([np.stack(st.values), np.stack(st.keys)], axis=2).transpose(1, 0, 2)


def cache_elements_per_token(n_groups: int, head_dim: int) -> int:
    """Section 3 / Section 4.3: 2 g d_h key-value elements per token and layer."""
    return 2 * n_groups * head_dim
