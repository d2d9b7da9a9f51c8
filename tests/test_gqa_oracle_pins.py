"""Pins for the comparison-attention oracle (MHA / MQA / GQA): no GPU needed."""
import math

import numpy as np
import pytest
import torch

from oracle import gqa_oracle as G
from oracle import mtla_oracle as O


def make(seed=0, d=24, nh=4, g=2, dh=8):
    rng = np.random.default_rng(seed)
    w = dict(w_q=rng.standard_normal((d, nh * dh)) / math.sqrt(d),
             w_k=rng.standard_normal((d, g * dh)) / math.sqrt(d),
             w_v=rng.standard_normal((d, g * dh)) / math.sqrt(d),
             w_o=rng.standard_normal((nh * dh, d)) / math.sqrt(nh * dh))
    return G.params_from_tensors(dict(d_model=d, n_heads=nh, n_groups=g, head_dim=dh), w)


def xs(seed, t, d=24):
    return np.random.default_rng(100 + seed).standard_normal((t, d))


@pytest.mark.parametrize("g", [1, 2, 4])
def test_incremental_equals_dense(g):
    p = make(seed=g, g=g)
    x = xs(g, 19)
    inc, st = G.decode_sequence(p, x)
    assert st.tokens == 19
    np.testing.assert_allclose(inc, G.forward_dense(p, x), rtol=0, atol=1e-12)


@pytest.mark.parametrize("g", [1, 2, 4])
def test_dense_equals_torch_sdpa(g):
    """The library routine gets the oracle's rotated q, k: it pins softmax, mask, grouping, scale."""
    p = make(seed=10 + g, g=g)
    x = xs(3, 13)
    t_len, nh, dh = 13, p.n_heads, p.head_dim
    q = (x @ p.w_q).reshape(t_len, nh, dh)
    k = (x @ p.w_k).reshape(t_len, g, dh)
    v = (x @ p.w_v).reshape(t_len, g, dh)
    for m in range(t_len):
        q[m], k[m] = G.rotate(q[m], m, p.rope_theta), G.rotate(k[m], m, p.rope_theta)
    rep = nh // g
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(rep, dim=0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(rep, dim=0)[None]
    att = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0]
    want = att.permute(1, 0, 2).reshape(t_len, nh * dh).numpy() @ p.w_o
    np.testing.assert_allclose(G.forward_dense(p, x), want, rtol=0, atol=1e-12)


def test_mqa_by_hand():
    """One shared key/value head, two tokens, no rotation at position 0: written out."""
    p = make(seed=7, nh=2, g=1)
    x = xs(7, 2)
    y, _ = G.decode_sequence(p, x)
    # Token 1 sees only itself: softmax over one score is 1, so every head returns v_1.
    v1 = x[0] @ p.w_v
    np.testing.assert_allclose(y[0], np.concatenate([v1, v1]) @ p.w_o, atol=1e-12)
    # Token 2: two scores per head against the shared keys.
    k = np.stack([x[0] @ p.w_k, G.rotate(x[1] @ p.w_k, 1, p.rope_theta)])
    v = np.stack([x[0] @ p.w_v, x[1] @ p.w_v])
    q = G.rotate((x[1] @ p.w_q).reshape(2, p.head_dim), 1, p.rope_theta)
    heads = []
    for h in range(2):
        e = k @ q[h] / math.sqrt(p.head_dim)
        w = np.exp(e - e.max())
        heads.append((w / w.sum()) @ v)
    np.testing.assert_allclose(y[1], np.concatenate(heads) @ p.w_o, atol=1e-12)


def test_mha_heads_are_independent():
    """g = n_h: changing head 3's key weights leaves the other heads' outputs alone."""
    p = make(seed=8, d=32, nh=4, g=4)
    p.w_o = np.eye(32)
    x = xs(8, 9, d=32)
    base = G.forward_dense(p, x)
    p.w_k = p.w_k.copy()
    p.w_k[:, 3 * p.head_dim:] *= -1.7
    other = G.forward_dense(p, x)
    np.testing.assert_allclose(base[:, :3 * p.head_dim], other[:, :3 * p.head_dim], atol=1e-12)
    assert np.abs(base[:, 3 * p.head_dim:] - other[:, 3 * p.head_dim:]).max() > 1e-3


def test_rotation_depends_on_relative_position_only():
    rng = np.random.default_rng(5)
    a, b = rng.standard_normal(16), rng.standard_normal(16)
    d0 = G.rotate(a, 3, 10000.0) @ G.rotate(b, 11, 10000.0)
    d1 = G.rotate(a, 40, 10000.0) @ G.rotate(b, 48, 10000.0)
    assert abs(d0 - d1) < 1e-12
    np.testing.assert_allclose(G.rotate(a, 0, 10000.0), a)
    # Pair k turns by pos * theta^(-2k/d): the first pair by pos radians.
    r = G.rotate(np.array([1.0, 0.0, 1.0, 0.0]), 2, 10000.0)
    np.testing.assert_allclose(r, [math.cos(2), math.sin(2), math.cos(0.02), math.sin(0.02)], atol=1e-15)
    # The same convention as the MTLA oracle's decoupled RoPE (written independently).
    np.testing.assert_allclose(G.rotate(a, 9, 10000.0), O.rope(a, 9, 10000.0), atol=1e-14)


def test_cache_sizes_the_paper_states():
    """Section 4.3: MLA keeps 4.5 d_h elements per token, "GQA with 2.25 groups"; MTLA at s = 2
    is GQA with 1.125 groups, about MQA."""
    dh = 64
    assert G.cache_elements_per_token(8, dh) == 2 * 8 * dh           # MHA, n_h = 8
    assert G.cache_elements_per_token(1, dh) == 2 * dh               # MQA
    mla = 4 * dh + dh // 2                                           # r = 4 d_h, d_R = d_h / 2
    assert mla / G.cache_elements_per_token(1, dh) == 2.25
    assert (mla / 2) / G.cache_elements_per_token(1, dh) == 1.125


def test_cache_round_trip():
    p = make(seed=9, g=2)
    _, st = G.decode_sequence(p, xs(9, 6), rows=[])
    arr = G.cache_array(st)
    assert arr.shape == (2, 6, 2 * p.head_dim)
    st2 = G.state_from_cache(arr)
    x = xs(1, 1)[0]
    np.testing.assert_allclose(G.decode_step(p, st, x), G.decode_step(p, st2, x), atol=1e-14)


def test_planted_mistakes_are_caught():
    """A wrong group mapping (interleaved instead of contiguous) and a dropped rotation of the
    keys both fail the dense / library pins."""
    p = make(seed=12, nh=4, g=2)
    x = xs(12, 11)
    want = G.forward_dense(p, x)
    st = G.GQAState()
    ys = []
    for m, row in enumerate(x):
        pos = st.tokens
        st.keys.append(G.rotate((row @ p.w_k).reshape(2, p.head_dim), pos, p.rope_theta))
        st.values.append((row @ p.w_v).reshape(2, p.head_dim))
        q = G.rotate((row @ p.w_q).reshape(4, p.head_dim), pos, p.rope_theta)
        keys, values = np.stack(st.keys), np.stack(st.values)
        heads = []
        for h in range(4):
            grp = h % 2                                  # the mistake
            e = keys[:, grp, :] @ q[h] / math.sqrt(p.head_dim)
            w = np.exp(e - e.max())
            heads.append((w / w.sum()) @ values[:, grp, :])
        ys.append(np.concatenate(heads) @ p.w_o)
    assert np.abs(np.stack(ys) - want).max() > 1e-3
