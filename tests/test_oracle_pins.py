"""Pins for the CPU oracle: everything here runs without a GPU.

Each test ties the oracle to something other than itself: the paper's worked example,
a second formulation of the same quantity (incremental vs dense masked vs plain MLA),
a library routine (torch LayerNorm / scaled_dot_product_attention), a closed form, or an
invariant.  The mutation tests at the end plant a plausible mistake in the oracle (on
the CPU) and check that the pins notice.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import mtla_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make_params(seed=0, s=2, d=16, nh=2, dh=8, r=8, dr=4, dw=4, **kw):
    rng = np.random.default_rng(seed)

    def mat(a, b):
        return rng.standard_normal((a, b)) / math.sqrt(a)

    weights = dict(
        w_q=mat(d, nh * dh), w_qr=mat(d, nh * dr), w_r=mat(d, r), w_kr=mat(d, dr),
        ln_gamma=1 + 0.1 * rng.standard_normal(r), ln_beta=0.1 * rng.standard_normal(r),
        w_k=mat(r, nh * dh), w_v=mat(r, nh * dh), w_o=mat(nh * dh, d),
        hyp_c_w=mat(r, dw), hyp_c_b=0.1 * rng.standard_normal(dw),
        hyp_pe_w=mat(r, dw), hyp_pe_b=0.1 * rng.standard_normal(dw))
    dims = dict(d_model=d, n_heads=nh, head_dim=dh, latent_rank=r, rope_dim=dr, hyper_dim=dw,
                stride=s)
    return O.params_from_tensors(dims, weights, **kw)


def inputs(seed, t_len, d=16):
    return np.random.default_rng(1000 + seed).standard_normal((t_len, d))


# ------------------------------------------------------------------ two formulations agree

@pytest.mark.parametrize("s", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("t_len", [1, 7, 12, 33])
def test_incremental_equals_dense_masked(s, t_len):
    """Section 4.2: the stride-aware mask makes the parallel form match decoding."""
    p = make_params(seed=s, s=s)
    xs = inputs(s * 100 + t_len, t_len)
    y_inc, st = O.decode_sequence(p, xs)
    y_dense = O.forward_dense(p, xs)
    assert st.n_slots == math.ceil(t_len / s)
    np.testing.assert_allclose(y_inc, y_dense, rtol=0, atol=1e-10)


def test_sampled_rows_equal_full_run():
    p = make_params(seed=3, s=3)
    xs = inputs(5, 20)
    y_all, _ = O.decode_sequence(p, xs)
    rows = [0, 4, 5, 19]
    y_rows, st = O.decode_sequence(p, xs, rows=rows)
    np.testing.assert_array_equal(y_rows, y_all[rows])
    np.testing.assert_array_equal(O.forward_dense(p, xs, rows=rows), O.forward_dense(p, xs)[rows])
    assert st.tokens == 20


@pytest.mark.parametrize("t_len", [1, 9, 24])
def test_stride_one_is_plain_mla(t_len):
    """s = 1 merges nothing, so MTLA must reduce to MLA (Eq. 5-6)."""
    p = make_params(seed=7, s=1)
    xs = inputs(t_len, t_len)
    y_inc, _ = O.decode_sequence(p, xs)
    np.testing.assert_allclose(y_inc, O.mla_forward(p, xs), rtol=0, atol=1e-10)


def test_mla_matches_torch_sdpa():
    """Form III against a library attention: heads see [q | q^R] . [k | k^R], scale 1/sqrt(d_h)."""
    p = make_params(seed=11, s=1)
    xs = inputs(2, 10)
    t_len, nh, dh, dr = 10, p.n_heads, p.head_dim, p.rope_dim
    X = torch.from_numpy(xs)
    c = torch.nn.functional.layer_norm(X @ torch.from_numpy(p.w_r), (p.latent_rank,),
                                       torch.from_numpy(p.ln_gamma),
                                       torch.from_numpy(p.ln_beta), p.ln_eps)
    k = (c @ torch.from_numpy(p.w_k)).reshape(t_len, nh, dh)
    v = (c @ torch.from_numpy(p.w_v)).reshape(t_len, nh, dh)
    q = (X @ torch.from_numpy(p.w_q)).reshape(t_len, nh, dh)

    def rot(a, pos):  # rotation written with complex numbers: (a0 + i a1) * exp(i * angle)
        z = torch.view_as_complex(a.reshape(*a.shape[:-1], -1, 2).contiguous())
        kk = torch.arange(a.shape[-1] // 2, dtype=torch.float64)
        ang = pos * p.rope_theta ** (-2 * kk / a.shape[-1])
        return torch.view_as_real(z * torch.polar(torch.ones_like(ang), ang)).reshape(a.shape)

    qr = torch.stack([rot((X[i] @ torch.from_numpy(p.w_qr)).reshape(nh, dr), i)
                      for i in range(t_len)])
    kr = torch.stack([rot(X[i] @ torch.from_numpy(p.w_kr), i) for i in range(t_len)])
    q_cat = torch.cat([q, qr], dim=-1).transpose(0, 1)                       # [nh][T][dh+dr]
    k_cat = torch.cat([k, kr[:, None, :].expand(t_len, nh, dr)], dim=-1).transpose(0, 1)
    out = torch.nn.functional.scaled_dot_product_attention(
        q_cat[None], k_cat[None], v.transpose(0, 1)[None], is_causal=True,
        scale=1.0 / math.sqrt(dh))[0]
    y = out.transpose(0, 1).reshape(t_len, nh * dh) @ torch.from_numpy(p.w_o)
    np.testing.assert_allclose(O.mla_forward(p, xs), y.numpy(), rtol=0, atol=1e-10)


# ------------------------------------------------------------------ the paper's worked example

def read_merge_example():
    slots, temp, stride = {}, [], None
    for line in open(os.path.join(GOLDEN, "merge_example_s2.txt")):
        tok = line.split("#")[0].split()
        if not tok:
            continue
        if tok[0] == "stride":
            stride = int(tok[1])
        elif tok[0] == "slot":
            slots[int(tok[1])] = [int(v) for v in tok[3:]]
        elif tok[0] == "temporary_steps":
            temp = [int(v) for v in tok[1:]]
    return stride, slots, temp


def test_worked_merge_example():
    """Section 4: c_hat_1 = w_1 c_1 + w_2 c_2, c_hat_2 = w_3 c_3 + w_4 c_4 at s = 2."""
    stride, slots, temp = read_merge_example()
    p = make_params(seed=5, s=stride)
    xs = inputs(9, 6)
    c = torch.nn.functional.layer_norm(
        torch.from_numpy(xs @ p.w_r), (p.latent_rank,), torch.from_numpy(p.ln_gamma),
        torch.from_numpy(p.ln_beta), p.ln_eps).numpy()
    st = O.State()
    opened_at = []
    for i, x in enumerate(xs, start=1):
        before = st.n_slots
        O.decode_step(p, st, x)
        if st.n_slots > before:
            opened_at.append(i)
    # a slot is still open (temporary) at step i iff i is not the last token of its chunk
    assert [i for i in range(1, 7) if i % stride != 0] == temp
    assert opened_at == [min(v) for v in slots.values()] + [5]
    for j, members in slots.items():
        w = [O.merge_weight(c[i - 1], j, p) for i in members]
        expect = sum(wi * c[i - 1] for wi, i in zip(w, members))
        np.testing.assert_allclose(st.c_hat[j - 1], expect, rtol=0, atol=1e-12)
        assert all(0.0 < wi < 1.0 for wi in w)


def test_zero_hypernetwork_gives_half_sums():
    """With the hyper-network zeroed, w = sigmoid(0) = 1/2 and each slot is half its chunk's sum."""
    p = make_params(seed=2, s=3)
    for name in ("hyp_c_w", "hyp_c_b", "hyp_pe_w", "hyp_pe_b"):
        setattr(p, name, np.zeros_like(getattr(p, name)))
    xs = inputs(4, 8)
    _, st = O.decode_sequence(p, xs)
    c = torch.nn.functional.layer_norm(
        torch.from_numpy(xs @ p.w_r), (p.latent_rank,), torch.from_numpy(p.ln_gamma),
        torch.from_numpy(p.ln_beta), p.ln_eps).numpy()
    np.testing.assert_allclose(st.c_hat[0], 0.5 * c[0:3].sum(0), atol=1e-12)
    np.testing.assert_allclose(st.c_hat[1], 0.5 * c[3:6].sum(0), atol=1e-12)
    np.testing.assert_allclose(st.c_hat[2], 0.5 * c[6:8].sum(0), atol=1e-12)   # open slot


def test_merge_weight_depends_on_slot_position_and_latent():
    p = make_params(seed=8, s=2)
    c = np.random.default_rng(0).standard_normal(p.latent_rank)
    w1, w2 = O.merge_weight(c, 1, p), O.merge_weight(c, 2, p)
    assert w1 != w2
    h = c @ p.hyp_c_w + p.hyp_c_b
    g = O.sinusoid_pe(2, p.latent_rank) @ p.hyp_pe_w + p.hyp_pe_b
    assert w2 == pytest.approx(float(torch.sigmoid(torch.tensor(float(h @ g), dtype=torch.float64))))


def test_rope_key_cache_keeps_latest_key_of_chunk():
    """Section 4.3: slot j holds the RoPE key of the most recent token of its chunk."""
    p = make_params(seed=4, s=3)
    xs = inputs(6, 8)
    _, st = O.decode_sequence(p, xs)
    for j, last in enumerate([2, 5, 7]):            # 0-based last token of each chunk so far
        np.testing.assert_allclose(st.kr_hat[j], O.rope(xs[last] @ p.w_kr, last, p.rope_theta),
                                   atol=1e-12)


# ------------------------------------------------------------------ mask and accounting

@pytest.mark.parametrize("s", [1, 2, 3, 4])
def test_mask_rows_admit_ceil_m_over_s_columns(s):
    allowed = O.stride_aware_mask(13, s)
    for m in range(1, 14):
        cols = [n for n in range(1, 14) if allowed[m - 1, n - 1]]
        assert len(cols) == math.ceil(m / s)                    # = cache length at step m
        assert cols == sorted(set([n for n in range(s, m, s)] + [m]))


def test_cache_accounting_matches_paper():
    for line in open(os.path.join(GOLDEN, "cache_accounting.txt")):
        tok = line.split("#")[0].split()
        if not tok:
            continue
        dh, s, per_slot, per_token = (int(v) for v in tok)
        p = make_params(s=s, dh=dh, r=4 * dh, dr=dh // 2, d=8, nh=1, dw=2)
        assert O.cache_elements(s, p) == per_slot
        assert per_slot == 9 * dh // 2
        tokens = 40 * s
        assert O.cache_elements(tokens, p) / tokens == per_token == 9 * dh / (2 * s)
    for t_len in range(0, 23):
        for s in (1, 2, 3, 4, 5):
            assert O.cache_slots(t_len, s) == math.ceil(t_len / s)


# ------------------------------------------------------------------ closed forms

def test_uniform_attention_closed_form():
    """W_Q = W_QR = 0 makes every score 0: y is the slot mean pushed through W_V W_O."""
    p = make_params(seed=6, s=2)
    p.w_q = np.zeros_like(p.w_q)
    p.w_qr = np.zeros_like(p.w_qr)
    xs = inputs(3, 9)
    ys, st = O.decode_sequence(p, xs)
    mean_slot = np.stack(st.c_hat).mean(0)
    np.testing.assert_allclose(ys[-1], mean_slot @ p.w_v @ p.w_o, atol=1e-12)


def test_single_slot_closed_form():
    """While only one slot exists (i <= s) the softmax is 1: y = c_hat_1 W_V W_O."""
    p = make_params(seed=9, s=4)
    xs = inputs(8, 3)
    st = O.State()
    for x in xs:
        y = O.decode_step(p, st, x)
        np.testing.assert_allclose(y, st.c_hat[0] @ p.w_v @ p.w_o, atol=1e-12)


def test_absorbed_form_identity():
    """Eq. 12/17: absorbing W_K into the query and W_V into the output changes nothing."""
    p = make_params(seed=10, s=2)
    xs = inputs(12, 11)
    ys, st = O.decode_sequence(p, xs)
    x = xs[-1]
    nh, dh, dr, r = p.n_heads, p.head_dim, p.rope_dim, p.latent_rank
    c_hat, kr_hat = np.stack(st.c_hat), np.stack(st.kr_hat)
    q = (x @ p.w_q).reshape(nh, dh)
    q_abs = np.einsum("hj,rhj->hr", q, p.w_k.reshape(r, nh, dh))          # x (W_Q W_K^T)
    qr = O.rope((x @ p.w_qr).reshape(nh, dr), 10, p.rope_theta)
    e = (q_abs @ c_hat.T + qr @ kr_hat.T) / math.sqrt(dh)
    o = torch.softmax(torch.from_numpy(e), dim=-1).numpy() @ c_hat        # [nh][r]
    y = np.einsum("hr,rhj->hj", o, p.w_v.reshape(r, nh, dh)).reshape(-1) @ p.w_o
    np.testing.assert_allclose(ys[-1], y, atol=1e-10)


def test_layer_norm_matches_torch():
    p = make_params(seed=12)
    a = np.random.default_rng(3).standard_normal((5, p.latent_rank)) * 3 + 1
    ref = torch.nn.functional.layer_norm(torch.from_numpy(a), (p.latent_rank,),
                                         torch.from_numpy(p.ln_gamma),
                                         torch.from_numpy(p.ln_beta), p.ln_eps).numpy()
    np.testing.assert_allclose(O.layer_norm(a, p), ref, atol=1e-12)


# ------------------------------------------------------------------ RoPE and sinusoid

def test_rope_properties():
    rng = np.random.default_rng(0)
    a, b = rng.standard_normal(8), rng.standard_normal(8)
    np.testing.assert_array_equal(O.rope(a, 0, 10000.0), a)                       # identity at 0
    assert np.linalg.norm(O.rope(a, 37, 10000.0)) == pytest.approx(np.linalg.norm(a))
    base = O.rope(a, 5, 10000.0) @ O.rope(b, 2, 10000.0)
    for shift in (1, 10, 1000):                                                   # relative only
        assert O.rope(a, 5 + shift, 10000.0) @ O.rope(b, 2 + shift, 10000.0) == pytest.approx(base)
    # first pair turns by exactly `pos` radians, the last by pos * theta^(-(d-2)/d)
    v = np.zeros(8)
    v[0] = 1.0
    np.testing.assert_allclose(O.rope(v, 3, 10000.0)[:2], [math.cos(3), math.sin(3)], atol=1e-15)
    v = np.zeros(8)
    v[6] = 1.0
    ang = 3 * 10000.0 ** (-6 / 8)
    np.testing.assert_allclose(O.rope(v, 3, 10000.0)[6:], [math.cos(ang), math.sin(ang)], atol=1e-15)


def test_outputs_depend_only_on_relative_positions():
    """Shifting every position by a constant leaves the plain-MLA outputs unchanged."""
    p = make_params(seed=13, s=1)
    xs = inputs(14, 6)
    base = O.mla_forward(p, xs)
    orig = O.rope
    try:
        O.rope = lambda v, pos, theta: orig(v, pos + 17, theta)
        shifted = O.mla_forward(p, xs)
    finally:
        O.rope = orig
    np.testing.assert_allclose(base, shifted, atol=1e-10)


def test_sinusoid_values():
    pe = O.sinusoid_pe(3, 8)
    np.testing.assert_allclose(pe[:2], [math.sin(3), math.cos(3)], atol=1e-15)
    np.testing.assert_allclose(pe[6:], [math.sin(3 / 10000 ** 0.75), math.cos(3 / 10000 ** 0.75)],
                               atol=1e-15)


def test_state_from_cache_round_trip():
    p = make_params(seed=14, s=3)
    xs = inputs(15, 10)
    ys, st = O.decode_sequence(p, xs)
    st2 = O.state_from_cache(O.cache_array(st), st.tokens, p)
    x_new = inputs(16, 1)[0]
    np.testing.assert_array_equal(O.decode_step(p, st, x_new), O.decode_step(p, st2, x_new))


# ------------------------------------------------------------------ beam re-parenting

def test_reorder_equals_hypotheses_decoded_from_scratch():
    """Two rounds of forking: every hypothesis equals the same token history run alone, and a
    planted mistake (children sharing their parent's arrays) is caught by the same check."""
    p = make_params(seed=5, s=3)
    prompt = inputs(40, 7)

    def run(reorder):
        _, root = O.decode_sequence(p, prompt)
        states = reorder([root], [0, 0, 0])
        histories = [list(prompt) for _ in range(3)]
        outs = None
        for step in range(9):
            xs = inputs(50 + step, 3)
            outs = [O.decode_step(p, states[b], xs[b]) for b in range(3)]
            for b in range(3):
                histories[b].append(xs[b])
            if step in (2, 5):
                parents = [2, 0, 2] if step == 2 else [1, 1, 0]
                states = reorder(states, parents)
                histories = [list(histories[q]) for q in parents]
        worst = 0.0
        for b in range(3):
            alone, st = O.decode_sequence(p, np.stack(histories[b]))
            assert st.tokens == states[b].tokens and st.n_slots == states[b].n_slots
            worst = max(worst, np.abs(outs[b] - alone[-1]).max(),
                        np.abs(O.cache_array(states[b]) - O.cache_array(st)).max())
        return worst

    assert run(O.reorder_states) < 1e-12

    def aliasing(states, parents):          # the mistake: no copies, siblings write one list
        return [states[q] for q in parents]
    with pytest.raises((AssertionError, IndexError)):
        assert run(aliasing) < 1e-12


# ------------------------------------------------------------------ planted mistakes are caught

def _forms_disagree(p, xs):
    y_inc, _ = O.decode_sequence(p, xs)
    return np.abs(y_inc - O.forward_dense(p, xs)).max() > 1e-6


def test_mutation_zero_based_mask_is_caught(monkeypatch):
    def bad_mask(t_len, s):
        m = np.arange(t_len)[:, None]
        n = np.arange(t_len)[None, :]
        return (n == m) | ((n < m) & (n % s == 0))
    monkeypatch.setattr(O, "stride_aware_mask", bad_mask)
    assert _forms_disagree(make_params(seed=1, s=2), inputs(1, 9))


def test_slot_count_follows_ceiling_at_every_step():
    """The literal "remainder of i/s equals 1" rule would never open a slot at s = 1 and is
    read as (i - 1) mod s == 0; only that reading gives ceil(i/s) slots at every step."""
    p = make_params(seed=1, s=3)
    xs = inputs(2, 9)
    st = O.State()
    counts = []
    for x in xs:
        O.decode_step(p, st, x)
        counts.append(st.n_slots)
    assert counts == [math.ceil(i / 3) for i in range(1, 10)]
    st1 = O.State()
    p1 = make_params(seed=1, s=1)
    for i, x in enumerate(xs, start=1):
        O.decode_step(p1, st1, x)
        assert st1.n_slots == i


def test_mutation_dropped_rope_term_is_caught(monkeypatch):
    p = make_params(seed=15, s=1)
    xs = inputs(17, 7)
    good = O.mla_forward(p, xs)
    p2 = make_params(seed=15, s=1)
    p2.w_qr = np.zeros_like(p2.w_qr)
    assert np.abs(good - O.mla_forward(p2, xs)).max() > 1e-4
    y_inc, _ = O.decode_sequence(p, xs)
    np.testing.assert_allclose(y_inc, good, atol=1e-10)


def test_mutation_key_from_first_token_is_caught(monkeypatch):
    """Keeping the chunk's first RoPE key instead of its latest one must break Form I = Form II."""
    p = make_params(seed=16, s=2)
    xs = inputs(18, 8)
    orig = O.decode_step

    def bad_step(p_, st, x, want_output=True):
        keep = list(st.kr_hat)
        opened = (st.tokens % p_.stride) == 0
        y = orig(p_, st, x, want_output=False)
        if not opened:
            st.kr_hat[-1] = keep[-1]
        q = x @ p_.w_q
        q_rope = O.rope((x @ p_.w_qr).reshape(p_.n_heads, p_.rope_dim), st.tokens - 1,
                        p_.rope_theta).reshape(-1)
        return O.attend(p_, q, q_rope, np.stack(st.c_hat), np.stack(st.kr_hat))

    st = O.State()
    y_bad = np.stack([bad_step(p, st, x) for x in xs])
    assert np.abs(y_bad - O.forward_dense(p, xs)).max() > 1e-6
