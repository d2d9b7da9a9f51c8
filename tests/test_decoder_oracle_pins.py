"""Pins of the decoder oracle (oracle/decoder_oracle.py) to things other than itself: torch's own
LayerNorm / Linear / ReLU modules, the MTLA oracle called directly, closed forms, the agreement of
its two evaluation orders, and planted mistakes that a pin must catch."""
import numpy as np
import pytest
import torch

from oracle import decoder_oracle as D
from oracle import mtla_oracle as O
from paper_2505_13544_b200 import synth
from tests import helpers as H


def small_stack(n_layers=3, stride=2, d_ff=96, seed=7):
    w = synth.Workload(name="dec_pin", dtype="fp32", batch=1, d_model=48, n_heads=2, head_dim=16,
                       latent_rank=24, rope_dim=8, hyper_dim=6, stride=stride, prefill_tokens=0,
                       context_tokens=0, decode_steps=0, seed=seed)
    sw = synth.StackWorkload("pin", w, n_layers, d_ff)
    return w, sw, synth.make_stack_weights(sw)


def to_params(w, weights):
    return H.oracle_stack_params(synth.StackWorkload("pin", w, len(weights["layers"]), 0), weights)


def torch_ln(x, gamma, beta):
    m = torch.nn.LayerNorm(len(gamma), eps=1e-5, dtype=torch.float64)
    with torch.no_grad():
        m.weight.copy_(torch.from_numpy(gamma))
        m.bias.copy_(torch.from_numpy(beta))
        return m(torch.from_numpy(np.asarray(x, dtype=np.float64))).numpy()


def torch_ffn(lp, v):
    l1 = torch.nn.Linear(lp.w1.shape[0], lp.w1.shape[1], dtype=torch.float64)
    l2 = torch.nn.Linear(lp.w2.shape[0], lp.w2.shape[1], dtype=torch.float64)
    with torch.no_grad():
        l1.weight.copy_(torch.from_numpy(lp.w1.T)); l1.bias.copy_(torch.from_numpy(lp.b1))
        l2.weight.copy_(torch.from_numpy(lp.w2.T)); l2.bias.copy_(torch.from_numpy(lp.b2))
        return l2(torch.relu(l1(torch.from_numpy(np.asarray(v, dtype=np.float64))))).numpy()


def inputs(w, t, seed=3):
    return synth.normal(seed, "dec_x", (t, w.d_model)).astype(np.float64)


def test_layer_norm_and_feed_forward_match_torch_modules():
    w, _, weights = small_stack()
    sp = to_params(w, weights)
    lp = sp.layers[0]
    x = inputs(w, 9)
    np.testing.assert_allclose(D.layer_norm(x, lp.ln2_gamma, lp.ln2_beta, lp.ln_eps),
                               torch_ln(x, lp.ln2_gamma, lp.ln2_beta), atol=1e-12)
    np.testing.assert_allclose(D.feed_forward(lp, x), torch_ffn(lp, x), atol=1e-12)
    # ReLU really clips: some hidden units are negative before it.
    assert ((x @ lp.w1 + lp.b1) < 0).any()


def test_attention_sublayer_is_the_mtla_oracle_on_the_normalised_input():
    """Feed-forward output matrix and bias zero: y = x + MTLA(LayerNorm_1(x)), with the
    LayerNorm from torch and the attention from the MTLA oracle called directly."""
    w, _, weights = small_stack(n_layers=1)
    sp = to_params(w, weights)
    lp = sp.layers[0]
    lp.w2 = np.zeros_like(lp.w2)
    lp.b2 = np.zeros_like(lp.b2)
    xs = inputs(w, 11)
    st, st_ref = O.State(), O.State()
    for x in xs:
        got = D.layer_decode_step(lp, st, x)
        want = x + O.decode_step(lp.attn, st_ref, torch_ln(x, lp.ln1_gamma, lp.ln1_beta))
        np.testing.assert_allclose(got, want, atol=1e-11)
    assert st.n_slots == -(-11 // w.stride)


def test_feed_forward_sublayer_alone_when_the_attention_output_is_zero():
    """W_O = 0: y = x + FFN(LayerNorm_2(x)) exactly, every piece from torch."""
    w, _, weights = small_stack(n_layers=1)
    sp = to_params(w, weights)
    lp = sp.layers[0]
    lp.attn.w_o = np.zeros_like(lp.attn.w_o)
    st = O.State()
    for x in inputs(w, 5):
        want = x + torch_ffn(lp, torch_ln(x, lp.ln2_gamma, lp.ln2_beta))
        np.testing.assert_allclose(D.layer_decode_step(lp, st, x), want, atol=1e-11)


@pytest.mark.parametrize("stride,t_len", [(1, 9), (2, 23), (3, 20)])
def test_token_by_token_equals_layer_by_layer(stride, t_len):
    w, _, weights = small_stack(n_layers=3, stride=stride)
    sp = to_params(w, weights)
    xs = inputs(w, t_len)
    y_tok, st_tok = D.stack_decode_sequence(sp, xs)
    y_lay, st_lay = D.stack_forward_by_layers(sp, xs)
    np.testing.assert_allclose(y_tok, y_lay, atol=1e-10)
    for a, b in zip(st_tok.layers, st_lay.layers):
        np.testing.assert_allclose(O.cache_array(a), O.cache_array(b), atol=1e-10)
        assert a.tokens == b.tokens == t_len
    rows = [0, 3, t_len - 1]
    y_rows, _ = D.stack_forward_by_layers(sp, xs, rows=rows)
    np.testing.assert_allclose(y_rows, y_tok[rows], atol=1e-10)
    # A prompt consumed layer by layer, then decoding token by token, continues the same sequence.
    cut = t_len // 2
    _, st = D.stack_forward_by_layers(sp, xs[:cut])
    y_tail, _ = D.stack_decode_sequence(sp, xs[cut:], st)
    np.testing.assert_allclose(y_tail, y_tok[cut:], atol=1e-10)


def test_two_layer_stack_is_the_composition_and_the_final_norm():
    w, _, weights = small_stack(n_layers=2)
    sp = to_params(w, weights)
    xs = inputs(w, 7)
    st = D.StackState.empty(2)
    s0, s1 = O.State(), O.State()
    for x in xs:
        got = D.stack_decode_step(sp, st, x)
        h1 = D.layer_decode_step(sp.layers[1], s1, D.layer_decode_step(sp.layers[0], s0, x))
        np.testing.assert_allclose(got, torch_ln(h1, sp.lnf_gamma, sp.lnf_beta), atol=1e-11)
    assert st.tokens == 7
    assert D.stack_cache_elements(sp, 7) == 2 * O.cache_elements(7, sp.layers[0].attn)


def test_planted_mistakes_are_caught(monkeypatch):
    w, _, weights = small_stack(n_layers=1)
    sp = to_params(w, weights)
    lp = sp.layers[0]
    x = inputs(w, 1)[0]

    def reference(x):
        st = O.State()
        h = x + O.decode_step(lp.attn, st, torch_ln(x, lp.ln1_gamma, lp.ln1_beta))
        return h + torch_ffn(lp, torch_ln(h, lp.ln2_gamma, lp.ln2_beta))

    np.testing.assert_allclose(D.layer_decode_step(lp, O.State(), x), reference(x), atol=1e-11)
    # (a) feed-forward without its output bias
    monkeypatch.setattr(D, "feed_forward", lambda lp_, v: np.maximum(v @ lp_.w1 + lp_.b1, 0.0) @ lp_.w2)
    assert np.abs(D.layer_decode_step(lp, O.State(), x) - reference(x)).max() > 1e-3
    monkeypatch.undo()
    # (b) LayerNorm with the unbiased variance
    def ln_unbiased(v, gamma, beta, eps):
        mu = v.mean(axis=-1, keepdims=True)
        return (v - mu) / np.sqrt(v.var(axis=-1, ddof=1, keepdims=True) + eps) * gamma + beta
    monkeypatch.setattr(D, "layer_norm", ln_unbiased)
    assert np.abs(D.layer_decode_step(lp, O.State(), x) - reference(x)).max() > 1e-3
    monkeypatch.undo()
    # (c) the second LayerNorm fed with x instead of h (a dropped residual inside the block)
    swapped = D.LayerParams(**{**lp.__dict__, "ln2_gamma": lp.ln1_gamma, "ln2_beta": lp.ln1_beta})
    assert np.abs(D.layer_decode_step(swapped, O.State(), x) - reference(x)).max() > 1e-3
