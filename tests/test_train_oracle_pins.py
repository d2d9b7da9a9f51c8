"""Pins of the training-path oracle (oracle/train_oracle.py).  Its forward must be the dense
parallel form the MTLA oracle already pins to incremental decoding; every gradient is checked
against central finite differences of THAT function (mtla_oracle.forward_dense, which
train_oracle does not define), along random directions; plus structural facts (no gradient
reaches the hyper-network at s = 1, sequences of a batch do not mix) and planted mistakes."""
import copy

import numpy as np
import pytest

from oracle import mtla_oracle as O
from oracle import train_oracle as TR
from paper_2505_13544_b200 import synth
from tests import helpers as H


def small(stride, seed=11, t_len=13):
    w = synth.Workload(name="train_pin", dtype="fp32", batch=1, d_model=24, n_heads=2, head_dim=8,
                       latent_rank=12, rope_dim=4, hyper_dim=5, stride=stride, prefill_tokens=t_len,
                       context_tokens=0, decode_steps=0, seed=seed)
    weights = {k: v.double() for k, v in synth.make_weights(w).items()}
    p = H.oracle_params(w, weights)
    xs = synth.normal(seed, "train_x", (t_len, w.d_model)).astype(np.float64)
    dy = synth.normal(seed, "train_dy", (t_len, w.d_model)).astype(np.float64)
    return w, p, xs, dy


def loss(p, xs, dy):
    return float((O.forward_dense(p, xs) * dy).sum())


def directional_fd(p, xs, dy, name, direction, eps=1e-6):
    def at(t):
        q = copy.deepcopy(p)
        x = xs
        if name == "x":
            x = xs + t * direction
        else:
            setattr(q, name, getattr(p, name) + t * direction)
        return loss(q, x, dy)
    return (at(eps) - at(-eps)) / (2 * eps)


@pytest.mark.parametrize("stride,t_len", [(1, 9), (2, 13), (3, 11), (4, 10)])
def test_forward_is_the_dense_form_and_every_gradient_matches_finite_differences(stride, t_len):
    w, p, xs, dy = small(stride, t_len=t_len)
    y, sv = TR.forward(p, xs)
    np.testing.assert_allclose(y, O.forward_dense(p, xs), atol=1e-12)
    dx, grads = TR.backward(p, sv, dy)
    rng = np.random.default_rng(5)
    checks = [("x", dx)] + [(n, grads[n]) for n in TR.PARAM_NAMES]
    for name, grad in checks:
        if stride == 1 and name.startswith("hyp_"):
            assert not grad.any()                      # w = 1: the hyper-network is not on the path
            continue
        for _ in range(2):
            v = rng.standard_normal(grad.shape)
            want = directional_fd(p, xs, dy, name, v)
            got = float((grad * v).sum())
            assert abs(got - want) <= 1e-6 * max(1.0, abs(want)), (name, got, want)


def test_batch_gradients_are_sums_and_sequences_do_not_mix():
    w, p, xs, dy = small(2)
    xs2 = np.stack([xs, synth.normal(3, "other_x", xs.shape).astype(np.float64)])
    dy2 = np.stack([dy, synth.normal(3, "other_dy", dy.shape).astype(np.float64)])
    y, dx, grads = TR.forward_backward_batch(p, xs2, dy2)
    for b in range(2):
        yb, sv = TR.forward(p, xs2[b])
        dxb, _ = TR.backward(p, sv, dy2[b])
        np.testing.assert_allclose(y[b], yb, atol=1e-12)
        np.testing.assert_allclose(dx[b], dxb, atol=1e-12)
    g0 = TR.backward(p, TR.forward(p, xs2[0])[1], dy2[0])[1]
    g1 = TR.backward(p, TR.forward(p, xs2[1])[1], dy2[1])[1]
    for name in TR.PARAM_NAMES:
        np.testing.assert_allclose(grads[name], g0[name] + g1[name], atol=1e-11)
    # Causality: the loss on rows < m does not depend on tokens >= m.
    dy_head = dy.copy()
    dy_head[5:] = 0.0
    dxh, _ = TR.backward(p, TR.forward(p, xs)[1], dy_head)
    assert not dxh[5:].any() and dxh[:5].any()


def test_planted_mistakes_fail_the_finite_difference_pin(monkeypatch):
    w, p, xs, dy = small(2)
    rng = np.random.default_rng(9)

    def worst_gap():
        _, sv = TR.forward(p, xs)
        dx, grads = TR.backward(p, sv, dy)
        gap = 0.0
        for name, grad in [("x", dx), ("w_r", grads["w_r"]), ("w_kr", grads["w_kr"]),
                           ("hyp_c_w", grads["hyp_c_w"])]:
            v = rng.standard_normal(grad.shape)
            want = directional_fd(p, xs, dy, name, v)
            gap = max(gap, abs(float((grad * v).sum()) - want) / max(1.0, abs(want)))
        return gap

    assert worst_gap() <= 1e-6
    # (a) the chunk mask forgotten when the gate's gradient is formed
    monkeypatch.setattr(TR, "chunk_mask", lambda t, s: np.tril(np.ones((t, t))))
    assert worst_gap() > 1e-3
    monkeypatch.undo()
    # (b) the rotation not inverted on the way back
    real = TR.rotate_rows
    monkeypatch.setattr(TR, "rotate_rows", lambda v, theta, sign=1.0: real(v, theta, 1.0))
    assert worst_gap() > 1e-3
    monkeypatch.undo()
    # (c) LayerNorm backward without the projection onto the normalised vector
    src = TR.backward

    def bad_backward(p_, sv, dy_):
        sv2 = copy.copy(sv)
        sv2.xhat = np.zeros_like(sv.xhat)
        dx, grads = src(p_, sv2, dy_)
        return dx, grads
    monkeypatch.setattr(TR, "backward", bad_backward)
    assert worst_gap() > 1e-3
