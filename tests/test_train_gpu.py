"""The training path on the GPU: mtla_prefill as the forward pass of Section 4.2's parallel
form and mtla_train_backward as its reverse, against the training oracle (dense T x T form in
fp64, itself pinned by finite differences).

Tolerances.  y: the specification's fp32 bound (max-abs 1e-4).  Gradients are sums of products
over the B * T rows, so their size varies by orders of magnitude between tensors; each tensor is
held to 1e-4 of its own largest entry (at least 1e-4 absolute), i.e. the same four digits."""
import numpy as np
import pytest
import torch

from oracle import train_oracle as TR
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def assert_grad_close(got, want, name):
    g = got.detach().double().cpu().numpy()
    assert g.shape == want.shape, (name, g.shape, want.shape)
    bound = 1e-4 * max(1.0, float(np.abs(want).max()))
    err = float(np.abs(g - want).max())
    assert err <= bound, f"{name}: max abs err {err:.3e} > {bound:.3e}"


def layer(d, nh, dh, r, dr, dw, stride, batch, t_len, seed=81):
    return synth.Workload(name="train", dtype="fp32", batch=batch, d_model=d, n_heads=nh, head_dim=dh,
                          latent_rank=r, rope_dim=dr, hyper_dim=dw, stride=stride, prefill_tokens=t_len,
                          context_tokens=0, decode_steps=2, seed=seed)


@pytest.mark.parametrize("d,nh,dh,r,dr,dw,stride,batch,t_len", [
    (128, 4, 64, 64, 32, 16, 2, 2, 37),      # odd length: the last chunk stays open
    (96, 2, 64, 128, 32, 24, 3, 3, 70),      # several 64-wide tiles of every product, ragged
    (128, 2, 128, 64, 64, 8, 4, 1, 130),     # d_h 128, d_R 64
    (64, 4, 64, 64, 32, 16, 1, 2, 33),       # s = 1: no gate, zero hyper-network gradients
    (128, 8, 64, 128, 32, 16, 2, 10, 250),   # enough tiles for the 128 x 128 and 128 x 64 kernels, ragged
                                             # edges in both; weight gradients summed in 4 pieces
    (64, 2, 64, 64, 32, 16, 2, 2, 256),      # 512 rows: weight gradients in 8 pieces of 64 rows
])
def test_forward_and_backward_match_the_training_oracle(d, nh, dh, r, dr, dw, stride, batch, t_len):
    w = layer(d, nh, dh, r, dr, dw, stride, batch, t_len)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    x = synth.prompt(w)
    dy = torch.stack([synth.stored(synth.normal(w.seed, f"dy/{b}", (t_len, d)), "fp32")
                      for b in range(batch)])
    h = H.gpu_handle(w, weights)
    try:
        y = M.mtla_prefill(h, x.cuda())
        dx, grads = M.mtla_train_backward(h, x.cuda(), dy.cuda())
        M.mtla_check(h)
        want_y, want_dx, want_g = TR.forward_backward_batch(p, x.double().numpy(), dy.double().numpy())
        H.assert_close(y, want_y, "fp32", "forward")
        assert_grad_close(dx, want_dx, "dx")
        for name in TR.PARAM_NAMES:
            assert_grad_close(grads[name], want_g[name], name)
        if stride == 1:
            for name in ("hyp_c_w", "hyp_c_b", "hyp_pe_w", "hyp_pe_b"):
                assert not grads[name].any()
        # Deterministic: the same call again gives the same bits.
        M.mtla_reset(h)
        M.mtla_prefill(h, x.cuda())
        dx2, grads2 = M.mtla_train_backward(h, x.cuda(), dy.cuda())
        assert torch.equal(dx, dx2) and all(torch.equal(grads[n], grads2[n]) for n in grads)
    finally:
        M.mtla_destroy(h)


def test_backward_needs_the_matching_forward_pass():
    w = layer(64, 4, 64, 64, 32, 16, 2, 2, 20)
    weights = synth.make_weights(w)
    x = synth.prompt(w).cuda()
    h = H.gpu_handle(w, weights)
    try:
        with pytest.raises(M.MTLAError) as e:
            M.mtla_train_backward(h, x, x)                      # no forward pass yet
        assert e.value.status == -7
        M.mtla_prefill(h, x)
        M.mtla_decode_step(h, synth.decode_input(w, 0).cuda())  # the step reuses the scratch
        with pytest.raises(M.MTLAError) as e:
            M.mtla_train_backward(h, x, x)
        assert e.value.status == -7
        M.mtla_reset(h)
        M.mtla_prefill(h, x)
        with pytest.raises(M.MTLAError) as e:
            M.mtla_train_backward(h, x[:1].contiguous(), x[:1].contiguous())   # another batch
        assert e.value.status == -7
        dx, _ = M.mtla_train_backward(h, x, x)
        assert torch.isfinite(dx).all()
    finally:
        M.mtla_destroy(h)
    wb = w.scaled(dtype="bf16", latent_rank=128)
    hb = H.gpu_handle(wb, synth.make_weights(wb))
    try:
        xb = synth.prompt(wb).cuda()
        M.mtla_prefill(hb, xb)
        with pytest.raises(M.MTLAError) as e:
            M.mtla_train_backward(hb, xb, xb)                   # bf16 layers have no backward pass
        assert e.value.status == -2
    finally:
        M.mtla_destroy(hb)
