"""The comparison layers (MHA / GQA / MQA over a key-value cache) on the GPU, through the C ABI,
against their CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import gqa_oracle as G
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def layer(w, n_kv, max_batch, max_tokens):
    weights = synth.make_baseline_weights(w, n_kv)
    p = G.params_from_tensors(
        dict(d_model=w.d_model, n_heads=w.n_heads, n_groups=n_kv, head_dim=w.head_dim),
        {k: v.double().numpy() for k, v in weights.items()}, rope_theta=w.rope_theta)
    h = M.mtla_baseline_create(d_model=w.d_model, n_heads=w.n_heads, n_kv_heads=n_kv,
                               head_dim=w.head_dim, max_batch=max_batch, max_tokens=max_tokens,
                               weights={k: v.cuda() for k, v in weights.items()},
                               rope_theta=w.rope_theta)
    return p, h


@pytest.mark.parametrize("heads,n_kv,dh", [(8, 8, 64), (8, 2, 64), (8, 1, 64), (32, 8, 128), (32, 1, 128),
                                           (4, 4, 128)])
def test_decode_from_empty_matches_the_oracle(heads, n_kv, dh):
    """Every step of 150 (three 64-token tiles with a ragged tail), three sequences."""
    w = synth.WORKLOADS["paper"].scaled(n_heads=heads, head_dim=dh, d_model=512, batch=3, seed=40 + n_kv)
    steps = 150
    p, h = layer(w, n_kv, w.batch, steps + 1)
    try:
        states = [G.GQAState() for _ in range(w.batch)]
        for i in range(steps):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (w.batch, w.d_model)), "bf16")
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([G.decode_step(p, states[b], x[b].double().numpy()) for b in range(w.batch)])
            H.assert_close(y, want, "bf16", f"step {i}")
        M.mtla_check(h)
        assert M.mtla_position(h) == (steps, steps, w.batch)
        assert M.mtla_cache_bytes(h) == w.batch * steps * G.cache_elements_per_token(n_kv, dh) * 2
        cache = M.mtla_cache_export(h)
        assert tuple(cache.shape) == (w.batch, n_kv, steps, 2 * dh)
        H.assert_cache_close(cache, np.stack([G.cache_array(st) for st in states]), "bf16")
    finally:
        M.mtla_destroy(h)


def test_import_continues_bit_identically():
    w = synth.WORKLOADS["paper"].scaled(batch=2, seed=50)
    p, h = layer(w, 2, w.batch, 300)
    _, h2 = layer(w, 2, w.batch, 400)
    try:
        for i in range(70):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (w.batch, w.d_model)), "bf16").cuda()
            M.mtla_decode_step(h, x)
        M.mtla_cache_import(h2, M.mtla_cache_export(h), 70)
        for i in range(70, 140):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (w.batch, w.d_model)), "bf16").cuda()
            assert torch.equal(M.mtla_decode_step(h, x), M.mtla_decode_step(h2, x))
        M.mtla_check(h)
        M.mtla_check(h2)
    finally:
        M.mtla_destroy(h)
        M.mtla_destroy(h2)


def test_long_imported_context_sampled():
    """4096-token stand-in caches (64 tiles per plane), outputs of all sequences at three steps."""
    w = synth.WORKLOADS["paper"].scaled(batch=4, seed=51)
    n_kv, ctx = 2, 4096
    p, h = layer(w, n_kv, w.batch, ctx + 8)
    try:
        cache = torch.stack([torch.stack([synth.kv_cache_plane(w, b, g, ctx) for g in range(n_kv)])
                             for b in range(w.batch)])
        M.mtla_cache_import(h, cache.cuda(), ctx)
        states = [G.state_from_cache(cache[b].double().numpy()) for b in range(w.batch)]
        for i in range(3):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (w.batch, w.d_model)), "bf16")
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([G.decode_step(p, states[b], x[b].double().numpy()) for b in range(w.batch)])
            H.assert_close(y, want, "bf16", f"step {i}")
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


def test_calls_that_do_not_apply_are_refused():
    w = synth.WORKLOADS["paper"].scaled(batch=1)
    _, h = layer(w, 1, 1, 8)
    try:
        x = synth.stored(synth.normal(0, "x", (1, 4, w.d_model)), "bf16").cuda()
        for call in (lambda: M.mtla_prefill(h, x), lambda: M.mtla_beam_reorder(h, [0]),
                     lambda: M.mtla_decode_step_static(h, x[0, :1].contiguous())):
            with pytest.raises(M.MTLAError) as err:
                call()
            assert err.value.status == -7
        with pytest.raises(M.MTLAError):
            M.mtla_baseline_create(d_model=512, n_heads=8, n_kv_heads=3, head_dim=64, max_batch=1,
                                   max_tokens=8, weights={k: v.cuda() for k, v in
                                                          synth.make_baseline_weights(w, 1).items()})
    finally:
        M.mtla_destroy(h)
