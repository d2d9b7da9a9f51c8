"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element.

Sizes here are ones the oracle finishes in seconds but that still span several attention
tiles, several splits and ragged tails.  Full-size configurations are in test_configs_gpu.py.
"""
import math

import numpy as np
import pytest
import torch

from oracle import mtla_oracle as O
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

SMALL_BF16 = synth.Workload(name="small_bf16", dtype="bf16", batch=3, d_model=128, n_heads=8,
                            head_dim=64, latent_rank=128, rope_dim=32, hyper_dim=32, stride=2,
                            prefill_tokens=0, context_tokens=0, decode_steps=0, seed=11)
SMALL_FP32 = SMALL_BF16.scaled(name="small_fp32", dtype="fp32", n_heads=4, latent_rank=64,
                               hyper_dim=16, seed=12)


def run_oracle_decode(w, weights, xs):
    """xs [steps][B][d] torch -> (ys [steps][B][d], per-sequence final states)."""
    p = H.oracle_params(w, weights)
    ys, states = [], []
    for b in range(xs.shape[1]):
        y, st = O.decode_sequence(p, xs[:, b].double().numpy())
        ys.append(y)
        states.append(st)
    return np.stack(ys, axis=1), states


def decode_inputs(w, steps, batch):
    return torch.stack([synth.decode_input(w.scaled(batch=batch), i) for i in range(steps)])


@pytest.mark.parametrize("base", [SMALL_FP32, SMALL_BF16], ids=["fp32", "bf16"])
@pytest.mark.parametrize("stride", [1, 2, 3, 4])
def test_decode_from_empty_cache_matches_oracle(base, stride):
    steps = 150 if stride <= 2 else 70      # > 64 slots so that the attention splits
    w = base.scaled(stride=stride, decode_steps=steps)
    weights = synth.make_weights(w)
    xs = decode_inputs(w, steps, w.batch)
    want, states = run_oracle_decode(w, weights, xs)
    h = H.gpu_handle(w, weights, max_tokens=steps, max_prefill_tokens=0)
    try:
        for i in range(steps):
            y = M.mtla_decode_step(h, xs[i].cuda())
            H.assert_close(y, want[i], w.dtype, f"step {i}")
            tokens, slots, batch = M.mtla_position(h)
            assert (tokens, slots, batch) == (i + 1, math.ceil((i + 1) / stride), w.batch)
            assert M.mtla_cache_bytes(h) == (w.batch * slots * w.slot_width
                                             * (4 if w.dtype == "fp32" else 2))
        cache = M.mtla_cache_export(h)
        want_cache = np.stack([O.cache_array(st) for st in states])
        H.assert_cache_close(cache, want_cache, w.dtype)
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("base", [SMALL_FP32, SMALL_BF16], ids=["fp32", "bf16"])
@pytest.mark.parametrize("stride,t_len", [(1, 70), (2, 129), (3, 100), (4, 66), (5, 7), (2, 1)])
def test_prefill_matches_oracle_and_hands_over_to_decode(base, stride, t_len):
    steps = 6
    w = base.scaled(stride=stride, prefill_tokens=t_len, decode_steps=steps, batch=2)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    prompt = synth.prompt(w)
    xs = decode_inputs(w, steps, w.batch)
    h = H.gpu_handle(w, weights)
    try:
        y = M.mtla_prefill(h, prompt.cuda())
        states = []
        for b in range(w.batch):
            want, st = O.decode_sequence(p, prompt[b].double().numpy())
            H.assert_close(y[b], want, w.dtype, f"prefill seq {b}")
            states.append(st)
        tokens, slots, batch = M.mtla_position(h)
        assert (tokens, slots, batch) == (t_len, math.ceil(t_len / stride), w.batch)
        H.assert_cache_close(M.mtla_cache_export(h),
                             np.stack([O.cache_array(st) for st in states]), w.dtype)
        for i in range(steps):
            yd = M.mtla_decode_step(h, xs[i].cuda())
            want = np.stack([O.decode_step(p, states[b], xs[i, b].double().numpy())
                             for b in range(w.batch)])
            H.assert_close(yd, want, w.dtype, f"decode step {i} after prefill")
        assert M.mtla_position(h)[1] == math.ceil((t_len + steps) / stride)
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


def test_prefill_equals_token_by_token_decode_on_the_gpu():
    """The GPU's own two paths agree (Section 4.2), independently of the oracle."""
    w = SMALL_FP32.scaled(stride=3, prefill_tokens=50, batch=2)
    weights = synth.make_weights(w)
    prompt = synth.prompt(w).cuda()
    h1 = H.gpu_handle(w, weights)
    h2 = H.gpu_handle(w, weights)
    try:
        y_par = M.mtla_prefill(h1, prompt)
        y_inc = torch.stack([M.mtla_decode_step(h2, prompt[:, i].contiguous())
                             for i in range(50)], dim=1)
        assert (y_par - y_inc).abs().max().item() <= 1e-4
        c1, c2 = M.mtla_cache_export(h1), M.mtla_cache_export(h2)
        assert c1.shape == c2.shape == (2, 17, w.slot_width)
        assert (c1 - c2).abs().max().item() <= 1e-5
    finally:
        M.mtla_destroy(h1)
        M.mtla_destroy(h2)


def test_stride_one_is_plain_mla_on_the_gpu():
    w = SMALL_FP32.scaled(stride=1, prefill_tokens=40, batch=1)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    prompt = synth.prompt(w)
    h = H.gpu_handle(w, weights)
    try:
        y = M.mtla_prefill(h, prompt.cuda())
        H.assert_close(y[0], O.mla_forward(p, prompt[0].double().numpy()), "fp32")
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_cache_import_export_and_open_slot(dtype):
    """An imported cache with an open last slot continues exactly like the oracle's state."""
    w = SMALL_BF16.scaled(dtype=dtype, stride=3, context_tokens=200, decode_steps=4, batch=2,
                          n_heads=4)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    n_slots = math.ceil(200 / 3)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(2)])
    xs = decode_inputs(w, 4, 2)
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        M.mtla_cache_import(h, cache.cuda(), 200)
        assert M.mtla_position(h) == (200, n_slots, 2)
        assert torch.equal(M.mtla_cache_export(h).cpu(), cache)
        states = [O.state_from_cache(cache[b].double().numpy(), 200, p) for b in range(2)]
        for i in range(4):
            y = M.mtla_decode_step(h, xs[i].cuda())
            want = np.stack([O.decode_step(p, states[b], xs[i, b].double().numpy())
                             for b in range(2)])
            H.assert_close(y, want, dtype, f"step {i}")
        assert M.mtla_position(h)[1] == math.ceil(204 / 3) == states[0].n_slots
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("r,stride", [(64, 2), (192, 3), (320, 1)])
def test_bf16_layers_off_the_tensor_core_shapes(r, stride):
    """bf16 layers whose latent rank is not a multiple of 128 run on the CUDA-core kernels
    (with the folded gate); prefill, hand-over and decode must still match the oracle."""
    w = SMALL_BF16.scaled(latent_rank=r, hyper_dim=r // 4, stride=stride, prefill_tokens=75,
                          decode_steps=5, batch=2)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    prompt = synth.prompt(w)
    xs = decode_inputs(w, w.decode_steps, w.batch)
    h = H.gpu_handle(w, weights)
    try:
        assert M.mtla_attention_variant(h) == "fma"
        y = M.mtla_prefill(h, prompt.cuda())
        states = []
        for b in range(w.batch):
            want, st = O.decode_sequence(p, prompt[b].double().numpy())
            H.assert_close(y[b], want, "bf16", f"prefill seq {b}")
            states.append(st)
        for i in range(w.decode_steps):
            yd = M.mtla_decode_step(h, xs[i].cuda())
            want = np.stack([O.decode_step(p, states[b], xs[i, b].double().numpy())
                             for b in range(w.batch)])
            H.assert_close(yd, want, "bf16", f"decode step {i}")
        H.assert_cache_close(M.mtla_cache_export(h),
                             np.stack([O.cache_array(st) for st in states]), "bf16")
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


def test_peaked_softmax_variant():
    """Queries scaled up 4x give a near one-hot softmax; parity must survive it."""
    w = SMALL_FP32.scaled(stride=2, decode_steps=90, batch=1)
    weights = synth.make_weights(w)
    weights["w_q"] = weights["w_q"] * 4
    weights["w_qr"] = weights["w_qr"] * 4
    xs = decode_inputs(w, 90, 1)
    want, _ = run_oracle_decode(w, weights, xs)
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        for i in range(90):
            H.assert_close(M.mtla_decode_step(h, xs[i].cuda()), want[i], "fp32", f"step {i}")
    finally:
        M.mtla_destroy(h)


def test_batch_rows_are_independent():
    w = SMALL_BF16.scaled(stride=2, decode_steps=20, batch=4)
    weights = synth.make_weights(w)
    xs = decode_inputs(w, 20, 4)
    perm = torch.tensor([2, 0, 3, 1])
    h1 = H.gpu_handle(w, weights, max_prefill_tokens=0)
    h2 = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        for i in range(20):
            y1 = M.mtla_decode_step(h1, xs[i].cuda())
            y2 = M.mtla_decode_step(h2, xs[i][perm].contiguous().cuda())
            assert torch.equal(y1[perm], y2)
    finally:
        M.mtla_destroy(h1)
        M.mtla_destroy(h2)


def test_host_buffer_entry_point_matches_device_entry_point():
    w = SMALL_BF16.scaled(stride=2, decode_steps=5, batch=3)
    weights = synth.make_weights(w)
    xs = decode_inputs(w, 5, 3)
    h1 = H.gpu_handle(w, weights, max_prefill_tokens=0)
    h2 = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        for i in range(5):
            y1 = M.mtla_decode_step(h1, xs[i].cuda())
            xh = xs[i].pin_memory()
            yh = torch.empty_like(xh).pin_memory()
            M.mtla_decode_step_host(h2, xh, yh)
            torch.cuda.synchronize()
            assert torch.equal(y1.cpu(), yh)
    finally:
        M.mtla_destroy(h1)
        M.mtla_destroy(h2)


def test_error_paths_leave_state_untouched():
    w = SMALL_FP32.scaled(stride=2, prefill_tokens=8, decode_steps=2, batch=2)
    weights = synth.make_weights(w)
    h = H.gpu_handle(w, weights, max_tokens=10, max_prefill_tokens=8)
    try:
        x = synth.decode_input(w, 0).cuda()
        with pytest.raises(M.MTLAError) as e:                     # prompt longer than workspace
            M.mtla_prefill(h, torch.zeros(2, 9, w.d_model, device="cuda"))
        assert e.value.status == -4
        with pytest.raises(M.MTLAError) as e:                     # batch beyond capacity
            M.mtla_decode_step(h, torch.zeros(3, w.d_model, device="cuda"))
        assert e.value.status == -4
        assert M.mtla_position(h) == (0, 0, 0)
        M.mtla_prefill(h, synth.prompt(w).cuda())
        with pytest.raises(M.MTLAError) as e:                     # prefill needs an empty cache
            M.mtla_prefill(h, synth.prompt(w).cuda())
        assert e.value.status == -7
        with pytest.raises(M.MTLAError) as e:                     # batch differs from the cache's
            M.mtla_decode_step(h, x[:1].contiguous())
        assert e.value.status == -5
        M.mtla_decode_step(h, x)
        M.mtla_decode_step(h, x)
        with pytest.raises(M.MTLAError) as e:                     # token 11 of 10
            M.mtla_decode_step(h, x)
        assert e.value.status == -4
        assert M.mtla_position(h) == (10, 5, 2)
        M.mtla_reset(h)
        assert M.mtla_position(h) == (0, 0, 0) and M.mtla_cache_bytes(h) == 0
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)
