"""mtla_decode_step_static: the decode step whose attention split workspace sits in the
library's built-in static device array, for callers that may not rely on allocated scratch
(a host that has given all device memory to its own pool, or runs under a no-allocation rule
once serving has started).

Collected last on purpose (file name): a run that stops at the first failure has then already
been through every other test.  The checks go through the C ABI and compare against the
ordinary entry point on two consecutive calls, which also shows that the shared array's
left-over contents (tickets, partials of the previous call) do no harm.
"""
import math

import pytest
import torch

from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def layer(dtype, n_heads, r, batch, context):
    return synth.Workload(name="static", dtype=dtype, batch=batch, d_model=256, n_heads=n_heads,
                          head_dim=64, latent_rank=r, rope_dim=32, hyper_dim=r // 4, stride=2,
                          prefill_tokens=0, context_tokens=context, decode_steps=2, seed=41)


@pytest.mark.parametrize("dtype,n_heads,r", [("bf16", 8, 256), ("fp32", 4, 64)],
                         ids=["tensor-core-path", "cuda-core-path"])
def test_static_scratch_step_matches_the_ordinary_step_twice_in_a_row(dtype, n_heads, r):
    w = layer(dtype, n_heads, r, batch=5, context=900)      # 450 slots: several splits / tiles
    weights = synth.make_weights(w)
    n_slots = math.ceil(w.context_tokens / w.stride)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(w.batch)]).cuda()
    ref = H.gpu_handle(w, weights, max_prefill_tokens=0)
    sta = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        M.mtla_cache_import(ref, cache, w.context_tokens)
        M.mtla_cache_import(sta, cache, w.context_tokens)
        for i in range(2):                                   # two calls in a row share the array
            x = synth.decode_input(w, i).cuda()
            want = M.mtla_decode_step(ref, x)
            got = M.mtla_decode_step_static(sta, x)
            M.mtla_check(sta)
            H.assert_close(got, want.double().cpu().numpy(), dtype, f"static step {i}")
        assert M.mtla_position(sta) == M.mtla_position(ref)
        assert torch.equal(M.mtla_cache_export(sta), M.mtla_cache_export(ref))
    finally:
        M.mtla_destroy(ref)
        M.mtla_destroy(sta)


def test_static_scratch_limit_is_reported_and_leaves_the_handle_untouched():
    # 32 heads x r 512: one partial is 64 KB, (148 + 2) of them are far beyond the 4 MiB array.
    w = synth.Workload(name="static_big", dtype="bf16", batch=2, d_model=256, n_heads=32,
                       head_dim=64, latent_rank=512, rope_dim=64, hyper_dim=128, stride=2,
                       prefill_tokens=0, context_tokens=0, decode_steps=2, seed=42)
    h = H.gpu_handle(w, synth.make_weights(w), max_prefill_tokens=0)
    try:
        x = synth.decode_input(w, 0).cuda()
        with pytest.raises(M.MTLAError) as e:
            M.mtla_decode_step_static(h, x)
        assert e.value.status == -9 and "static scratch" in str(e.value)
        assert M.mtla_position(h) == (0, 0, 0)
        M.mtla_decode_step(h, x)                             # the ordinary call still works
        assert M.mtla_position(h) == (1, 1, 2)
    finally:
        M.mtla_destroy(h)


def test_static_scratch_step_allocates_nothing():
    """With y preallocated, neither torch's allocator nor the driver hands out memory during the call."""
    w = layer("bf16", 8, 256, batch=5, context=900).scaled(decode_steps=8)
    weights = synth.make_weights(w)
    n_slots = math.ceil(w.context_tokens / w.stride)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(w.batch)]).cuda()
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        M.mtla_cache_import(h, cache, w.context_tokens)
        x = synth.decode_input(w, 0).cuda()
        y = torch.empty_like(x)
        M.mtla_decode_step_static(h, x, y)                   # first call: symbol lookup, attributes
        torch.cuda.synchronize()
        torch_before = torch.cuda.memory_allocated()
        free_before, _ = torch.cuda.mem_get_info()
        for _ in range(3):
            M.mtla_decode_step_static(h, x, y)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == torch_before
        assert torch.cuda.mem_get_info()[0] == free_before
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


def test_static_scratch_step_on_a_paged_ragged_handle():
    """Per-sequence lengths in paged storage: the static-scratch step against the ordinary one."""
    w = layer("bf16", 8, 256, batch=4, context=0)
    weights = synth.make_weights(w)
    lengths = [130, 900, 901, 2500]
    cfg = M.make_config(**H.dims_of(w), max_batch=w.batch, max_tokens=max(lengths) + 4,
                        max_prefill_tokens=0, dtype="bf16")
    dev = {k: v.cuda() for k, v in weights.items()}
    ref, sta = M.mtla_create_paged(cfg, dev), M.mtla_create_paged(cfg, dev)
    try:
        for b, t in enumerate(lengths):
            row = synth.context_cache_row(w, b, math.ceil(t / w.stride))[None].cuda()
            M.mtla_cache_import_seqs(ref, b, row, t)
            M.mtla_cache_import_seqs(sta, b, row, t)
        for i in range(2):
            x = synth.decode_input(w, i).cuda()
            want = M.mtla_decode_step(ref, x)
            got = M.mtla_decode_step_static(sta, x)
            M.mtla_check(sta)
            H.assert_close(got, want.double().cpu().numpy(), "bf16", f"paged static step {i}")
        assert M.mtla_seq_positions(sta) == M.mtla_seq_positions(ref)
    finally:
        M.mtla_destroy(ref)
        M.mtla_destroy(sta)


def test_static_scratch_limit_boundary_for_the_paper_layer():
    """8 heads, r 256 on the tensor-core path: B = 359 is the largest batch whose partials,
    (maximum, denominator) pairs and tickets fit the 4 MiB array; B = 360 is refused."""
    w = layer("bf16", 8, 256, batch=360, context=0)
    weights = synth.make_weights(w)
    for batch, fits in ((359, True), (360, False)):
        h = H.gpu_handle(w, weights, max_batch=360, max_tokens=8, max_prefill_tokens=0)
        ref = H.gpu_handle(w, weights, max_batch=360, max_tokens=8, max_prefill_tokens=0)
        try:
            x = synth.stored(synth.normal(w.seed, "x_boundary", (batch, w.d_model)), "bf16").cuda()
            if fits:
                got = M.mtla_decode_step_static(h, x)
                want = M.mtla_decode_step(ref, x)
                M.mtla_check(h)
                H.assert_close(got, want.double().cpu().numpy(), "bf16", "boundary batch")
            else:
                with pytest.raises(M.MTLAError) as e:
                    M.mtla_decode_step_static(h, x)
                assert e.value.status == -9
                assert M.mtla_position(h) == (0, 0, 0)
        finally:
            M.mtla_destroy(h)
            M.mtla_destroy(ref)
