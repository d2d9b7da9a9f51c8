"""The tcgen05 projection GEMMs (input projection, query absorption, value and output
projections) through whole decode steps and prefills, against the oracle.

Shapes exercise every activation box height (batch 1 .. 300), a model width that is not a
multiple of the 64-column K block (zero-filled tail), split-K with the ticketed reduction
(few weight tiles) and the unsplit case (many tiles), and per-head K offsets for both head dims.
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


def layer(batch, d, nh, dh, r, dr, stride=2, context=300, steps=3, prefill=0, seed=31):
    return synth.Workload(name="proj", dtype="bf16", batch=batch, d_model=d, n_heads=nh,
                          head_dim=dh, latent_rank=r, rope_dim=dr, hyper_dim=r // 4,
                          stride=stride, prefill_tokens=prefill, context_tokens=context,
                          decode_steps=steps, seed=seed)


@pytest.mark.parametrize("batch,d,nh,dh,r,dr", [
    (1, 256, 8, 64, 128, 32),        # 16-row box, one valid row
    (17, 200, 8, 64, 128, 32),       # 32-row box; d = 200 leaves a K tail of 8 columns
    (33, 512, 8, 64, 256, 32),       # 64-row box, the paper's layer
    (100, 1024, 16, 64, 512, 64),    # 128-row box
    (130, 512, 32, 128, 256, 64),    # 256-row box, head_dim 128
    (300, 256, 4, 64, 128, 32),      # two activation tiles of 256 rows
])
def test_decode_projections_match_oracle(batch, d, nh, dh, r, dr):
    w = layer(batch, d, nh, dh, r, dr)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    n_slots = math.ceil(w.context_tokens / w.stride)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(batch)])
    rows = sorted({0, batch // 2, batch - 1})
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        assert M.mtla_attention_variant(h) == "tcgen05"
        M.mtla_cache_import(h, cache.cuda(), w.context_tokens)
        states = {b: O.state_from_cache(cache[b].double().numpy(), w.context_tokens, p)
                  for b in rows}
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            y = M.mtla_decode_step(h, x.cuda())
            M.mtla_check(h)
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in rows])
            H.assert_close(y[rows], want, "bf16", f"step {i}")
        got = M.mtla_cache_export(h)[rows]
        H.assert_cache_close(got, np.stack([O.cache_array(states[b]) for b in rows]), "bf16")
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("batch,t_len,d,nh,dh,r,dr,stride", [
    (2, 200, 200, 8, 64, 128, 32, 3),      # 400 prompt rows: 3 full panels + a ragged one
    (1, 130, 512, 16, 64, 256, 64, 2),
    (3, 77, 256, 8, 128, 128, 32, 4),
])
def test_prefill_projections_match_oracle(batch, t_len, d, nh, dh, r, dr, stride):
    w = layer(batch, d, nh, dh, r, dr, stride=stride, context=0, steps=2, prefill=t_len)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    prompt = synth.prompt(w)
    h = H.gpu_handle(w, weights)
    try:
        y = M.mtla_prefill(h, prompt.cuda())
        M.mtla_check(h)
        states = []
        for b in range(batch):
            want, st = O.decode_sequence(p, prompt[b].double().numpy())
            H.assert_close(y[b], want, "bf16", f"prefill seq {b}")
            states.append(st)
        H.assert_cache_close(M.mtla_cache_export(h),
                             np.stack([O.cache_array(st) for st in states]), "bf16")
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            yd = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy())
                             for b in range(batch)])
            H.assert_close(yd, want, "bf16", f"decode step {i} after prefill")
    finally:
        M.mtla_destroy(h)


def test_split_k_reduction_is_deterministic():
    """Two handles fed the same inputs give bit-identical outputs (fixed summation order)."""
    w = layer(5, 1024, 8, 64, 128, 32, context=100, steps=4)
    weights = synth.make_weights(w)
    n_slots = math.ceil(w.context_tokens / w.stride)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(5)]).cuda()
    outs = []
    for _ in range(2):
        h = H.gpu_handle(w, weights, max_prefill_tokens=0)
        try:
            M.mtla_cache_import(h, cache, w.context_tokens)
            outs.append(torch.stack([M.mtla_decode_step(h, synth.decode_input(w, i).cuda())
                                     for i in range(w.decode_steps)]).cpu())
        finally:
            M.mtla_destroy(h)
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("batch", [2, 20, 40, 100, 200])
def test_large_layer_projections_match_oracle(batch):
    """The layer of the large workload (d 4096, 32 heads x 128, r 512): the input and output
    projections have few 128-row weight tiles and a 64-block reduction, so they run split over
    K with the ticketed sum of the partials.  One batch per activation box height, 16 to 256
    rows; sampled rows against the oracle, and the whole run twice for bit-equality."""
    w = synth.WORKLOADS["large"].scaled(name="stream", batch=batch, context_tokens=200, decode_steps=3)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    n_slots = math.ceil(w.context_tokens / w.stride)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(batch)])
    rows = sorted({0, 1, batch // 2, batch - 1})
    outs = []
    for rep in range(2):
        h = H.gpu_handle(w, weights, max_prefill_tokens=0)
        try:
            M.mtla_cache_import(h, cache.cuda(), w.context_tokens)
            states = {b: O.state_from_cache(cache[b].double().numpy(), w.context_tokens, p)
                      for b in rows}
            ys = []
            for i in range(w.decode_steps):
                x = synth.decode_input(synth.WORKLOADS["large"], i, batch=batch) if batch <= 128 else \
                    synth.stored(synth.normal(w.seed, f"x200/{i}", (batch, w.d_model)), "bf16")
                y = M.mtla_decode_step(h, x.cuda())
                M.mtla_check(h)
                ys.append(y.cpu())
                if rep == 0:
                    want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in rows])
                    H.assert_close(y[rows], want, "bf16", f"step {i}")
            outs.append(torch.stack(ys))
        finally:
            M.mtla_destroy(h)
    assert torch.equal(outs[0], outs[1])
