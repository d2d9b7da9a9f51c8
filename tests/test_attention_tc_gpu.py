"""The tcgen05 decode-attention kernel against the oracle (and against the CUDA-core kernel).

Shapes cover both head paddings (16 / 32), every latent block count r/128 in 1..4, both
RoPE widths, single-tile splits, multi-tile pipelines with ring wrap-around, and ragged tails.
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


def workload(nh, dh, r, dr, batch, context, stride=2, d=256, seed=21):
    return synth.Workload(name="tc", dtype="bf16", batch=batch, d_model=d, n_heads=nh,
                          head_dim=dh, latent_rank=r, rope_dim=dr, hyper_dim=r // 4,
                          stride=stride, prefill_tokens=0, context_tokens=context,
                          decode_steps=3, seed=seed)


def run(w, rows, variant=None):
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    n_slots = math.ceil(w.context_tokens / w.stride)
    cache = torch.stack([synth.context_cache_row(w, b, n_slots) for b in range(w.batch)])
    h = H.gpu_handle(w, weights, max_prefill_tokens=0,
                     kernel_path=M.MTLA_PATH_CUDA_CORE if variant == "fma" else M.MTLA_PATH_AUTO)
    outs = []
    try:
        assert M.mtla_attention_variant(h) == (variant or "tcgen05")
        M.mtla_cache_import(h, cache.cuda(), w.context_tokens)
        states = {b: O.state_from_cache(cache[b].double().numpy(), w.context_tokens, p)
                  for b in rows}
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            y = M.mtla_decode_step(h, x.cuda())
            M.mtla_check(h)
            outs.append(y.cpu())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in rows])
            H.assert_close(y[list(rows)], want, "bf16", f"step {i}")
    finally:
        M.mtla_destroy(h)
    return torch.stack(outs)


SHAPES = [
    # nh, dh,  r,  dr, batch, context tokens
    (32, 128, 512, 64, 2, 700),      # 3 splits of one tile each, ragged last tile
    (32, 128, 512, 64, 80, 700),     # one CTA per sequence, 3 tiles through the ring
    (8, 64, 256, 32, 3, 1500),       # padded heads (16), 32-wide RoPE chunk zero-filled by TMA
    (16, 64, 512, 64, 80, 900),
    (4, 64, 128, 32, 80, 2100),      # one pair per tile
    (32, 64, 384, 64, 80, 1100),     # three pairs per tile
    (32, 128, 512, 64, 76, 10200),   # 40 tiles per CTA: ring and barrier phases wrap many times
]


@pytest.mark.parametrize("nh,dh,r,dr,batch,context", SHAPES)
def test_tc_attention_matches_oracle(nh, dh, r, dr, batch, context):
    w = workload(nh, dh, r, dr, batch, context)
    rows = sorted({0, 1, batch - 1})
    run(w, rows)


def test_tc_and_fma_kernels_agree():
    w = workload(32, 128, 512, 64, 5, 3000, stride=3)
    y_tc = run(w, [0, 4])
    y_fma = run(w, [0, 4], "fma")
    diff = (y_tc.float() - y_fma.float()).abs().max().item()
    assert diff <= 2e-2


def test_tc_attention_single_slot_and_tile_boundaries():
    """Decode from an empty cache across the 128 / 129 slot boundary at s = 1."""
    w = workload(32, 64, 256, 32, 2, 0, stride=1).scaled(decode_steps=131)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        states = [O.State(), O.State()]
        for i in range(131):
            x = synth.decode_input(w, i)
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in range(2)])
            if i in (0, 1, 2, 126, 127, 128, 129, 130):
                H.assert_close(y, want, "bf16", f"step {i}")
        M.mtla_check(h)
        assert M.mtla_position(h) == (131, 131, 2)
    finally:
        M.mtla_destroy(h)
