"""Decoder layers and stacks on the GPU (mtla_stack_* through the C ABI) against the decoder
oracle: pre-norm layers of MTLA self-attention plus a ReLU feed-forward block, a final LayerNorm
(Section 5.2 and the appendix on hyper-parameters: 9 layers, d 512, feed-forward 2048, 8 heads).

The prompt goes through the parallel prefill of every layer (the oracle's layer-by-layer order),
decoding continues token by token; every output and every layer's cache are compared."""
import math

import numpy as np
import pytest
import torch

from oracle import decoder_oracle as D
from oracle import mtla_oracle as O
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def stack_workload(dtype, n_layers, d, nh, dh, r, dr, d_ff, stride, batch, prompt, steps, seed=71):
    w = synth.Workload(name="stack", dtype=dtype, batch=batch, d_model=d, n_heads=nh, head_dim=dh,
                       latent_rank=r, rope_dim=dr, hyper_dim=max(r // 4, 8), stride=stride,
                       prefill_tokens=prompt, context_tokens=0, decode_steps=steps, seed=seed)
    return synth.StackWorkload("stack", w, n_layers, d_ff)


def run_stack(sw, seqs=None, prefill_rows=None, steps_checked=None):
    w = sw.layer
    weights = synth.make_stack_weights(sw)
    sp = H.oracle_stack_params(sw, weights)
    s = H.gpu_stack(sw, weights)
    seqs = list(range(w.batch)) if seqs is None else seqs
    try:
        prompts = synth.prompt(w)
        y = M.mtla_stack_prefill(s, prompts.cuda())
        M.mtla_stack_check(s)
        states = {}
        for b in seqs:
            want, st = D.stack_forward_by_layers(sp, prompts[b].double().numpy(), rows=prefill_rows)
            got = y[b] if prefill_rows is None else y[b, prefill_rows]
            H.assert_close_stack(got, want, w.dtype, sw.n_layers, f"prefill seq {b}")
            states[b] = st
        slots = math.ceil(w.prefill_tokens / w.stride)
        elem = 4 if w.dtype == "fp32" else 2
        assert M.mtla_stack_cache_bytes(s) == sw.n_layers * w.batch * slots * w.slot_width * elem
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            yd = M.mtla_stack_decode_step(s, x.cuda())
            check = steps_checked is None or i in steps_checked
            want = [D.stack_decode_step(sp, states[b], x[b].double().numpy()) for b in seqs]
            if check:
                H.assert_close_stack(yd[seqs], np.stack(want), w.dtype, sw.n_layers, f"decode step {i}")
        M.mtla_stack_check(s)
        tokens = w.prefill_tokens + w.decode_steps
        # Cache rows: a layer inside a stack reads the bf16 rounding of LayerNorm_1(stream), which
        # the oracle does not round, and from the second layer on also the error the stream has
        # accumulated; the single-layer bound (a few storage ulps) is therefore taken three times
        # wider at the first layer and grows like the outputs' bound, with sqrt(layer).
        for n in range(sw.n_layers):
            layer = M.mtla_stack_layer(s, n)
            assert M.mtla_position(layer) == (tokens, math.ceil(tokens / w.stride), w.batch)
            cache = M.mtla_cache_export(layer)
            H.assert_cache_close(cache[seqs], np.stack([O.cache_array(states[b].layers[n]) for b in seqs]),
                                 w.dtype, scale=3.0 * math.sqrt(n + 1))
    finally:
        M.mtla_stack_destroy(s)


@pytest.mark.parametrize("dtype,n_layers,d,nh,dh,r,dr,d_ff,stride,batch,prompt,steps", [
    ("fp32", 2, 128, 4, 64, 64, 32, 256, 2, 2, 37, 6),       # CUDA-core path end to end
    ("bf16", 3, 256, 8, 64, 128, 32, 512, 3, 3, 70, 6),      # tensor-core path, ragged last chunk
    ("bf16", 2, 256, 4, 128, 256, 64, 1024, 1, 2, 130, 4),   # d_h 128, plain-MLA layers (s = 1)
    ("bf16", 2, 192, 4, 64, 64, 32, 384, 2, 2, 33, 4),       # bf16 off the tensor-core path (r = 64)
])
def test_small_stacks_every_output(dtype, n_layers, d, nh, dh, r, dr, d_ff, stride, batch, prompt, steps):
    run_stack(stack_workload(dtype, n_layers, d, nh, dh, r, dr, d_ff, stride, batch, prompt, steps))


def test_the_papers_decoder():
    """9 layers, d 512, 8 heads x 64, r 256, d_R 32, hyper-network 64, feed-forward 2048, s 2:
    a 300-token prompt for 8 sequences, then 24 decode steps."""
    base = synth.STACK_WORKLOADS["decoder_paper"]
    sw = synth.StackWorkload("decoder_paper_test", base.layer.scaled(batch=8, prefill_tokens=300,
                                                                     decode_steps=24), 9, 2048)
    rows = sorted(set(range(0, 300, 7)) | {298, 299})
    run_stack(sw, seqs=[0, 3, 7], prefill_rows=rows, steps_checked={0, 1, 2, 11, 23})


def test_decode_from_empty_and_errors():
    sw = stack_workload("bf16", 2, 256, 8, 64, 128, 32, 512, 2, 2, 0, 5)
    w = sw.layer
    weights = synth.make_stack_weights(sw)
    sp = H.oracle_stack_params(sw, weights)
    s = H.gpu_stack(sw, weights, max_prefill_tokens=0)
    try:
        x_bad = synth.stored(synth.normal(1, "xb", (3, w.d_model)), "bf16").cuda()
        with pytest.raises(M.MTLAError) as e:
            M.mtla_stack_decode_step(s, x_bad)               # batch beyond max_batch
        assert e.value.status == -4
        with pytest.raises(M.MTLAError) as e:
            M.mtla_stack_prefill(s, x_bad[None][:, :2].contiguous())   # no prefill workspace
        assert e.value.status == -4
        states = [D.StackState.empty(2) for _ in range(w.batch)]
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            y = M.mtla_stack_decode_step(s, x.cuda())
            want = np.stack([D.stack_decode_step(sp, states[b], x[b].double().numpy())
                             for b in range(w.batch)])
            H.assert_close_stack(y, want, "bf16", 2, f"step {i}")
        with pytest.raises(M.MTLAError) as e:
            M.mtla_stack_decode_step(s, synth.decode_input(w, 0).cuda())   # max_tokens reached
        assert e.value.status == -4
        M.mtla_stack_reset(s)
        assert M.mtla_stack_cache_bytes(s) == 0
        assert M.mtla_stack_launch_count(s) > 0
    finally:
        M.mtla_stack_destroy(s)
