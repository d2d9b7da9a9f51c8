"""The five benchmark configurations at their full sizes, in the launch configuration the
benchmark times, against the CPU oracle on sampled outputs.

The oracle cannot follow every row of these workloads, so each test follows a few whole
sequences through the oracle's state updates (cheap) and asks it for the attention output only
at sampled prefill rows and decode steps; slot counts, cache bytes and positions are checked
exactly for the whole batch, and the exported cache of the sampled sequences element by element.
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


def elem_bytes(w):
    return 4 if w.dtype == "fp32" else 2


def check_positions(h, w, tokens):
    slots = math.ceil(tokens / w.stride)
    assert M.mtla_position(h) == (tokens, slots, w.batch)
    assert M.mtla_cache_bytes(h) == w.batch * slots * w.slot_width * elem_bytes(w)


def run_prefill_then_decode(w, seqs, prefill_rows, decode_steps_checked, rows_by_seq=None):
    """Prefill the whole batch, then decode w.decode_steps steps; compare sampled outputs.
    rows_by_seq overrides the sampled prefill rows for individual sequences."""
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    h = H.gpu_handle(w, weights)
    try:
        x = torch.empty(w.batch, w.prefill_tokens, w.d_model, dtype=synth.torch_dtype(w.dtype),
                        device="cuda")
        prompts = {}
        for b in range(w.batch):
            row = synth.stored(synth.normal(w.seed, f"prompt/{b}", (w.prefill_tokens, w.d_model)),
                               w.dtype)
            x[b].copy_(row)
            if b in seqs:
                prompts[b] = row.double().numpy()
        y = M.mtla_prefill(h, x)
        M.mtla_check(h)
        check_positions(h, w, w.prefill_tokens)
        states = {}
        for b in seqs:
            rows_b = (rows_by_seq or {}).get(b, prefill_rows)
            want, st = O.decode_sequence(p, prompts[b], rows=rows_b)
            H.assert_close(y[b, rows_b], want, w.dtype, f"prefill seq {b}")
            states[b] = st
        cache = M.mtla_cache_export(h)
        H.assert_cache_close(cache[seqs], np.stack([O.cache_array(states[b]) for b in seqs]), w.dtype)
        del x, y, cache
        for i in range(w.decode_steps):
            xi = synth.decode_input(w, i)
            yi = M.mtla_decode_step(h, xi.cuda())
            check = i in decode_steps_checked
            want = [O.decode_step(p, states[b], xi[b].double().numpy(), want_output=check)
                    for b in seqs]
            if check:
                M.mtla_check(h)
                H.assert_close(yi[seqs], np.stack(want), w.dtype, f"decode step {i}")
        check_positions(h, w, w.prefill_tokens + w.decode_steps)
        cache = M.mtla_cache_export(h)
        H.assert_cache_close(cache[seqs], np.stack([O.cache_array(states[b]) for b in seqs]), w.dtype)
    finally:
        M.mtla_destroy(h)


def test_config_tiny_every_output():
    """fp32, batch 1: every prefill row and every decode step is compared."""
    w = synth.WORKLOADS["tiny"]
    run_prefill_then_decode(w, [0], list(range(w.prefill_tokens)), set(range(w.decode_steps)))


def test_config_paper_scale():
    w = synth.WORKLOADS["paper"]
    rows = [0, 1, 2, 3, 127, 128, 129, 511, 1000, 1022, 1023]
    steps = {0, 1, 2, 63, 64, 500, 1022, 1023}
    run_prefill_then_decode(w, [0, 17, 31], rows, steps)


@pytest.mark.parametrize("s", [1, 2, 3, 4])
def test_config_stride_sweep(s):
    """4096 = 3 * 1365 + 1: at s = 3 the prompt leaves an open slot that decoding continues."""
    w = synth.WORKLOADS[f"sweep_s{s}"]
    rows = [0, 1, 5, 6, 63, 64, 65, 2047, 4094, 4095]
    steps = {0, 1, 2, 3, 128, 255}
    run_prefill_then_decode(w, [0, 63], rows, steps)


def test_config_long_context_prefill():
    """Sequence 0: every row of the first, a middle and the last pair of 128-row query tiles (one
    CTA of the two-tile kernel each); sequence 7: scattered rows."""
    w = synth.WORKLOADS["longctx"]
    rows = [0, 3, 4, 255, 256, 8191, 16380, 16383]
    pairs = sorted(set(range(0, 256)) | set(range(8192, 8448)) | set(range(16128, 16384)) | set(rows))
    run_prefill_then_decode(w, [0, 7], rows, {0, 1, 3, 4, 63}, rows_by_seq={0: pairs})


def test_large_layer_prefill_then_decode():
    """The layer of the large workload (d 4096, 32 heads x 128, r 512, d_R 64, s 2) through the
    prefill and into decoding: B 2, T 2048.  Whole first and last query tiles, the rows around the
    middle, then six decode steps from the handed-over state."""
    w = synth.WORKLOADS["large"].scaled(name="large_prefill", batch=2, prefill_tokens=2048,
                                        context_tokens=0, decode_steps=6)
    rows = sorted(set(range(0, 128)) | set(range(1016, 1032)) | set(range(1920, 2048)))
    run_prefill_then_decode(w, [0, 1], rows, set(range(6)))


def test_config_large_decode():
    """Batch 128 over an imported 32768-token context, as bench.py runs it."""
    w = synth.WORKLOADS["large"]
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    seqs = [0, 1, w.batch - 1]
    n_slots = math.ceil(w.context_tokens / w.stride)
    cfg = M.make_config(**H.dims_of(w), max_batch=w.batch,
                        max_tokens=w.context_tokens + w.decode_steps, max_prefill_tokens=0,
                        dtype=w.dtype, ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    h = M.mtla_create(cfg, {k: v.cuda() for k, v in weights.items()})
    try:
        cache = torch.empty(w.batch, n_slots, w.slot_width, dtype=torch.bfloat16, device="cuda")
        states = {}
        for b in range(w.batch):
            row = synth.context_cache_row(w, b)
            cache[b].copy_(row)
            if b in seqs:
                states[b] = O.state_from_cache(row.double().numpy(), w.context_tokens, p)
        M.mtla_cache_import(h, cache, w.context_tokens)
        del cache
        check_positions(h, w, w.context_tokens)
        checked = {0, 1, 2, 64, 127}
        for i in range(w.decode_steps):
            xi = synth.decode_input(w, i)
            yi = M.mtla_decode_step(h, xi.cuda())
            check = i in checked
            want = [O.decode_step(p, states[b], xi[b].double().numpy(), want_output=check)
                    for b in seqs]
            if check:
                M.mtla_check(h)
                H.assert_close(yi[seqs], np.stack(want), "bf16", f"decode step {i}")
        check_positions(h, w, w.context_tokens + w.decode_steps)
        # The 64 slots the decode steps wrote, element by element, for the sampled sequences.
        tail = M.mtla_cache_export(h)[seqs, n_slots:]
        want_tail = np.stack([O.cache_array(states[b])[n_slots:] for b in seqs])
        H.assert_cache_close(tail, want_tail, "bf16")
    finally:
        M.mtla_destroy(h)


def run_beam_workload(bw, utts, beams_checked, steps_checked):
    """Beam search on a paged handle at the workload's full size: ragged contexts imported per
    utterance, forked into beams, a re-parenting after every step.  The oracle follows whole
    beams of the sampled utterances (state updates every step, outputs at the sampled steps)."""
    w = bw.layer
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    contexts = bw.contexts()
    s, beam = w.stride, bw.beam

    def pages(tokens):
        return -(-math.ceil(tokens / s) // M.PAGE_SLOTS)

    cfg = M.make_config(**H.dims_of(w), max_batch=bw.n_seq, max_tokens=max(contexts) + bw.decode_steps,
                        max_prefill_tokens=0, dtype=w.dtype, ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    # A pool that only fits because beams share their utterance's closed pages.
    n_pages = sum(pages(t) for t in contexts) + bw.n_seq * (pages(bw.decode_steps) + 2)
    assert n_pages < sum(beam * pages(t + bw.decode_steps) for t in contexts)
    h = M.mtla_create_paged(cfg, {k: v.cuda() for k, v in weights.items()}, n_pages=n_pages)
    try:
        states = {}
        for u, t in enumerate(contexts):
            row = synth.context_cache_row(w, u, math.ceil(t / s))
            M.mtla_cache_import_seqs(h, u, row[None].cuda(), t)
            if u in utts:
                states[u] = [O.state_from_cache(row.double().numpy(), t, p)]
        assert M.mtla_seq_positions(h) == contexts
        M.mtla_beam_reorder(h, [u for u in range(bw.n_utt) for _ in range(beam)])
        for u in utts:
            states[u] = O.reorder_states(states[u], [0] * beam)
        assert M.mtla_pages_in_use(h) == sum(pages(t) for t in contexts)
        for i in range(bw.decode_steps):
            x = synth.stored(synth.normal(w.seed, f"beam_x/{i}", (bw.n_seq, w.d_model)), w.dtype)
            y = M.mtla_decode_step(h, x.cuda())
            check = i in steps_checked
            for u in utts:
                for k in range(beam):
                    b = u * beam + k
                    want = O.decode_step(p, states[u][k], x[b].double().numpy(),
                                         want_output=check and k in beams_checked)
                    if want is not None:
                        H.assert_close(y[b], want, w.dtype, f"step {i}, utterance {u}, beam {k}")
            if check:
                M.mtla_check(h)
            parents = synth.beam_parents(w.seed, i, bw.n_utt, beam)
            M.mtla_beam_reorder(h, parents)
            for u in utts:
                states[u] = O.reorder_states(states[u], [q - u * beam for q in parents[u * beam:(u + 1) * beam]])
        M.mtla_check(h)
        assert M.mtla_seq_positions(h) == [t + bw.decode_steps for t in contexts for _ in range(beam)]
        assert M.mtla_position(h) == (max(contexts) + bw.decode_steps,
                                      math.ceil((max(contexts) + bw.decode_steps) / s), bw.n_seq)
        assert M.mtla_cache_bytes(h) == sum(beam * math.ceil((t + bw.decode_steps) / s) for t in contexts) * (
            w.slot_width * elem_bytes(w))
        assert M.mtla_pages_in_use(h) <= n_pages
        for u in utts:
            for k in beams_checked:
                H.assert_cache_close(M.mtla_cache_export_seq(h, u * beam + k),
                                     O.cache_array(states[u][k]), w.dtype)
    finally:
        M.mtla_destroy(h)


def test_beam_search_paper_scale():
    """24 utterances x beam 10 on the paper's layer; three whole beams followed at every step."""
    bw = synth.BEAM_WORKLOADS["beam_paper"]
    run_beam_workload(bw, [0, 11, 23], set(range(bw.beam)), set(range(bw.decode_steps)))


def test_beam_search_large():
    """16 utterances x beam 8 at the large layer's size, contexts of 8k to 32k tokens."""
    bw = synth.BEAM_WORKLOADS["beam_large"]
    run_beam_workload(bw, [0, 15], {0, 3, 7}, {0, 1, 40, 71})
