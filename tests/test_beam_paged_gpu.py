"""Paged cache, ragged batches and beam re-parenting on the GPU, through the C ABI, against
the CPU oracle's per-sequence states (copied on every re-parenting)."""
import numpy as np
import pytest
import torch

from oracle import mtla_oracle as O
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

PAGE = 64


def paged_handle(w, weights, max_batch, max_tokens, max_prefill, n_pages=0):
    cfg = M.make_config(**H.dims_of(w), max_batch=max_batch, max_tokens=max_tokens,
                        max_prefill_tokens=max_prefill, dtype=w.dtype, ln_eps=w.ln_eps,
                        rope_theta=w.rope_theta)
    return M.mtla_create_paged(cfg, {k: v.cuda() for k, v in weights.items()}, n_pages=n_pages)


def slots_of(tokens, s):
    return -(-tokens // s)


def beam_search_against_oracle(w, n_utt, beam, lengths, steps, reorder_every=1, want_gang=None):
    """Ragged prompts (one per utterance, copied to its `beam` hypotheses by a re-parenting),
    then decode steps with a re-parenting in between; every output is compared.  want_gang:
    the gang size every decode step's attention launch must report."""
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    n_seq = n_utt * beam
    h = paged_handle(w, weights, n_seq, max(lengths) + steps, max(lengths))
    try:
        # One prefill call per utterance builds the ragged batch of n_utt sequences.
        states = []
        for u, t_len in enumerate(lengths):
            x = synth.stored(synth.normal(w.seed, f"utt/{u}", (1, t_len, w.d_model)), w.dtype)
            y = M.mtla_prefill_seqs(h, u, x.cuda())
            want, st = O.decode_sequence(p, x[0].double().numpy())
            H.assert_close(y[0], want, w.dtype, f"prefill of utterance {u}")
            states.append(st)
        assert M.mtla_seq_positions(h) == list(lengths)
        assert M.mtla_pages_in_use(h) == sum(-(-slots_of(t, w.stride) // PAGE) for t in lengths)
        # Fork every utterance into its beam.
        parents = [u for u in range(n_utt) for _ in range(beam)]
        M.mtla_beam_reorder(h, parents)
        states = O.reorder_states(states, parents)
        assert M.mtla_pages_in_use(h) == sum(-(-slots_of(t, w.stride) // PAGE) for t in lengths)
        for i in range(steps):
            x = synth.stored(synth.normal(w.seed, f"beam_x/{i}", (n_seq, w.d_model)), w.dtype)
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in range(n_seq)])
            H.assert_close(y, want, w.dtype, f"decode step {i}")
            assert M.mtla_seq_positions(h) == [st.tokens for st in states]
            if want_gang is not None:
                assert M.mtla_attention_gang(h) == want_gang, f"decode step {i}"
            if (i + 1) % reorder_every == 0:
                parents = synth.beam_parents(w.seed, i, n_utt, beam)
                M.mtla_beam_reorder(h, parents)
                states = O.reorder_states(states, parents)
        M.mtla_check(h)
        assert M.mtla_cache_bytes(h) == sum(st.n_slots for st in states) * w.slot_width * (
            4 if w.dtype == "fp32" else 2)
        for b in range(n_seq):
            H.assert_cache_close(M.mtla_cache_export_seq(h, b), O.cache_array(states[b]), w.dtype)
        # Shared pages count once: never more than unshared storage would need.
        assert M.mtla_pages_in_use(h) <= sum(-(-st.n_slots // PAGE) for st in states)
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("s", [1, 2, 3])
def test_beam_search_fp32(s):
    """CUDA-core path at fp32 tolerance; prompts below, at and above a page boundary."""
    w = synth.WORKLOADS["tiny"].scaled(stride=s, seed=20 + s)
    lengths = [PAGE * s - 1, PAGE * s, PAGE * s + 1, 5, 2 * PAGE * s + s + 1]
    beam_search_against_oracle(w, n_utt=5, beam=3, lengths=lengths, steps=2 * s + 70)


@pytest.mark.parametrize("s,heads", [(2, 8), (3, 32)])
def test_beam_search_bf16_tensor_cores(s, heads):
    w = synth.WORKLOADS["paper"].scaled(stride=s, n_heads=heads, seed=30 + s)
    lengths = [PAGE * s * 2 + 3, 17, PAGE * s, 3 * PAGE * s - 1]
    beam_search_against_oracle(w, n_utt=4, beam=4, lengths=lengths, steps=40)


@pytest.mark.parametrize("beam,gang,heads,s", [(4, 4, 8, 2), (8, 8, 32, 2), (5, 5, 8, 3), (50, 10, 8, 2),
                                               (3, 3, 16, 1)])
def test_beams_walk_shared_pages_as_a_gang(beam, gang, heads, s):
    """Every utterance is longer than a page, so its beams share their first page and the
    attention launch co-schedules them (gang = the largest divisor of the beam that leaves at
    most a tenth of the SMs idle: 50 -> 10).  Utterances of different lengths: the gangs' shares
    end inside and at the ends of sequences; the step count crosses a page boundary, where every
    beam opens a page of its own."""
    w = synth.WORKLOADS["paper"].scaled(stride=s, n_heads=heads, seed=40 + beam)
    n_utt = 3 if beam < 50 else 2
    lengths = [PAGE * s * 3 + 5, PAGE * s + 1, PAGE * s * 6 - 2 * s][:n_utt]
    beam_search_against_oracle(w, n_utt=n_utt, beam=beam, lengths=lengths, steps=3 * s + 6,
                               want_gang=gang)


def test_gang_needs_most_blocks_to_share_their_first_page():
    """One utterance shorter than a page (each beam copies and writes that page: nothing
    shared) among longer ones keeps the gangs; a batch of mostly short utterances does not."""
    w = synth.WORKLOADS["paper"].scaled(stride=2, seed=47)
    beam_search_against_oracle(w, n_utt=3, beam=4, lengths=[PAGE * 2 * 2 + 3, 17, PAGE * 2 * 3],
                               steps=5, want_gang=4)
    beam_search_against_oracle(w, n_utt=3, beam=4, lengths=[9, 17, PAGE * 2 * 3], steps=5, want_gang=1)


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("paper", {"prefill_tokens": 300, "decode_steps": 140})])
def test_lock_step_on_a_paged_handle_is_bit_identical(name, kw):
    """Same kernels, same order of operations: only the slot addresses differ."""
    w = synth.WORKLOADS[name].scaled(batch=3, **kw)
    weights = synth.make_weights(w)
    flat = H.gpu_handle(w, weights, max_tokens=w.max_tokens + 1)
    paged = paged_handle(w, weights, w.batch, w.max_tokens + 1, w.prefill_tokens)
    try:
        x = synth.prompt(w).cuda()
        assert torch.equal(M.mtla_prefill(flat, x), M.mtla_prefill(paged, x))
        for i in range(w.decode_steps):
            xi = synth.decode_input(w, i).cuda()
            assert torch.equal(M.mtla_decode_step(flat, xi), M.mtla_decode_step(paged, xi)), i
        assert torch.equal(M.mtla_cache_export(flat), M.mtla_cache_export(paged))
        assert M.mtla_position(flat) == M.mtla_position(paged)
        # Export, re-import into the paged handle, continue: still identical.
        cache = M.mtla_cache_export(flat)
        tokens = M.mtla_position(flat)[0]
        M.mtla_cache_import(paged, cache, tokens)
        xi = synth.decode_input(w, 0).cuda()
        assert torch.equal(M.mtla_decode_step(flat, xi), M.mtla_decode_step(paged, xi))
        M.mtla_check(flat)
        M.mtla_check(paged)
    finally:
        M.mtla_destroy(flat)
        M.mtla_destroy(paged)


def test_pool_exhaustion_is_reported_before_anything_runs():
    w = synth.WORKLOADS["tiny"].scaled(batch=2)
    weights = synth.make_weights(w)
    h = paged_handle(w, weights, 2, 4 * PAGE * w.stride, 2 * PAGE * w.stride, n_pages=3)
    try:
        x = synth.prompt(w, batch=2, tokens=PAGE * w.stride).cuda()      # one full page each
        M.mtla_prefill(h, x)
        xi = synth.decode_input(w, 0, batch=2).cuda()
        with pytest.raises(M.MTLAError) as err:      # both sequences need a second page; one is left
            M.mtla_decode_step(h, xi)
        assert err.value.status == -4
        assert M.mtla_seq_positions(h) == [PAGE * w.stride] * 2 and M.mtla_pages_in_use(h) == 2
        M.mtla_beam_reorder(h, [1])                  # keep one hypothesis: its page need fits
        M.mtla_decode_step(h, xi[:1].contiguous())
        assert M.mtla_seq_positions(h) == [PAGE * w.stride + 1] and M.mtla_pages_in_use(h) == 2
        M.mtla_reset(h)
        assert M.mtla_pages_in_use(h) == 0 and M.mtla_position(h) == (0, 0, 0)
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


def test_paging_calls_are_refused_without_paging():
    w = synth.WORKLOADS["tiny"]
    h = H.gpu_handle(w, synth.make_weights(w))
    try:
        with pytest.raises(M.MTLAError) as err:
            M.mtla_beam_reorder(h, [0])
        assert err.value.status == -7
        with pytest.raises(M.MTLAError) as err:
            M.mtla_prefill_seqs(h, 0, synth.prompt(w).cuda())
        assert err.value.status == -7
        assert M.mtla_pages_in_use(h) == -1
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_prefill_of_several_sequences_behind_existing_ones(dtype):
    """mtla_prefill_seqs with B > 1 and seq0 > 0, and a cache import in between."""
    base = synth.WORKLOADS["tiny"] if dtype == "fp32" else synth.WORKLOADS["paper"]
    w = base.scaled(stride=3, seed=77)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    h = paged_handle(w, weights, 6, 400, 150)
    try:
        states = []

        def prefill(seq0, n, t_len):
            x = synth.stored(synth.normal(w.seed, f"pp/{seq0}", (n, t_len, w.d_model)), w.dtype)
            y = M.mtla_prefill_seqs(h, seq0, x.cuda())
            for b in range(n):
                want, st = O.decode_sequence(p, x[b].double().numpy())
                H.assert_close(y[b], want, w.dtype, f"prefill of sequence {seq0 + b}")
                states.append(st)

        prefill(0, 1, 100)
        prefill(1, 3, 70)                     # three sequences behind the first
        row = synth.context_cache_row(w, 4, 41)          # 122 tokens: the last slot is open
        M.mtla_cache_import_seqs(h, 4, row[None].cuda(), 122)
        states.append(O.state_from_cache(row.double().numpy(), 122, p))
        prefill(5, 1, 150)
        assert M.mtla_seq_positions(h) == [100, 70, 70, 70, 122, 150]
        for i in range(8):
            x = synth.stored(synth.normal(w.seed, f"px/{i}", (6, w.d_model)), w.dtype)
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in range(6)])
            H.assert_close(y, want, w.dtype, f"decode step {i}")
        M.mtla_check(h)
        with pytest.raises(M.MTLAError) as err:       # sequence 2 is not empty
            M.mtla_prefill_seqs(h, 2, synth.prompt(w, batch=1, tokens=8).cuda())
        assert err.value.status == -7
    finally:
        M.mtla_destroy(h)
