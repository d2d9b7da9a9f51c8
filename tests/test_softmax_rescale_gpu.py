"""Parity on inputs that drive the tensor-core attention kernels through their rare branches.

Both attention kernels keep a per-head (decode) or per-row (prefill) softmax reference that is
raised only when a tile's scores outgrow it by more than 2^8; a raise after the first tile
rescales the running output in tensor memory by a factor below one.  With ordinary random inputs
the first tile sets the reference and no later tile ever outgrows it, so these tests build
inputs in which the score level moves from tile to tile:

  * decode: an imported cache whose latent component 0 (or key component 0 of a comparison
    layer) is a constant per 64-slot tile that rises and falls along the sequence, with row 0 of
    W_V zeroed and row 0 of W_K set to a constant, so that the component shifts a tile's scores
    by (a per-head, per-step coefficient) x (the tile's level) and never reaches the values;
  * prefill: input feature 0 carries a level that is constant over the tokens of one key tile
    and climbs along the prompt (three tiles up, one down); it feeds only one component of the
    RoPE key (the slowest pair, with a RoPE base of 1e6 under which that pair turns by a few
    milliradians over the prompt), and a constant feature 1 feeds the same component of every
    head's RoPE query, so every row's scores against a key tile are shifted by the tile's level.

Within a tile the shift is common to all slots and the planted values are exact in bf16, so
neither the rounding of the query nor the bf16 storage of the keys moves the softmax, and the
stated tolerances still apply.

Each test recomputes the scores on the host with the oracle's own pieces, replays the kernels'
reference rule on them (same tile order, same split of the tile list over the CTAs), and asserts
that raises after the first tile - i.e. rescales with a factor below one - really occur.
"""
import math

import numpy as np
import pytest
import torch

from oracle import gqa_oracle as G
from oracle import mtla_oracle as O
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

TILE = 64
RAISE = 8.0          # log2 units: the kernels' threshold
LOG2E = 1.4426950408889634


def sm_count():
    return torch.cuda.get_device_properties(0).multi_processor_count


def tile_levels(n_tiles, step, period=6):
    """Level of tile t: step * (0, 1, .., period, period - 1, .., 1, 0, 1, ..): exact in bf16."""
    t = np.arange(n_tiles) % (2 * period)
    return step * np.where(t <= period, t, 2 * period - t).astype(np.float64)


def shares(tiles_per_seq, grid):
    """The kernel's deal of the sequence-major tile list: for every sequence, the runs of its
    tiles [first, last] that one CTA processes in a row (each run starts a fresh reference)."""
    starts = np.concatenate([[0], np.cumsum(tiles_per_seq)])
    total = int(starts[-1])
    grid = min(grid, total)
    bounds = [c * total // grid for c in range(grid + 1)]
    runs = {b: [] for b in range(len(tiles_per_seq))}
    for c in range(grid):
        g = bounds[c]
        while g < bounds[c + 1]:
            b = int(np.searchsorted(starts, g, side="right") - 1)
            end = min(bounds[c + 1], int(starts[b + 1]))
            runs[b].append((g - int(starts[b]), end - 1 - int(starts[b])))
            g = end
    return runs


def count_raises(scores, runs):
    """scores [heads][slots] in log2 units; replays the lazy reference over each run of tiles.
    Returns (raises after a run's first tile, tiles in which some heads rose and others did not)."""
    n_heads, n = scores.shape
    late, mixed = 0, 0
    for first, last in runs:
        ref = np.full(n_heads, -np.inf)
        for t in range(first, last + 1):
            mt = scores[:, t * TILE:min(n, (t + 1) * TILE)].max(axis=1)
            rise = mt > ref + RAISE
            if t > first:
                late += int(rise.sum())
                mixed += int(rise.any() and not rise.all())
            ref = np.where(rise, mt, ref)
    return late, mixed


def mtla_scores(p, st, x):
    """Eq. 17's scores of the token just consumed against every slot, [heads][slots], in log2
    units (state `st` already holds the token)."""
    pos = st.tokens - 1
    c_hat, kr_hat = np.stack(st.c_hat), np.stack(st.kr_hat)
    q = (x @ p.w_q).reshape(p.n_heads, p.head_dim)
    q_rope = O.rope((x @ p.w_qr).reshape(p.n_heads, p.rope_dim), pos, p.rope_theta)
    keys = (c_hat @ p.w_k).reshape(-1, p.n_heads, p.head_dim)
    e = np.einsum("nhd,hd->hn", keys, q) + q_rope @ kr_hat.T
    return e * LOG2E / math.sqrt(p.head_dim)


def planted_layer(w, key_gain):
    """Weights of w with latent component 0 cut off from the values and given one constant key row."""
    weights = synth.make_weights(w)
    weights["w_v"][0, :] = 0.0
    weights["w_k"][0, :] = key_gain
    return weights


def planted_cache(w, seq, n_slots, step):
    row = synth.context_cache_row(w, seq, n_slots)
    levels = tile_levels(math.ceil(n_slots / TILE), step)
    row[:, 0] = torch.from_numpy(np.repeat(levels, TILE)[:n_slots]).to(row.dtype)
    assert torch.equal(row[:, 0].double(), torch.from_numpy(np.repeat(levels, TILE)[:n_slots]))
    return row


def layer_workload(nh, dh, r, dr, batch, stride, seed):
    return synth.Workload(name="rescale", dtype="bf16", batch=batch, d_model=256, n_heads=nh,
                          head_dim=dh, latent_rank=r, rope_dim=dr, hyper_dim=r // 4, stride=stride,
                          prefill_tokens=0, context_tokens=0, decode_steps=3, seed=seed)


# nh, dh, r, dr, batch, context tokens, stride: many tiles per CTA with the fused combine; a
# sequence spread over many CTAs with the combine as its own launch; the paper's layer shape.
LOCKSTEP = [
    (32, 128, 512, 64, 76, 10200, 2),
    (32, 128, 512, 64, 3, 40000, 2),
    (8, 64, 256, 32, 40, 9000, 3),
]


@pytest.mark.parametrize("nh,dh,r,dr,batch,context,stride", LOCKSTEP)
def test_decode_reference_raises_lockstep(nh, dh, r, dr, batch, context, stride):
    w = layer_workload(nh, dh, r, dr, batch, stride, seed=61).scaled(context_tokens=context)
    weights = planted_layer(w, 0.5)
    p = H.oracle_params(w, weights)
    n_slots = math.ceil(context / stride)
    rows = sorted({0, 1, batch - 1})
    cache = torch.stack([planted_cache(w, b, n_slots, 24.0) for b in range(batch)])
    h = H.gpu_handle(w, weights, max_prefill_tokens=0)
    try:
        assert M.mtla_attention_variant(h) == "tcgen05"
        M.mtla_cache_import(h, cache.cuda(), context)
        states = {b: O.state_from_cache(cache[b].double().numpy(), context, p) for b in rows}
        late = mixed = 0
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            y = M.mtla_decode_step(h, x.cuda())
            M.mtla_check(h)
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in rows])
            H.assert_close(y[rows], want, "bf16", f"step {i}")
            slots_now = states[rows[0]].n_slots
            runs = shares([math.ceil(slots_now / TILE)] * batch, sm_count())
            for b in rows:
                a, m = count_raises(mtla_scores(p, states[b], x[b].double().numpy()), runs[b])
                late, mixed = late + a, mixed + m
        assert late >= 20 and mixed >= 5, (late, mixed)
    finally:
        M.mtla_destroy(h)


def test_decode_reference_raises_ragged_paged():
    """The RAGGED instantiation: sequences of different lengths in 64-slot pages."""
    w = layer_workload(32, 128, 512, 64, 6, 2, seed=62)
    lengths = [700, 5001, 9000, 12000, 12001, 16000]
    weights = planted_layer(w, 0.5)
    p = H.oracle_params(w, weights)
    cfg = M.make_config(**H.dims_of(w), max_batch=w.batch, max_tokens=max(lengths) + 8,
                        max_prefill_tokens=0, dtype="bf16")
    h = M.mtla_create_paged(cfg, {k: v.cuda() for k, v in weights.items()})
    try:
        states = []
        for b, t in enumerate(lengths):
            row = planted_cache(w, b, math.ceil(t / w.stride), 24.0)
            M.mtla_cache_import_seqs(h, b, row[None].cuda(), t)
            states.append(O.state_from_cache(row.double().numpy(), t, p))
        late = mixed = 0
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            y = M.mtla_decode_step(h, x.cuda())
            M.mtla_check(h)
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in range(w.batch)])
            H.assert_close(y, want, "bf16", f"step {i}")
            runs = shares([math.ceil(st.n_slots / TILE) for st in states], sm_count())
            for b in range(w.batch):
                a, m = count_raises(mtla_scores(p, states[b], x[b].double().numpy()), runs[b])
                late, mixed = late + a, mixed + m
        assert late >= 20 and mixed >= 5, (late, mixed)
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("heads,n_kv,dh", [(32, 4, 128), (8, 8, 64)])
def test_decode_reference_raises_comparison_layer(heads, n_kv, dh):
    """The same kernel under mtla_baseline_create: key component 0 carries the tile level."""
    w = synth.WORKLOADS["paper"].scaled(n_heads=heads, head_dim=dh, batch=3, seed=63)
    ctx, step = 6000, 96.0
    weights = synth.make_baseline_weights(w, n_kv)
    p = G.params_from_tensors(
        dict(d_model=w.d_model, n_heads=heads, n_groups=n_kv, head_dim=dh),
        {k: v.double().numpy() for k, v in weights.items()}, rope_theta=w.rope_theta)
    h = M.mtla_baseline_create(d_model=w.d_model, n_heads=heads, n_kv_heads=n_kv, head_dim=dh,
                               max_batch=w.batch, max_tokens=ctx + 8,
                               weights={k: v.cuda() for k, v in weights.items()},
                               rope_theta=w.rope_theta)
    try:
        levels = torch.from_numpy(np.repeat(tile_levels(math.ceil(ctx / TILE), step), TILE)[:ctx])
        cache = torch.stack([torch.stack([synth.kv_cache_plane(w, b, g, ctx) for g in range(n_kv)])
                             for b in range(w.batch)])
        cache[:, :, :, dh] = levels.to(cache.dtype)          # key component 0 of every row
        assert torch.equal(cache[0, 0, :, dh].double(), levels)
        M.mtla_cache_import(h, cache.cuda(), ctx)
        states = [G.state_from_cache(cache[b].double().numpy()) for b in range(w.batch)]
        per_group = heads // n_kv
        late = mixed = 0
        for i in range(3):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (w.batch, w.d_model)), "bf16")
            y = M.mtla_decode_step(h, x.cuda())
            M.mtla_check(h)
            want = np.stack([G.decode_step(p, states[b], x[b].double().numpy()) for b in range(w.batch)])
            H.assert_close(y, want, "bf16", f"step {i}")
            # One "sequence" of the kernel per (sequence, key/value head) plane.
            n_tok = states[0].tokens
            runs = shares([math.ceil(n_tok / TILE)] * (w.batch * n_kv), sm_count())
            for b in range(w.batch):
                q = G.rotate((x[b].double().numpy() @ p.w_q).reshape(heads, dh), n_tok - 1, p.rope_theta)
                keys = np.stack(states[b].keys)                         # [T][g][d_h]
                for g in range(n_kv):
                    e = q[g * per_group:(g + 1) * per_group] @ keys[:, g, :].T * LOG2E / math.sqrt(dh)
                    a, m = count_raises(e, runs[b * n_kv + g])
                    late, mixed = late + a, mixed + m
        assert late >= 20 and (mixed >= 5 or per_group == 1), (late, mixed)
    finally:
        M.mtla_destroy(h)


# ------------------------------------------------------------------------------------ prefill

def climbing_levels(n_tiles, step):
    """Level of key tile t: step * (0, 1, 2, 3, 2, 3, 4, 5, 4, ..): up three tiles, down one."""
    t = np.arange(n_tiles)
    return step * (t - 2 * (t // 4)).astype(np.float64)


def planted_prompt_layer(w, q_gain, step):
    """Feature 0 of the prompt is the level of the key tile its token falls in and reaches only
    the slowest pair of the RoPE key; feature 1 is constant 1 and reaches only the same pair of
    every head's RoPE query.  Both features are cut off from every other projection."""
    weights = synth.make_weights(w)
    pair = w.rope_dim // 2 - 1
    for name in ("w_q", "w_qr", "w_r", "w_kr"):
        weights[name][0:2, :] = 0.0
    # Nothing else reaches that pair, so the stored key component is the level itself, exactly.
    weights["w_kr"][:, 2 * pair:2 * pair + 2] = 0.0
    weights["w_kr"][0, 2 * pair] = 1.0
    for hh in range(w.n_heads):
        weights["w_qr"][:, hh * w.rope_dim + 2 * pair:hh * w.rope_dim + 2 * pair + 2] = 0.0
        weights["w_qr"][1, hh * w.rope_dim + 2 * pair] = q_gain
    prompts = synth.prompt(w)
    tokens_per_tile = TILE * w.stride
    levels = climbing_levels(math.ceil(w.prefill_tokens / tokens_per_tile), step)
    per_token = np.repeat(levels, tokens_per_tile)[: w.prefill_tokens]
    prompts[:, :, 0] = torch.from_numpy(per_token).to(prompts.dtype)
    prompts[:, :, 1] = 1.0
    assert torch.equal(prompts[0, :, 0].double(), torch.from_numpy(per_token))
    return weights, prompts


def replay_prefill_warp(scores, closed, kt=TILE):
    """Replays the prefill kernels' per-warp softmax schedule on the closed-slot scores of 32
    consecutive rows: scores [32][n_closed_max] (log2 units), closed[i] = slots row i may see.
    Returns (fallbacks: fully visible tiles whose sum left the safe range, late raises)."""
    ref = np.full(32, -np.inf)
    fallbacks = raises = 0
    for t in range(math.ceil(int(closed.max()) / kt)):
        lim = closed - t * kt
        tile = scores[:, t * kt:(t + 1) * kt]
        if tile.shape[1] < kt:
            tile = np.pad(tile, ((0, 0), (0, kt - tile.shape[1])), constant_values=-np.inf)
        fast = bool((lim >= kt).all() and np.isfinite(ref).all())
        if fast:
            sums = np.exp2(np.minimum(tile - ref[:, None], 200.0)).sum(axis=1)
            if (sums <= 32768.0).all():
                continue
            fallbacks += 1
        masked = np.where(np.arange(kt)[None, :] < lim[:, None], tile, -np.inf)
        mt = masked.max(axis=1)
        rise = mt > ref + RAISE
        raises += int((rise & np.isfinite(ref)).sum())
        ref = np.where(rise, mt, ref)
    return fallbacks, raises


def prefill_workload(dh, dr, nh, stride, T, batch=2):
    return synth.Workload(name="rescale_pf", dtype="bf16", batch=batch, d_model=256, n_heads=nh,
                          head_dim=dh, latent_rank=256, rope_dim=dr, hyper_dim=64, stride=stride,
                          prefill_tokens=T, context_tokens=0, decode_steps=4, seed=64,
                          rope_theta=1.0e6)


@pytest.mark.parametrize("dh,dr,nh,stride,T", [
    (64, 32, 8, 1, 1100),     # two query tiles per CTA (d_h = 64), plain MLA mask
    (64, 32, 8, 3, 1500),     # stride-aware mask, ragged last chunk
    (128, 64, 4, 1, 1100),    # one query tile per CTA (d_h = 128)
    (128, 64, 4, 3, 1500),
])
def test_prefill_reference_raises(dh, dr, nh, stride, T):
    w = prefill_workload(dh, dr, nh, stride, T)
    weights, prompts = planted_prompt_layer(w, 8.0 if dh == 64 else 12.0, 8.0)
    p = H.oracle_params(w, weights)
    h = H.gpu_handle(w, weights)
    try:
        assert M.mtla_attention_variant(h) == "tcgen05"
        y = M.mtla_prefill(h, prompts.cuda())
        M.mtla_check(h)
        rows = sorted(set(range(0, T, 37)) | set(range(T - 130, T)))
        states = []
        for b in range(w.batch):
            want, st = O.decode_sequence(p, prompts[b].double().numpy(), rows=rows)
            H.assert_close(y[b, rows], want, "bf16", f"prefill seq {b}")
            states.append(st)
        cache = M.mtla_cache_export(h)
        H.assert_cache_close(cache, np.stack([O.cache_array(st) for st in states]), "bf16")
        # The branch really runs: replay the last warp of sequence 0 (rows T-32 .. T-1), head 0.
        fallbacks, raises = replay_last_warp(p, states[0], prompts[0].double().numpy())
        assert fallbacks >= 3 and raises >= 96, (fallbacks, raises)
        # Hand-over: decoding continues from the prefilled state.
        for i in range(w.decode_steps):
            x = synth.decode_input(w, i)
            yd = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in range(w.batch)])
            H.assert_close(yd, want, "bf16", f"decode step {i}")
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


def replay_last_warp(p, st, xs):
    """Scores of rows T-32 .. T-1 (head 0) against the closed slots, through the replay."""
    T, dh, dr, stride = xs.shape[0], p.head_dim, p.rope_dim, p.stride
    n_closed = (T - 1) // stride
    c_hat, kr_hat = np.stack(st.c_hat)[:n_closed], np.stack(st.kr_hat)[:n_closed]
    keys = c_hat @ p.w_k[:, :dh]
    ms = np.arange(T - 32, T)
    q = xs[ms] @ p.w_q[:, :dh]
    q_rope = np.stack([O.rope(xs[m] @ p.w_qr[:, :dr], m, p.rope_theta) for m in ms])
    scores = (q @ keys.T + q_rope @ kr_hat.T) * LOG2E / math.sqrt(dh)
    return replay_prefill_warp(scores, ms // stride)
