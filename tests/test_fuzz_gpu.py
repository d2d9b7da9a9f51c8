"""Seeded random layer shapes and call sequences through the C ABI against the CPU oracle:
head counts that are not powers of two, odd hyper-network widths, strides up to 6, ranks on and
off the tensor-core path, contiguous and paged storage, ragged prompts, re-parenting."""
import numpy as np
import pytest
import torch

from oracle import mtla_oracle as O
from paper_2505_13544_b200 import binding as M
from paper_2505_13544_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def assert_close_scaled(got, want, dtype, what):
    """The specification's tolerance, with the bf16 absolute bound following the output's size:
    random layers at s = 5, 6 give outputs above 4, where rounding y to bf16 alone costs up to
    2^-8 |y| and the bf16 storage of the merged latents about as much again, so the bound is
    max(2e-2, 2^-7 max|y|); the relative L2 bound stays as it is."""
    if dtype == "fp32":
        return H.assert_close(got, want, dtype, what)
    g = got.detach().double().cpu().numpy()
    want = np.asarray(want, dtype=np.float64)
    assert g.shape == want.shape and np.isfinite(g).all(), what
    err = np.abs(g - want).max()
    bound = max(H.BF16_MAX_ABS, 2.0 ** -7 * np.abs(want).max())
    rel = np.linalg.norm(g - want) / max(np.linalg.norm(want), 1e-30)
    assert err <= bound, f"{what}: max abs err {err:.3e} > {bound:.3e}"
    assert rel <= H.BF16_REL_L2, f"{what}: rel L2 err {rel:.3e} > {H.BF16_REL_L2}"


def draw(seed):
    g = np.random.Generator(np.random.Philox(key=[seed, 0x5eed]))
    dtype = "fp32" if seed % 3 == 2 else "bf16"
    pick = lambda xs: xs[int(g.integers(len(xs)))]
    w = synth.Workload(
        name=f"fuzz{seed}", dtype=dtype, batch=int(g.integers(1, 7)),
        d_model=8 * int(g.integers(8, 49)), n_heads=int(g.integers(1, 9 if dtype == "fp32" else 33)),
        head_dim=pick([64, 128]), latent_rank=64 * int(g.integers(1, 9)), rope_dim=pick([32, 64]),
        hyper_dim=int(g.integers(1, 65)), stride=int(g.integers(1, 7)),
        prefill_tokens=0, context_tokens=0, decode_steps=int(g.integers(8, 25)), seed=1000 + seed)
    paged = bool(g.integers(2))
    lengths = [int(g.integers(1, 201)) for _ in range(w.batch)]
    if not paged:
        lengths = [lengths[0]] * w.batch
    reorders = {int(v) for v in g.integers(0, w.decode_steps, size=3)} if paged else set()
    return w, paged, lengths, reorders, g


@pytest.mark.parametrize("seed", range(64))
def test_random_layer_and_call_sequence(seed):
    w, paged, lengths, reorders, g = draw(seed)
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    cfg = M.make_config(**H.dims_of(w), max_batch=w.batch, max_tokens=max(lengths) + w.decode_steps,
                        max_prefill_tokens=max(lengths), dtype=w.dtype, ln_eps=w.ln_eps,
                        rope_theta=w.rope_theta)
    dev = {k: v.cuda() for k, v in weights.items()}
    h = M.mtla_create_paged(cfg, dev) if paged else M.mtla_create(cfg, dev)
    try:
        states = []
        if paged:
            for b, t in enumerate(lengths):
                x = synth.stored(synth.normal(w.seed, f"p/{b}", (1, t, w.d_model)), w.dtype)
                y = M.mtla_prefill_seqs(h, b, x.cuda())
                want, st = O.decode_sequence(p, x[0].double().numpy())
                assert_close_scaled(y[0], want, w.dtype, f"prefill {b}")
                states.append(st)
        else:
            x = torch.stack([synth.stored(synth.normal(w.seed, f"p/{b}", (lengths[0], w.d_model)), w.dtype)
                             for b in range(w.batch)])
            y = M.mtla_prefill(h, x.cuda())
            for b in range(w.batch):
                want, st = O.decode_sequence(p, x[b].double().numpy())
                assert_close_scaled(y[b], want, w.dtype, f"prefill {b}")
                states.append(st)
        for i in range(w.decode_steps):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (w.batch, w.d_model)), w.dtype)
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in range(w.batch)])
            assert_close_scaled(y, want, w.dtype, f"step {i}")
            if i in reorders:
                parents = [int(v) for v in g.integers(0, w.batch, size=w.batch)]
                M.mtla_beam_reorder(h, parents)
                states = O.reorder_states(states, parents)
        M.mtla_check(h)
        assert M.mtla_seq_positions(h) == [st.tokens for st in states]
        for b in range(w.batch):
            H.assert_cache_close(M.mtla_cache_export_seq(h, b), O.cache_array(states[b]), w.dtype)
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("seed", range(32))
def test_random_long_contexts_on_the_tensor_core_attention(seed):
    """Imported contexts of up to 6000 tokens (ragged on paged handles), batches up to 24: tile
    lists whose shares cut sequences at arbitrary places, sequences spread over many CTAs, CTAs
    holding many short sequences.  Sampled sequences are followed by the oracle."""
    g = np.random.Generator(np.random.Philox(key=[seed, 0xa77e]))
    pick = lambda xs: xs[int(g.integers(len(xs)))]
    batch = int(g.integers(1, 25))
    w = synth.Workload(
        name=f"fuzz_ctx{seed}", dtype="bf16", batch=batch, d_model=8 * int(g.integers(8, 33)),
        n_heads=int(g.integers(1, 33)), head_dim=pick([64, 128]), latent_rank=pick([128, 256, 384, 512]),
        rope_dim=pick([32, 64]), hyper_dim=int(g.integers(1, 65)), stride=int(g.integers(1, 5)),
        prefill_tokens=0, context_tokens=0, decode_steps=3, seed=2000 + seed)
    paged = bool(g.integers(2))
    longest = int(g.integers(1, 6001))
    lengths = [int(g.integers(1, longest + 1)) for _ in range(batch)] if paged else [longest] * batch
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    cfg = M.make_config(**H.dims_of(w), max_batch=batch, max_tokens=max(lengths) + w.decode_steps,
                        max_prefill_tokens=0, dtype="bf16", ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    dev = {k: v.cuda() for k, v in weights.items()}
    h = M.mtla_create_paged(cfg, dev) if paged else M.mtla_create(cfg, dev)
    sampled = sorted({0, batch // 2, batch - 1})
    try:
        assert M.mtla_attention_variant(h) == "tcgen05"
        rows = [synth.context_cache_row(w, b, -(-t // w.stride)) for b, t in enumerate(lengths)]
        if paged:
            for b, t in enumerate(lengths):
                M.mtla_cache_import_seqs(h, b, rows[b][None].cuda(), t)
        else:
            M.mtla_cache_import(h, torch.stack(rows).cuda(), longest)
        states = {b: O.state_from_cache(rows[b].double().numpy(), lengths[b], p) for b in sampled}
        for i in range(w.decode_steps):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (batch, w.d_model)), "bf16")
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in sampled])
            assert_close_scaled(y[sampled], want, "bf16", f"step {i}")
        M.mtla_check(h)
        assert M.mtla_seq_positions(h) == [t + w.decode_steps for t in lengths]
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("seed", range(16))
def test_random_comparison_layers(seed):
    """MHA / GQA / MQA layers of random width and grouping with an imported context."""
    from oracle import gqa_oracle as G
    g = np.random.Generator(np.random.Philox(key=[seed, 0x69a]))
    pick = lambda xs: xs[int(g.integers(len(xs)))]
    n_kv = pick([1, 2, 3, 4, 8])
    per = pick([1, 2, 4, 5, 8, 32]) if n_kv <= 2 else pick([1, 2, 4])
    batch, ctx = int(g.integers(1, 9)), int(g.integers(1, 1500))
    w = synth.Workload(
        name=f"fuzz_kv{seed}", dtype="bf16", batch=batch, d_model=8 * int(g.integers(8, 49)),
        n_heads=n_kv * per, head_dim=pick([64, 128]), latent_rank=128, rope_dim=32, hyper_dim=8, stride=1,
        prefill_tokens=0, context_tokens=0, decode_steps=4, seed=3000 + seed)
    weights = synth.make_baseline_weights(w, n_kv)
    p = G.params_from_tensors(
        dict(d_model=w.d_model, n_heads=w.n_heads, n_groups=n_kv, head_dim=w.head_dim),
        {k: v.double().numpy() for k, v in weights.items()}, rope_theta=w.rope_theta)
    h = M.mtla_baseline_create(d_model=w.d_model, n_heads=w.n_heads, n_kv_heads=n_kv, head_dim=w.head_dim,
                               max_batch=batch, max_tokens=ctx + w.decode_steps,
                               weights={k: v.cuda() for k, v in weights.items()}, rope_theta=w.rope_theta)
    try:
        cache = torch.stack([torch.stack([synth.kv_cache_plane(w, b, k, ctx) for k in range(n_kv)])
                             for b in range(batch)])
        M.mtla_cache_import(h, cache.cuda(), ctx)
        states = [G.state_from_cache(cache[b].double().numpy()) for b in range(batch)]
        for i in range(w.decode_steps):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (batch, w.d_model)), "bf16")
            y = M.mtla_decode_step(h, x.cuda())
            want = np.stack([G.decode_step(p, states[b], x[b].double().numpy()) for b in range(batch)])
            assert_close_scaled(y, want, "bf16", f"step {i}")
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)


@pytest.mark.parametrize("seed", range(10))
def test_random_large_batches(seed):
    """Batches of 100-400 sequences (more sequences than CTAs, several activation tiles in the
    projections) with short ragged contexts; the step is taken through the device, the static
    scratch and the host entry points in turn."""
    g = np.random.Generator(np.random.Philox(key=[seed, 0xb16]))
    pick = lambda xs: xs[int(g.integers(len(xs)))]
    batch = int(g.integers(100, 401))
    w = synth.Workload(
        name=f"fuzz_big{seed}", dtype="bf16", batch=batch, d_model=8 * int(g.integers(8, 25)),
        n_heads=int(g.integers(1, 17)), head_dim=64, latent_rank=pick([128, 256]), rope_dim=pick([32, 64]),
        hyper_dim=int(g.integers(1, 33)), stride=int(g.integers(1, 4)),
        prefill_tokens=0, context_tokens=0, decode_steps=3, seed=4000 + seed)
    paged = bool(g.integers(2))
    longest = int(g.integers(1, 201))
    lengths = [int(g.integers(1, longest + 1)) for _ in range(batch)] if paged else [longest] * batch
    weights = synth.make_weights(w)
    p = H.oracle_params(w, weights)
    cfg = M.make_config(**H.dims_of(w), max_batch=batch, max_tokens=max(lengths) + w.decode_steps,
                        max_prefill_tokens=0, dtype="bf16", ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    dev = {k: v.cuda() for k, v in weights.items()}
    h = M.mtla_create_paged(cfg, dev) if paged else M.mtla_create(cfg, dev)
    sampled = sorted({0, 1, batch // 3, batch // 2, batch - 2, batch - 1})
    try:
        rows = [synth.context_cache_row(w, b, -(-t // w.stride)) for b, t in enumerate(lengths)]
        if paged:
            for b, t in enumerate(lengths):
                M.mtla_cache_import_seqs(h, b, rows[b][None].cuda(), t)
        else:
            M.mtla_cache_import(h, torch.stack(rows).cuda(), longest)
        states = {b: O.state_from_cache(rows[b].double().numpy(), lengths[b], p) for b in sampled}
        for i in range(w.decode_steps):
            x = synth.stored(synth.normal(w.seed, f"x/{i}", (batch, w.d_model)), "bf16")
            if i == 0:
                y = M.mtla_decode_step(h, x.cuda())
            elif i == 1:
                try:
                    y = M.mtla_decode_step_static(h, x.cuda())
                except M.MTLAError as err:            # the workspace of a large batch may not fit
                    assert err.status == -9
                    y = M.mtla_decode_step(h, x.cuda())
            else:
                yh = torch.empty(batch, w.d_model, dtype=torch.bfloat16).pin_memory()
                M.mtla_decode_step_host(h, x.pin_memory(), yh)
                torch.cuda.synchronize()
                y = yh
            want = np.stack([O.decode_step(p, states[b], x[b].double().numpy()) for b in sampled])
            assert_close_scaled(y[sampled], want, "bf16", f"step {i}")
        M.mtla_check(h)
    finally:
        M.mtla_destroy(h)
