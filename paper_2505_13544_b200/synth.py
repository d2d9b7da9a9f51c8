"""Seeded synthetic workloads: shapes and random tensors only.

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests/benchmarks.  It holds no MTLA arithmetic: it names the five
benchmark configurations, draws normal random tensors from a counter-based
generator (numpy's Philox, keyed by seed and tensor name, so any tensor can be
regenerated on its own) and rounds them to the configuration's storage type so
that both sides start from identical bits.

The paper evaluates on speech/text corpora; only the tensor shapes matter to
the decode/prefill path, so unit-normal activations and fan-in-scaled weights
of the paper's model shape (Section 5.2: d 512, 8 heads, r 256, RoPE dim 32,
hyper-network width 64, s 2..4) stand in for them.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str            # "fp32" | "bf16": storage type of weights, activations, cache
    batch: int
    d_model: int
    n_heads: int
    head_dim: int
    latent_rank: int      # r
    rope_dim: int         # d_h^R
    hyper_dim: int        # d_w
    stride: int           # s
    prefill_tokens: int   # prompt length run through the parallel prefill (0: none)
    context_tokens: int   # tokens represented by an imported cache (0: none)
    decode_steps: int
    seed: int
    ln_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def slot_width(self) -> int:
        return self.latent_rank + self.rope_dim

    @property
    def max_tokens(self) -> int:
        return self.prefill_tokens + self.context_tokens + self.decode_steps

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def _paper_layer(**kw) -> dict:
    base = dict(dtype="bf16", d_model=512, n_heads=8, head_dim=64, latent_rank=256,
                rope_dim=32, hyper_dim=64, context_tokens=0)
    base.update(kw)
    return base


WORKLOADS: dict[str, Workload] = {
    "tiny": Workload(name="tiny", dtype="fp32", batch=1, d_model=256, n_heads=4, head_dim=64,
                     latent_rank=64, rope_dim=32, hyper_dim=16, stride=2, prefill_tokens=128,
                     context_tokens=0, decode_steps=128, seed=0),
    "paper": Workload(name="paper", **_paper_layer(batch=32, stride=2, prefill_tokens=1024,
                                                  decode_steps=1024, seed=1)),
    **{f"sweep_s{s}": Workload(name=f"sweep_s{s}",
                               **_paper_layer(batch=64, stride=s, prefill_tokens=4096,
                                              decode_steps=256, seed=2))
       for s in (1, 2, 3, 4)},
    "longctx": Workload(name="longctx", dtype="bf16", batch=8, d_model=1024, n_heads=16,
                        head_dim=64, latent_rank=512, rope_dim=64, hyper_dim=128, stride=4,
                        prefill_tokens=16384, context_tokens=0, decode_steps=64, seed=3),
    "large": Workload(name="large", dtype="bf16", batch=128, d_model=4096, n_heads=32,
                      head_dim=128, latent_rank=512, rope_dim=64, hyper_dim=128, stride=2,
                      prefill_tokens=0, context_tokens=32768, decode_steps=128, seed=4),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def _generator(seed: int, name: str) -> np.random.Generator:
    key = (int(seed) << 32) | zlib.crc32(name.encode())
    return np.random.Generator(np.random.Philox(key=key))


def normal(seed: int, name: str, shape, scale: float = 1.0, shift: float = 0.0) -> np.ndarray:
    """float32 array of shift + scale * N(0, 1), reproducible from (seed, name)."""
    out = _generator(seed, name).standard_normal(size=shape, dtype=np.float32)
    if scale != 1.0:
        out *= np.float32(scale)
    if shift != 0.0:
        out += np.float32(shift)
    return out


def stored(a: np.ndarray, dtype: str) -> torch.Tensor:
    """Round to the storage type; the returned CPU tensor is what both sides consume."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(torch_dtype(dtype))


def make_weights(w: Workload, prefix: str = "") -> dict[str, torch.Tensor]:
    """All layer parameters, row-major [in][out], already rounded to w.dtype.

    Weight matrices are N(0,1)/sqrt(fan_in); LayerNorm gain 1 + 0.1 N(0,1), its bias and
    the hyper-network biases 0.1 N(0,1).  `prefix` names the layer inside a stack.
    """
    d, nh, dh, r, dr, dw = (w.d_model, w.n_heads, w.head_dim, w.latent_rank, w.rope_dim,
                            w.hyper_dim)

    def mat(name, fan_in, fan_out):
        return stored(normal(w.seed, prefix + name, (fan_in, fan_out), scale=fan_in ** -0.5), w.dtype)

    def vec(name, n, scale, shift=0.0):
        return stored(normal(w.seed, prefix + name, (n,), scale=scale, shift=shift), w.dtype)

    return {
        "w_q": mat("w_q", d, nh * dh),
        "w_qr": mat("w_qr", d, nh * dr),
        "w_r": mat("w_r", d, r),
        "w_kr": mat("w_kr", d, dr),
        "ln_gamma": vec("ln_gamma", r, 0.1, 1.0),
        "ln_beta": vec("ln_beta", r, 0.1),
        "w_k": mat("w_k", r, nh * dh),
        "w_v": mat("w_v", r, nh * dh),
        "w_o": mat("w_o", nh * dh, d),
        "hyp_c_w": mat("hyp_c_w", r, dw),
        "hyp_c_b": vec("hyp_c_b", dw, 0.1),
        "hyp_pe_w": mat("hyp_pe_w", r, dw),
        "hyp_pe_b": vec("hyp_pe_b", dw, 0.1),
    }


@dataclass(frozen=True)
class StackWorkload:
    """The paper's decoder (Section 5.2, appendix on hyper-parameters): n_layers layers of MTLA
    self-attention + feed-forward block of width d_ff, the encoder output being the first
    prompt_tokens rows of the input sequence."""
    name: str
    layer: Workload       # attention dims, dtype, batch, prompt length (prefill_tokens), steps, seed
    n_layers: int
    d_ff: int


STACK_WORKLOADS: dict[str, StackWorkload] = {
    # 9 layers, d 512, feed-forward 2048, 8 heads, r 256, d_R 32, s 2; a 512-frame prompt.
    "decoder_paper": StackWorkload("decoder_paper", WORKLOADS["paper"].scaled(
        name="decoder_paper", prefill_tokens=512, decode_steps=256), n_layers=9, d_ff=2048),
}


def make_stack_weights(sw: StackWorkload) -> dict:
    """Parameters of every layer of the stack plus the final LayerNorm, rounded to the storage
    type: {"layers": [{attention weights..., ln1_gamma, ln1_beta, ln2_gamma, ln2_beta, w1, b1,
    w2, b2}], "lnf_gamma", "lnf_beta"}.  Matrices N(0,1)/sqrt(fan_in), row-major [in][out];
    LayerNorm gains 1 + 0.1 N(0,1); biases 0.1 N(0,1)."""
    w = sw.layer
    d = w.d_model

    def vec(name, n, shift=0.0):
        return stored(normal(w.seed, name, (n,), scale=0.1, shift=shift), w.dtype)

    layers = []
    for n in range(sw.n_layers):
        pre = f"layer{n}/"
        lw = make_weights(w, prefix=pre)
        lw.update({
            "ln1_gamma": vec(pre + "ln1_gamma", d, 1.0), "ln1_beta": vec(pre + "ln1_beta", d),
            "ln2_gamma": vec(pre + "ln2_gamma", d, 1.0), "ln2_beta": vec(pre + "ln2_beta", d),
            "w1": stored(normal(w.seed, pre + "w1", (d, sw.d_ff), scale=d ** -0.5), w.dtype),
            "b1": vec(pre + "b1", sw.d_ff),
            "w2": stored(normal(w.seed, pre + "w2", (sw.d_ff, d), scale=sw.d_ff ** -0.5), w.dtype),
            "b2": vec(pre + "b2", d),
        })
        layers.append(lw)
    return {"layers": layers, "lnf_gamma": vec("lnf_gamma", d, 1.0), "lnf_beta": vec("lnf_beta", d)}


def make_baseline_weights(w: Workload, n_kv_heads: int) -> dict[str, torch.Tensor]:
    """Parameters of a comparison layer (MHA / GQA / MQA) of w's width: N(0,1)/sqrt(fan_in),
    row-major [in][out], rounded to w.dtype."""
    d, nh, dh = w.d_model, w.n_heads, w.head_dim

    def mat(name, fan_in, fan_out):
        return stored(normal(w.seed, f"baseline/{n_kv_heads}/{name}", (fan_in, fan_out),
                             scale=fan_in ** -0.5), w.dtype)

    return {"w_q": mat("w_q", d, nh * dh), "w_k": mat("w_k", d, n_kv_heads * dh),
            "w_v": mat("w_v", d, n_kv_heads * dh), "w_o": mat("w_o", nh * dh, d)}


def kv_cache_plane(w: Workload, seq: int, kv_head: int, tokens: int) -> torch.Tensor:
    """A stand-in key-value cache [tokens][2 d_h] (value then key, unit normal) for one
    (sequence, key/value head) of a comparison layer, where the context is too long to decode."""
    return stored(normal(w.seed, f"kv/{seq}/{kv_head}", (tokens, 2 * w.head_dim)), w.dtype)


def prompt(w: Workload, batch: int | None = None, tokens: int | None = None) -> torch.Tensor:
    """Prompt activations [B][T][d] ~ N(0,1), generated one sequence at a time."""
    b = w.batch if batch is None else batch
    t = w.prefill_tokens if tokens is None else tokens
    rows = [stored(normal(w.seed, f"prompt/{i}", (t, w.d_model)), w.dtype) for i in range(b)]
    return torch.stack(rows) if rows else torch.empty(0, t, w.d_model, dtype=torch_dtype(w.dtype))


def decode_input(w: Workload, step: int, batch: int | None = None) -> torch.Tensor:
    """Activations [B][d] ~ N(0,1) for decode step `step` (0-based)."""
    b = w.batch if batch is None else batch
    return stored(normal(w.seed, f"decode/{step}", (w.batch, w.d_model))[:b], w.dtype)


def context_cache_row(w: Workload, seq: int, n_slots: int | None = None) -> torch.Tensor:
    """A stand-in compressed cache [n_slots][r + d_R] for sequence `seq`.

    Each latent slot is distributed like a stride-s merge of unit-normal latents with
    independent sigmoid(N(0,1)) weights: given the weights a_k the sum of a_k * z_k is
    N(0, sum a_k^2), so one normal per element is scaled by sqrt(sum_k a_k^2) per slot.
    RoPE keys are unit normal.  Used where the context is too long to prefill
    (the "large" workload), and imported through mtla_cache_import.
    """
    n = -(-w.context_tokens // w.stride) if n_slots is None else n_slots
    gate_logits = normal(w.seed, f"ctx_gate/{seq}", (n, w.stride))
    gains = np.sqrt(((1.0 / (1.0 + np.exp(-gate_logits))) ** 2).sum(axis=1, keepdims=True))
    row = normal(w.seed, f"ctx/{seq}", (n, w.slot_width))
    row[:, : w.latent_rank] *= gains.astype(np.float32)
    return stored(row, w.dtype)


@dataclass(frozen=True)
class BeamWorkload:
    """Beam-search decoding over utterances of different lengths: n_utt utterances with `beam`
    hypotheses each (batch index = utterance * beam + rank), contexts of min_context ..
    max_context tokens, a re-parenting after every decode step."""
    name: str
    layer: Workload       # dims, dtype, seed; its batch / context fields are not used
    n_utt: int
    beam: int
    min_context: int
    max_context: int
    decode_steps: int

    @property
    def n_seq(self) -> int:
        return self.n_utt * self.beam

    def contexts(self) -> list[int]:
        return ragged_lengths(self.layer.seed, self.n_utt, self.min_context, self.max_context)


def _beam_workloads() -> dict:
    # The paper decodes with beam sizes 10 to 50 on its d 512 models; the second entry is the
    # beam-search counterpart of the "large" decode workload (16 x 8 = its 128 sequences).
    return {
        "beam_paper": BeamWorkload("beam_paper", WORKLOADS["paper"], n_utt=24, beam=10,
                                   min_context=64, max_context=1024, decode_steps=64),
        "beam_large": BeamWorkload("beam_large", WORKLOADS["large"], n_utt=16, beam=8,
                                   min_context=8192, max_context=32768, decode_steps=72),
    }


def ragged_lengths(seed: int, n: int, lo: int, hi: int) -> list[int]:
    """n prompt lengths drawn uniformly from [lo, hi], a stand-in for utterances of
    different durations (the paper's test sets are variable-length speech and text)."""
    return [int(v) for v in _generator(seed, "ragged_lengths").integers(lo, hi + 1, size=n)]


def beam_parents(seed: int, step: int, n_utt: int, beam: int) -> list[int]:
    """Parent indices of one beam-search step for n_utt utterances with `beam` hypotheses
    each (batch index = utterance * beam + rank).  Every surviving hypothesis continues one of
    its own utterance's hypotheses; better-ranked parents are chosen more often (rank k with
    weight 1 / (k + 1)), as in a real search where most survivors extend the top entries."""
    g = _generator(seed, f"beam_parents/{step}")
    weights = 1.0 / (1.0 + np.arange(beam))
    weights /= weights.sum()
    out = []
    for u in range(n_utt):
        picks = np.sort(g.choice(beam, size=beam, p=weights))
        out += [u * beam + int(k) for k in picks]
    return out


BEAM_WORKLOADS: dict[str, BeamWorkload] = _beam_workloads()
