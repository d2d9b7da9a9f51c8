"""CPU oracle for the paper's decoder: layers of MTLA self-attention plus a feed-forward block,
stacked.  TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU leg may
import it, the product path never does.  Plain fp64 numpy; the attention itself is the MTLA oracle
(mtla_oracle.py), this file adds only what Section 5.2 and the appendix on hyper-parameters put
around it: a Transformer decoder without cross-attention (the encoder output is simply the first
part of the input sequence), 9 layers, model width 512, feed-forward width 2048, 8 heads.

One layer, for the token vector x [d] (pre-norm residual form):

    h = x + MTLA(LayerNorm_1(x))                      self-attention sub-layer, Section 4
    y = h + W_2 act(W_1 LayerNorm_2(h) + b_1) + b_2   feed-forward sub-layer

and the stack applies the layers in order and a final LayerNorm to the last one's output.

Readings of points the paper leaves open (free conventions, shared with the CUDA path):
  * pre-norm placement (LayerNorm in front of each sub-layer and one after the last layer) and
    ReLU as the feed-forward activation: the paper builds on the Fairseq speech-translation
    example and states neither; these are that family's usual settings;
  * LayerNorm: affine, biased variance, eps 1e-5 inside the square root;
  * both feed-forward matrices carry a bias; no dropout at inference;
  * the prompt (encoder output) is just the first rows of the input: the stack sees one sequence.

Two evaluation orders are written out so they can be checked against each other:
  * token by token: each token goes through all layers before the next token starts
    (what incremental decoding does);
  * layer by layer: one layer consumes the whole sequence before the next layer starts
    (what a parallel prefill does).
They agree because every layer is causal.

Parity pins (tests/test_decoder_oracle_pins.py): the feed-forward sub-layer and the LayerNorms
against torch.nn modules; the attention sub-layer against the MTLA oracle called directly; the
two evaluation orders against each other; closed forms (zero feed-forward output matrix, zero
attention output matrix); a two-layer stack against the explicit composition; planted mistakes.
Parity unpinned (the paper does not fix them): pre- versus post-norm, the activation, the final
LayerNorm, bias presence.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from oracle import mtla_oracle as O


@dataclass
class LayerParams:
    attn: O.Params            # the MTLA self-attention of this layer
    ln1_gamma: np.ndarray     # [d]
    ln1_beta: np.ndarray      # [d]
    ln2_gamma: np.ndarray     # [d]
    ln2_beta: np.ndarray      # [d]
    w1: np.ndarray            # [d][d_ff]
    b1: np.ndarray            # [d_ff]
    w2: np.ndarray            # [d_ff][d]
    b2: np.ndarray            # [d]
    ln_eps: float = 1e-5


@dataclass
class StackParams:
    layers: list              # LayerParams, first layer first
    lnf_gamma: np.ndarray     # [d] final LayerNorm
    lnf_beta: np.ndarray      # [d]
    ln_eps: float = 1e-5


@dataclass
class StackState:
    """Decoding state of one sequence: one MTLA cache per layer."""
    layers: list = field(default_factory=list)     # O.State per layer

    @classmethod
    def empty(cls, n_layers: int) -> "StackState":
        return cls(layers=[O.State() for _ in range(n_layers)])

    @property
    def tokens(self) -> int:
        return self.layers[0].tokens if self.layers else 0


def layer_norm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * gamma + beta


def feed_forward(lp: LayerParams, v: np.ndarray) -> np.ndarray:
    """W_2 relu(W_1 v + b_1) + b_2 for v [..., d]."""
    return np.maximum(v @ lp.w1 + lp.b1, 0.0) @ lp.w2 + lp.b2


def layer_decode_step(lp: LayerParams, st: O.State, x: np.ndarray) -> np.ndarray:
    """One token through one layer; st is that layer's MTLA cache (updated)."""
    x = np.asarray(x, dtype=np.float64)
    h = x + O.decode_step(lp.attn, st, layer_norm(x, lp.ln1_gamma, lp.ln1_beta, lp.ln_eps))
    return h + feed_forward(lp, layer_norm(h, lp.ln2_gamma, lp.ln2_beta, lp.ln_eps))


def stack_decode_step(sp: StackParams, st: StackState, x: np.ndarray) -> np.ndarray:
    """One token through all layers and the final LayerNorm (token-by-token order)."""
    h = np.asarray(x, dtype=np.float64)
    for lp, layer_state in zip(sp.layers, st.layers):
        h = layer_decode_step(lp, layer_state, h)
    return layer_norm(h, sp.lnf_gamma, sp.lnf_beta, sp.ln_eps)


def stack_decode_sequence(sp: StackParams, xs: np.ndarray, st: StackState | None = None):
    """Token-by-token order over xs [T][d]; returns (Y [T][d], state)."""
    st = StackState.empty(len(sp.layers)) if st is None else st
    ys = [stack_decode_step(sp, st, x) for x in np.asarray(xs, dtype=np.float64)]
    return (np.stack(ys) if ys else np.zeros((0, len(sp.lnf_gamma)))), st


def stack_forward_by_layers(sp: StackParams, xs: np.ndarray, st: StackState | None = None,
                            rows=None):
    """Layer-by-layer order over a whole sequence xs [T][d]: each layer consumes every token
    before the next layer starts.  Returns (Y, state); Y holds all rows, or only `rows` of the
    LAST layer (earlier layers always produce every row, the next layer needs them)."""
    st = StackState.empty(len(sp.layers)) if st is None else st
    h = np.asarray(xs, dtype=np.float64)
    last = len(sp.layers) - 1
    for n, (lp, layer_state) in enumerate(zip(sp.layers, st.layers)):
        u = layer_norm(h, lp.ln1_gamma, lp.ln1_beta, lp.ln_eps)
        want = rows if (n == last and rows is not None) else None
        a, _ = O.decode_sequence(lp.attn, u, layer_state, rows=want)
        if want is not None:
            h = h[list(want)]
        h = h + a
        h = h + feed_forward(lp, layer_norm(h, lp.ln2_gamma, lp.ln2_beta, lp.ln_eps))
    return layer_norm(h, sp.lnf_gamma, sp.lnf_beta, sp.ln_eps), st


def stack_cache_elements(sp: StackParams, tokens: int, batch: int = 1) -> int:
    """Cache elements held by the stack: every layer keeps ceil(T/s) slots of r + d_R (the
    paper's per-layer count times the number of layers l, Section 4.3)."""
    return sum(O.cache_elements(tokens, lp.attn, batch) for lp in sp.layers)
