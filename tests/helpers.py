"""Shared test plumbing: build an oracle Params and a GPU handle from the same seeded tensors."""
from __future__ import annotations

import numpy as np
import torch

from oracle import mtla_oracle as O
from paper_2505_13544_b200 import synth

# Tolerances of the benchmark specification: fp32 max-abs 1e-4; bf16 max-abs 2e-2 and
# relative L2 1e-2.  Slot counts and cache lengths must match exactly.
FP32_MAX_ABS = 1e-4
BF16_MAX_ABS = 2e-2
BF16_REL_L2 = 1e-2


def dims_of(w: synth.Workload) -> dict:
    return dict(d_model=w.d_model, n_heads=w.n_heads, head_dim=w.head_dim,
                latent_rank=w.latent_rank, rope_dim=w.rope_dim, hyper_dim=w.hyper_dim,
                stride=w.stride)


def oracle_params(w: synth.Workload, weights: dict) -> O.Params:
    return O.params_from_tensors(dims_of(w), {k: v.double().numpy() for k, v in weights.items()},
                                 ln_eps=w.ln_eps, rope_theta=w.rope_theta)


def gpu_handle(w: synth.Workload, weights: dict, max_batch=None, max_tokens=None,
               max_prefill_tokens=None, device="cuda:0", kernel_path=0):
    from paper_2505_13544_b200 import binding as M
    cfg = M.make_config(**dims_of(w), max_batch=max_batch or w.batch,
                        max_tokens=max_tokens or w.max_tokens,
                        max_prefill_tokens=(w.prefill_tokens if max_prefill_tokens is None
                                            else max_prefill_tokens),
                        dtype=w.dtype, ln_eps=w.ln_eps, rope_theta=w.rope_theta,
                        kernel_path=kernel_path)
    dev_weights = {k: v.to(device) for k, v in weights.items()}
    return M.mtla_create(cfg, dev_weights, device=device)


def assert_close(got: torch.Tensor, want: np.ndarray, dtype: str, what: str = "y") -> None:
    """Applies the specification's tolerance for the storage type."""
    g = got.detach().double().cpu().numpy()
    want = np.asarray(want, dtype=np.float64)
    assert g.shape == want.shape, (what, g.shape, want.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite values"
    err = np.abs(g - want).max() if g.size else 0.0
    if dtype == "fp32":
        assert err <= FP32_MAX_ABS, f"{what}: max abs err {err:.3e} > {FP32_MAX_ABS}"
    else:
        rel = np.linalg.norm(g - want) / max(np.linalg.norm(want), 1e-30)
        assert err <= BF16_MAX_ABS, f"{what}: max abs err {err:.3e} > {BF16_MAX_ABS}"
        assert rel <= BF16_REL_L2, f"{what}: rel L2 err {rel:.3e} > {BF16_REL_L2}"


def assert_close_stack(got: torch.Tensor, want: np.ndarray, dtype: str, n_layers: int,
                       what: str = "y") -> None:
    """Outputs of an n_layers-deep stack.  The specification's bf16 bound (max-abs 2e-2) is the
    error budget of ONE attention layer's output; in a stack each layer's attention adds an
    error of that size to the fp32 residual stream (on top of the bf16 rounding of the
    sub-layer inputs and outputs, 2^-9 relative each), the errors of different layers are
    independent and add in quadrature, and the final LayerNorm rescales the stream to unit
    size: max-abs <= 2e-2 * sqrt(n_layers).  The relative-L2 bound stays 1e-2; fp32 stays 1e-4
    per layer, i.e. 1e-4 * sqrt(n_layers)."""
    g = got.detach().double().cpu().numpy()
    want = np.asarray(want, dtype=np.float64)
    assert g.shape == want.shape, (what, g.shape, want.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite values"
    err = np.abs(g - want).max() if g.size else 0.0
    scale = max(1.0, float(n_layers)) ** 0.5
    if dtype == "fp32":
        assert err <= FP32_MAX_ABS * scale, f"{what}: max abs err {err:.3e} > {FP32_MAX_ABS * scale:.1e}"
    else:
        rel = np.linalg.norm(g - want) / max(np.linalg.norm(want), 1e-30)
        assert err <= BF16_MAX_ABS * scale, f"{what}: max abs err {err:.3e} > {BF16_MAX_ABS * scale:.1e}"
        assert rel <= BF16_REL_L2, f"{what}: rel L2 err {rel:.3e} > {BF16_REL_L2}"
    print(f"[stack parity] {what}: layers {n_layers} max abs {err:.3e} "
          f"rel L2 {np.linalg.norm(g - want) / max(np.linalg.norm(want), 1e-30):.3e} max |y| {np.abs(want).max():.2f}")


def assert_cache_close(got: torch.Tensor, want: np.ndarray, dtype: str, scale: float = 1.0) -> None:
    """Cache contents: fp32 to 1e-4; bf16 to a few storage ulps (2^-7 relative, 2^-7 absolute).
    `scale` widens both for the deeper layers of a stack, whose inputs already carry the
    accumulated error of the layers below (see assert_close_stack)."""
    g = got.detach().double().cpu().numpy()
    want = np.asarray(want, dtype=np.float64)
    assert g.shape == want.shape, (g.shape, want.shape)
    if dtype == "fp32":
        assert np.abs(g - want).max() <= FP32_MAX_ABS * scale
    else:
        ratio = float((np.abs(g - want) / (2.0 ** -7 * (1.0 + np.abs(want)))).max())
        assert ratio <= scale, f"cache rows: worst error {ratio:.2f} x the bf16 bound (allowed {scale:.2f})"


ATTN_WEIGHT_NAMES = ("w_q", "w_qr", "w_r", "w_kr", "ln_gamma", "ln_beta", "w_k", "w_v", "w_o",
                     "hyp_c_w", "hyp_c_b", "hyp_pe_w", "hyp_pe_b")
LAYER_EXTRA_NAMES = ("ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta", "w1", "b1", "w2", "b2")


def oracle_stack_params(sw: synth.StackWorkload, weights: dict):
    """The decoder oracle's parameters from a stack's stored weights."""
    from oracle import decoder_oracle as D
    w = sw.layer
    layers = []
    for lw in weights["layers"]:
        f = {k: v.double().numpy() for k, v in lw.items()}
        attn = O.params_from_tensors(dims_of(w), {k: f[k] for k in ATTN_WEIGHT_NAMES},
                                     ln_eps=w.ln_eps, rope_theta=w.rope_theta)
        layers.append(D.LayerParams(attn=attn, **{k: f[k] for k in LAYER_EXTRA_NAMES}))
    return D.StackParams(layers=layers, lnf_gamma=weights["lnf_gamma"].double().numpy(),
                         lnf_beta=weights["lnf_beta"].double().numpy())


def gpu_stack(sw: synth.StackWorkload, weights: dict, max_batch=None, max_tokens=None,
              max_prefill_tokens=None, device="cuda:0"):
    from paper_2505_13544_b200 import binding as M
    w = sw.layer
    cfg = M.make_config(**dims_of(w), max_batch=max_batch or w.batch,
                        max_tokens=max_tokens or w.max_tokens,
                        max_prefill_tokens=(w.prefill_tokens if max_prefill_tokens is None
                                            else max_prefill_tokens),
                        dtype=w.dtype, ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    dev = {"layers": [{k: v.to(device) for k, v in lw.items()} for lw in weights["layers"]],
           "lnf_gamma": weights["lnf_gamma"].to(device), "lnf_beta": weights["lnf_beta"].to(device)}
    return M.mtla_stack_create(cfg, sw.n_layers, sw.d_ff, dev, device=device)
