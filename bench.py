#!/usr/bin/env python
"""Benchmark of the MTLA decode step (and, as extras, the prefill) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one full decode step (input projections, LayerNorm + gate + slot update,
query absorption, attention over the compressed cache, output projections) for the whole
batch; the metric is decode tokens/s = B * K / time.  With N > 1 every rank runs an
independent replica of the workload on its own GPU (sequences never interact, so there is
no collective on the data path) and the value is the sum over ranks divided by the
slowest rank's device time.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2505_13544_b200 import synth  # noqa: E402

METRIC = "mtla_decode_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0          # the "~8 TB/s" the benchmark specification quotes


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def code_hash(texts) -> str:
    """sha256 of source texts with comments and blank space removed."""
    out = ""
    for text in texts:
        for line in text.splitlines():
            code = line.split("//")[0].strip()
            if code:
                out += " ".join(code.split()) + "\n"
    return hashlib.sha256(out.encode()).hexdigest()


def kernel_code_hash() -> str:
    """Hash of the decode-attention kernel's code (comments and blank space removed), to tell
    whether the committed ncu counters still describe the kernel that is being timed."""
    csrc = os.path.join(ROOT, "paper_2505_13544_b200", "csrc")
    return code_hash(open(os.path.join(csrc, name)).read()
                     for name in ("decode_attn_tc.cuh", "sm100_ptx.cuh"))


def algorithmic_work(w: synth.Workload, n_slots: float) -> dict:
    """Bytes and FLOP one decode step must move/compute (weights once, cache once)."""
    e = 2 if w.dtype == "bf16" else 4
    d, nh, dh, r, dr, dw = (w.d_model, w.n_heads, w.head_dim, w.latent_rank, w.rope_dim,
                            w.hyper_dim)
    params = (d * nh * dh + d * nh * dr + d * r + d * dr + 2 * r + 2 * r * nh * dh
              + nh * dh * d + 2 * (r * dw + dw))
    cache = w.batch * n_slots * (r + dr) * e
    return {"weight_bytes": params * e, "cache_bytes": cache,
            "attn_flop": w.batch * nh * n_slots * (2 * (r + dr) + 2 * r),
            "proj_flop": 2 * w.batch * params}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.mem_samples, self.power_samples = [], []
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nvml = None

    def _run(self):
        n = self._nvml
        names = {
            "sw_power_cap": getattr(n, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(n, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(n, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(n, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "hw_power_brake": getattr(n, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM))
                self.mem_samples.append(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_MEM))
                self.power_samples.append(n.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
                try:
                    mask = n.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = n.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.002)

    def __enter__(self):
        if self._nvml is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self) -> dict:
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "samples": len(self.samples),
                "reasons": sorted(self.reasons),
                "mem_mhz": float(np.median(self.mem_samples)) if self.mem_samples else None,
                "power_w": float(np.median(self.power_samples)) if self.power_samples else None,
                "power_w_max": float(max(self.power_samples)) if self.power_samples else None}


def dims_of(w: synth.Workload) -> dict:
    return dict(d_model=w.d_model, n_heads=w.n_heads, head_dim=w.head_dim,
                latent_rank=w.latent_rank, rope_dim=w.rope_dim, hyper_dim=w.hyper_dim,
                stride=w.stride)


# --------------------------------------------------------------------------- CPU oracle legs

def oracle_decode_sample(w: synth.Workload, n_seq: int, budget_s: float, max_steps: int,
                         exact_steps: int | None = None) -> dict:
    """Times the CPU oracle's decode step, as it stands, on a bounded sample: n_seq sequences
    at the workload's full context, as many steps as fit the budget.  State building (the
    prompt or the imported cache) is outside the timed region, like the GPU's."""
    from oracle import mtla_oracle as O
    from threadpoolctl import threadpool_info

    weights = synth.make_weights(w)
    p = O.params_from_tensors(dims_of(w), {k: v.double().numpy() for k, v in weights.items()},
                              ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    states = []
    for b in range(n_seq):
        if w.context_tokens:
            cache = synth.context_cache_row(w, b).double().numpy()
            states.append(O.state_from_cache(cache, w.context_tokens, p))
        else:
            prompt = synth.normal(w.seed, f"prompt/{b}", (w.prefill_tokens, w.d_model))
            prompt = synth.stored(prompt, w.dtype).double().numpy()
            _, st = O.decode_sequence(p, prompt, rows=[])
            states.append(st)
    steps, t0 = 0, time.perf_counter()
    limit = exact_steps if exact_steps is not None else max_steps
    while steps < limit:
        x = synth.decode_input(w, steps, batch=n_seq).double().numpy()
        for b in range(n_seq):
            O.decode_step(p, states[b], x[b])
        steps += 1
        if exact_steps is None and time.perf_counter() - t0 >= budget_s:
            break
    elapsed = time.perf_counter() - t0
    cores = max([int(i.get("num_threads", 1)) for i in threadpool_info()] + [1])
    return {"value": n_seq * steps / elapsed, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n_seq} of {w.batch} sequences x {steps} decode steps at full context "
                      f"({states[0].n_slots} slots), {elapsed:.1f} s",
            "seconds": elapsed, "steps": steps}


def pick_workload(args) -> synth.Workload:
    """The named workload, optionally shrunk (the name then says how)."""
    w = synth.WORKLOADS[args.workload]
    if args.batch:
        w = w.scaled(batch=args.batch, name=f"{w.name}[batch={args.batch}]")
    if args.context_tokens and w.context_tokens:
        w = w.scaled(context_tokens=args.context_tokens,
                     name=f"{w.name}[context_tokens={args.context_tokens}]")
    return w


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = pick_workload(args)
    n_seq = 1 if w.batch * w.latent_rank >= 8192 else min(w.batch, 4)
    # warm-up steps are run and discarded, then exactly --steps sample steps are timed
    oracle_decode_sample(w, n_seq, 0.0, 0, exact_steps=min(args.warmup, 1))
    res = oracle_decode_sample(w, n_seq, 0.0, 0, exact_steps=args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": res["seconds"] / max(res["steps"], 1) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "batch": n_seq, "of_batch": w.batch,
                   "note": "CPU oracle on host cores; each step is one decode step of a bounded "
                           "sample of sequences at full context"},
        "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU arm

def build_layer(w: synth.Workload, extra_steps: int, device, paged: bool = False):
    from paper_2505_13544_b200 import binding as M
    weights = synth.make_weights(w)
    cfg = M.make_config(**dims_of(w), max_batch=w.batch,
                        max_tokens=w.prefill_tokens + w.context_tokens + extra_steps,
                        max_prefill_tokens=w.prefill_tokens, dtype=w.dtype, ln_eps=w.ln_eps,
                        rope_theta=w.rope_theta)
    dev_weights = {k: v.to(device) for k, v in weights.items()}
    h = (M.mtla_create_paged(cfg, dev_weights, device=device) if paged
         else M.mtla_create(cfg, dev_weights, device=device))
    return M, h


def run_beam(args, bw: synth.BeamWorkload, device, local: int) -> None:
    """Beam-search decoding on a paged handle: ragged contexts, one re-parenting per step.
    A step is mtla_decode_step for all hypotheses followed by mtla_beam_reorder."""
    from paper_2505_13544_b200 import binding as M
    w = bw.layer
    K, W = args.steps, max(args.warmup, 3)
    contexts = bw.contexts()
    e = 2 if w.dtype == "bf16" else 4
    weights = synth.make_weights(w)
    cfg = M.make_config(**dims_of(w), max_batch=bw.n_seq, max_tokens=max(contexts) + 2 * (K + W) + 32,
                        max_prefill_tokens=0, dtype=w.dtype, ln_eps=w.ln_eps, rope_theta=w.rope_theta)
    h = M.mtla_create_paged(cfg, {k: v.to(device) for k, v in weights.items()}, device=device)
    for u, t in enumerate(contexts):
        row = synth.context_cache_row(w, u, -(-t // w.stride))
        M.mtla_cache_import_seqs(h, u, row[None].to(device), t)
    M.mtla_beam_reorder(h, [u for u in range(bw.n_utt) for _ in range(bw.beam)])
    dt = synth.torch_dtype(w.dtype)
    xs = [synth.stored(synth.normal(w.seed, f"beam_x/{i}", (bw.n_seq, w.d_model)), w.dtype).to(device)
          for i in range(8)]
    y = torch.empty(bw.n_seq, w.d_model, dtype=dt, device=device)
    # int32 arrays, as a search loop would hold them: the binding passes them without a copy.
    parents = [np.asarray(synth.beam_parents(w.seed, i, bw.n_utt, bw.beam), dtype=np.int32)
               for i in range(64)]

    def logical_bytes():
        return sum(-(-t // w.stride) for t in M.mtla_seq_positions(h)) * w.slot_width * e

    def page_bytes():
        return M.mtla_pages_in_use(h) * M.PAGE_SLOTS * w.slot_width * e

    step = 0
    for _ in range(W):
        M.mtla_decode_step(h, xs[step % 8], y)
        M.mtla_beam_reorder(h, parents[step % 64])
        step += 1
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # Host time of a step (argument marshalling, page bookkeeping, launches), over a run short
    # enough that the stream's launch queue never fills and throttles the host to device speed.
    n_host = min(32, K)
    torch.cuda.synchronize(device)
    host0 = time.perf_counter()
    for _ in range(n_host):
        M.mtla_decode_step(h, xs[step % 8], y)
        M.mtla_beam_reorder(h, parents[step % 64])
        step += 1
    host_issue_s = (time.perf_counter() - host0) / n_host
    torch.cuda.synchronize(device)
    bytes0, launches0 = logical_bytes(), M.mtla_launch_count(h)
    M.mtla_profile_begin_attention(h, K)
    with ClockSampler(local) as clocks:
        torch.cuda.synchronize(device)
        ev0.record()
        for _ in range(K):
            M.mtla_decode_step(h, xs[step % 8], y)
            M.mtla_beam_reorder(h, parents[step % 64])
            step += 1
        ev1.record()
        torch.cuda.synchronize(device)
    ms = ev0.elapsed_time(ev1)
    attn_ms, attn_steps = M.mtla_profile_end(h)
    launches = M.mtla_launch_count(h) - launches0
    bytes1, distinct = logical_bytes(), page_bytes()
    M.mtla_check(h)
    assert torch.isfinite(y.float()).all()

    xh = [x.cpu().pin_memory() for x in xs]
    yh = torch.empty(bw.n_seq, w.d_model, dtype=dt).pin_memory()
    for _ in range(W):
        M.mtla_decode_step_host(h, xh[step % 8], yh)
        M.mtla_beam_reorder(h, parents[step % 64])
        step += 1
    torch.cuda.synchronize(device)
    ev0.record()
    for _ in range(K):
        M.mtla_decode_step_host(h, xh[step % 8], yh)
        M.mtla_beam_reorder(h, parents[step % 64])
        step += 1
    ev1.record()
    torch.cuda.synchronize(device)
    e2e_ms = ev0.elapsed_time(ev1)
    M.mtla_check(h)

    peaks = measured_peaks()
    cache_bytes = 0.5 * (bytes0 + bytes1)
    attn_s = attn_ms * 1e-3 / max(attn_steps, 1)
    achieved = cache_bytes / attn_s / 1e9
    line = {
        "metric": METRIC, "value": bw.n_seq * K / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K,
        "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": bw.name, "utterances": bw.n_utt, "beam": bw.beam, "batch": bw.n_seq,
                   "context_tokens": [min(contexts), max(contexts)], "d_model": w.d_model,
                   "n_heads": w.n_heads, "head_dim": w.head_dim, "latent_rank": w.latent_rank,
                   "rope_dim": w.rope_dim, "stride": w.stride, "storage": "paged, 64-slot pages",
                   "step": "decode step + beam re-parenting",
                   "l2": "logical cache read per step %.0f MB, distinct pages %.0f MB (L2 126 MB)"
                         % (cache_bytes / 1e6, distinct / 1e6),
                   "attention_variant": M.mtla_attention_variant(h)},
        "roofline": {"bound": "hbm", "kernel": "decode attention (a7), ragged paged",
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
                     "launch_ms": attn_s * 1e3, "traffic": None,
                     "note": "achieved counts every hypothesis' slots (logical bytes); beams of one "
                             "utterance share pages, so part of it is served by L2 and the fraction "
                             "can exceed 1"},
        "cache": {"logical_bytes": cache_bytes, "distinct_page_bytes": distinct},
        "e2e": {"value": bw.n_seq * K / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": bw.n_seq * w.d_model * e + 4 * bw.n_seq,
                "d2h_bytes_per_step": bw.n_seq * w.d_model * e},
        "host_issue_us_per_step": host_issue_s * 1e6,
        "gpu_launches": int(launches),
        "clocks": clocks.summary(),
    }
    M.mtla_destroy(h)
    del h
    torch.cuda.empty_cache()
    if not args.no_cpu_baseline:
        from oracle import mtla_oracle as O
        p = O.params_from_tensors(dims_of(w), {k: v.double().numpy() for k, v in weights.items()},
                                  ln_eps=w.ln_eps, rope_theta=w.rope_theta)
        t = contexts[0]
        row = synth.context_cache_row(w, 0, -(-t // w.stride)).double().numpy()
        states = O.reorder_states([O.state_from_cache(row, t, p)], [0] * bw.beam)
        n, t0 = 0, time.perf_counter()
        while n < 64 and time.perf_counter() - t0 < 12.0:
            x = xs[n % 8][: bw.beam].double().cpu().numpy()
            for k in range(bw.beam):
                O.decode_step(p, states[k], x[k])
            states = O.reorder_states(states, [q for q in parents[n % 64][: bw.beam]])
            n += 1
        el = time.perf_counter() - t0
        from threadpoolctl import threadpool_info
        cores = max([int(i.get("num_threads", 1)) for i in threadpool_info()] + [1])
        line["cpu_baseline"] = {"value": bw.beam * n / el, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"the {bw.beam} hypotheses of utterance 0 ({t} context tokens) x "
                                          f"{n} steps with re-parenting, {el:.1f} s"}
    print(json.dumps(line))


def fill_context(M, h, w: synth.Workload, device) -> dict:
    """Brings the cache to the workload's context: a timed parallel prefill, or an import."""
    info = {}
    if w.prefill_tokens:
        x = torch.empty(w.batch, w.prefill_tokens, w.d_model, dtype=synth.torch_dtype(w.dtype),
                        device=device)
        for b in range(w.batch):
            x[b].copy_(synth.stored(synth.normal(w.seed, f"prompt/{b}",
                                                 (w.prefill_tokens, w.d_model)), w.dtype))
        y = torch.empty_like(x)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = []
        for _ in range(3):                       # one warm-up run, then two timed ones
            M.mtla_reset(h)
            torch.cuda.synchronize(device)
            ev0.record()
            M.mtla_prefill(h, x, y)
            ev1.record()
            torch.cuda.synchronize(device)
            times.append(ev0.elapsed_time(ev1))
        ms = min(times[1:])
        info = {"prefill_tokens_per_s": w.batch * w.prefill_tokens / (ms * 1e-3),
                "prefill_ms": ms, "prefill_tokens": w.prefill_tokens, "timed_runs": 2,
                "first_run_ms": times[0]}
        del x, y
    elif w.context_tokens:
        n_slots = -(-w.context_tokens // w.stride)
        cache = torch.empty(w.batch, n_slots, w.slot_width, dtype=synth.torch_dtype(w.dtype),
                            device=device)
        for b in range(w.batch):
            cache[b].copy_(synth.context_cache_row(w, b))
        M.mtla_cache_import(h, cache, w.context_tokens)
        torch.cuda.synchronize(device)
        del cache
    torch.cuda.empty_cache()
    return info


def run_compare(args, device, local: int) -> None:
    """The paper's comparison (Tables 1 and 5 are ratios against MHA, MQA, GQA and MLA), restated
    on this GPU: the same layer width, batch and context for every method, decode steps timed
    the same way; cache bytes per token from the library's own accounting."""
    from paper_2505_13544_b200 import binding as M
    base = synth.WORKLOADS[args.workload]
    ctx = args.context_tokens or (8192 if base.name == "large" else 4096)
    K, W = args.steps, max(args.warmup, 3)
    dt = torch.bfloat16
    rows = []

    def time_steps(h, xs, y):
        for i in range(W):
            M.mtla_decode_step(h, xs[i % 8], y)
        torch.cuda.synchronize(device)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        M.mtla_profile_begin_attention(h, K)
        ev0.record()
        for i in range(K):
            M.mtla_decode_step(h, xs[i % 8], y)
        ev1.record()
        torch.cuda.synchronize(device)
        attn_ms, n = M.mtla_profile_end(h)
        M.mtla_check(h)
        assert torch.isfinite(y.float()).all()
        return ev0.elapsed_time(ev1) / K, attn_ms / max(n, 1)

    xs = [synth.decode_input(base, i).to(device) for i in range(8)]
    y = torch.empty(base.batch, base.d_model, dtype=dt, device=device)
    kv_variants = [("MHA", base.n_heads)] + [("GQA", g) for g in sorted({max(base.n_heads // 4, 2), 2},
                                                                          reverse=True)] + [("MQA", 1)]
    for name, n_kv in kv_variants:
        weights = synth.make_baseline_weights(base, n_kv)
        h = M.mtla_baseline_create(d_model=base.d_model, n_heads=base.n_heads, n_kv_heads=n_kv,
                                   head_dim=base.head_dim, max_batch=base.batch,
                                   max_tokens=ctx + 2 * (K + W), device=device,
                                   weights={k: v.to(device) for k, v in weights.items()})
        # Four distinct seeded sequences, tiled over the batch (the values do not affect timing).
        distinct = [torch.stack([synth.kv_cache_plane(base, b, g, ctx) for g in range(n_kv)]).to(device)
                    for b in range(min(4, base.batch))]
        cache = torch.empty(base.batch, n_kv, ctx, 2 * base.head_dim, dtype=dt, device=device)
        for b in range(base.batch):
            cache[b].copy_(distinct[b % len(distinct)])
        M.mtla_cache_import(h, cache, ctx)
        torch.cuda.synchronize(device)
        del cache, distinct
        torch.cuda.empty_cache()
        per_token = M.mtla_cache_bytes(h) / (base.batch * ctx)
        ms, attn = time_steps(h, xs, y)
        rows.append({"method": name, "kv_heads": n_kv, "ms_per_step": ms, "attention_us": attn * 1e3,
                     "tokens_per_s": base.batch / (ms * 1e-3), "cache_bytes_per_token": per_token})
        M.mtla_destroy(h)
        del h
        torch.cuda.empty_cache()
    for s in (1, 2, 3, 4):
        w = base.scaled(stride=s, prefill_tokens=0, context_tokens=ctx, name=f"{base.name}[s={s}]")
        Mx, h = build_layer(w, extra_steps=2 * (K + W), device=device)
        fill_context(Mx, h, w, device)
        per_token = M.mtla_cache_bytes(h) / (w.batch * ctx)
        ms, attn = time_steps(h, xs, y)
        rows.append({"method": "MLA" if s == 1 else "MTLA", "stride": s, "ms_per_step": ms,
                     "attention_us": attn * 1e3, "tokens_per_s": w.batch / (ms * 1e-3),
                     "cache_bytes_per_token": per_token})
        M.mtla_destroy(h)
        del h
        torch.cuda.empty_cache()
    mha = rows[0]
    peaks = measured_peaks()
    for r in rows:
        r["speedup_vs_mha"] = mha["ms_per_step"] / r["ms_per_step"]
        r["cache_reduction_vs_mha"] = mha["cache_bytes_per_token"] / r["cache_bytes_per_token"]
        # The attention kernel's roofline: the cache read once per step against the copy peak.
        r["attention_gbs"] = r["cache_bytes_per_token"] * base.batch * ctx / (r["attention_us"] * 1e-6) / 1e9
        r["attention_frac_of_hbm_peak"] = r["attention_gbs"] / peaks["hbm_gbs"]
    print(json.dumps({
        "metric": METRIC, "unit": UNIT, "comparison": rows, "n_gpus": 1, "steps": K, "warmup": W,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"compare[{base.name}]", "batch": base.batch, "d_model": base.d_model,
                   "n_heads": base.n_heads, "head_dim": base.head_dim, "latent_rank": base.latent_rank,
                   "rope_dim": base.rope_dim, "context_tokens": ctx,
                   "note": "same width, batch and context for every method; decode steps with inputs "
                           "resident; attention_us from two events around the attention kernel"}}))


def prefill_flop(w: synth.Workload) -> dict:
    """FLOP the prefill must execute: un-absorbed attention over the pairs the stride-aware
    mask admits (row m sees ceil(m/s) columns), the fused input projection, the key / value
    up-projection of the running states and the output projection."""
    B, T, s = w.batch, w.prefill_tokens, w.stride
    d, nh, dh, r, dr = w.d_model, w.n_heads, w.head_dim, w.latent_rank, w.rope_dim
    m = np.arange(1, T + 1, dtype=np.int64)
    pairs = B * nh * int(((m + s - 1) // s).sum())
    parts = {"attention": pairs * (2 * (dh + dr) + 2 * dh),
             "input_proj": 2 * B * T * d * (nh * dh + nh * dr + r + dr),
             "kv_up_proj": 2 * B * T * r * 2 * nh * dh,
             "output_proj": 2 * B * T * nh * dh * d}
    parts["total"] = sum(parts.values())
    return parts


def fill_prompt(w: synth.Workload, device, distinct: int = 4) -> torch.Tensor:
    """Prompt activations [B][T][d]: `distinct` seeded sequences tiled over the batch (the values
    do not affect the timing; the parity tests use one seeded prompt per sequence)."""
    x = torch.empty(w.batch, w.prefill_tokens, w.d_model, dtype=synth.torch_dtype(w.dtype), device=device)
    rows = [synth.stored(synth.normal(w.seed, f"prompt/{b}", (w.prefill_tokens, w.d_model)), w.dtype).to(device)
            for b in range(min(distinct, w.batch))]
    for b in range(w.batch):
        x[b].copy_(rows[b % len(rows)])
    return x


def time_prefill(M, h, w: synth.Workload, x: torch.Tensor, device, runs: int = 3) -> dict:
    """One warm-up prefill, then `runs` timed ones (each from an empty cache); the median."""
    y = torch.empty_like(x)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    launches = 0
    for i in range(runs + 1):
        M.mtla_reset(h)
        torch.cuda.synchronize(device)
        l0 = M.mtla_launch_count(h)
        ev0.record()
        M.mtla_prefill(h, x, y)
        ev1.record()
        torch.cuda.synchronize(device)
        launches = M.mtla_launch_count(h) - l0
        times.append(ev0.elapsed_time(ev1))
    M.mtla_check(h)
    assert torch.isfinite(y[:, -1].float()).all()
    ms = float(np.median(times[1:]))
    peaks = measured_peaks()
    flop = prefill_flop(w)
    tensor_ms = flop["total"] / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
    return {"workload": w.name, "tokens_per_s": w.batch * w.prefill_tokens / (ms * 1e-3), "ms": ms,
            "ms_min": float(min(times[1:])), "first_run_ms": times[0], "timed_runs": runs,
            "batch": w.batch, "tokens": w.prefill_tokens, "algorithmic_tflop": flop["total"] / 1e12,
            "achieved_tflops": flop["total"] / (ms * 1e-3) / 1e12,
            "roofline": {"bound": "tensor", "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "peak_source": f"sustained bf16, of {peaks['source']}",
                         "roofline_ms": tensor_ms, "frac": tensor_ms / ms},
            "gpu_launches": int(launches)}


def time_decode(M, h, w: synth.Workload, device, steps: int, warmup: int) -> dict:
    """Decode steps with inputs resident, from the handle's current context."""
    dt = synth.torch_dtype(w.dtype)
    xs = [synth.decode_input(w, i).to(device) for i in range(8)]
    y = torch.empty(w.batch, w.d_model, dtype=dt, device=device)
    for i in range(warmup):
        M.mtla_decode_step(h, xs[i % 8], y)
    torch.cuda.synchronize(device)
    slots0, l0 = M.mtla_position(h)[1], M.mtla_launch_count(h)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(steps):
        M.mtla_decode_step(h, xs[i % 8], y)
    ev1.record()
    torch.cuda.synchronize(device)
    ms = ev0.elapsed_time(ev1) / steps
    slots1 = M.mtla_position(h)[1]
    M.mtla_check(h)
    assert torch.isfinite(y.float()).all()
    peaks = measured_peaks()
    work = algorithmic_work(w, 0.5 * (slots0 + 1 + slots1))
    hbm_s = (work["weight_bytes"] + work["cache_bytes"]) / (peaks["hbm_gbs"] * 1e9)
    tensor_s = (work["attn_flop"] + work["proj_flop"]) / (peaks["bf16_tflops_sustained"] * 1e12)
    return {"workload": w.name, "batch": w.batch, "stride": w.stride, "context_slots": [slots0, slots1],
            "decode_tokens_per_s": w.batch / (ms * 1e-3), "us_per_step": ms * 1e3,
            "roofline_us": max(hbm_s, tensor_s) * 1e6,
            "step_roofline_frac": max(hbm_s, tensor_s) / (ms * 1e-3),
            "launches_per_step": (M.mtla_launch_count(h) - l0) / steps, "steps": steps,
            "attention_variant": M.mtla_attention_variant(h)}


def stack_work(sw: synth.StackWorkload, n_slots: float) -> dict:
    """Bytes and FLOP of one decode step of the stack: every layer's attention work plus its
    feed-forward block (two d x d_ff matrices and their biases, the LayerNorm vectors)."""
    w = sw.layer
    e = 2 if w.dtype == "bf16" else 4
    a = algorithmic_work(w, n_slots)
    ffn_params = 2 * w.d_model * sw.d_ff + sw.d_ff + w.d_model + 4 * w.d_model
    return {"weight_bytes": sw.n_layers * (a["weight_bytes"] + ffn_params * e),
            "cache_bytes": sw.n_layers * a["cache_bytes"],
            "flop": sw.n_layers * (a["attn_flop"] + a["proj_flop"] + 2 * w.batch * ffn_params)}


def time_stack(sw: synth.StackWorkload, device, steps: int, warmup: int) -> dict:
    """The decoder stack: parallel prefill of the prompt through every layer, then decode steps
    (one token per sequence through all layers) with inputs resident."""
    from paper_2505_13544_b200 import binding as M
    w = sw.layer
    weights = synth.make_stack_weights(sw)
    cfg = M.make_config(**dims_of(w), max_batch=w.batch,
                        max_tokens=w.prefill_tokens + steps + warmup + 8,
                        max_prefill_tokens=w.prefill_tokens, dtype=w.dtype, ln_eps=w.ln_eps,
                        rope_theta=w.rope_theta)
    dev = {"layers": [{k: v.to(device) for k, v in lw.items()} for lw in weights["layers"]],
           "lnf_gamma": weights["lnf_gamma"].to(device), "lnf_beta": weights["lnf_beta"].to(device)}
    s = M.mtla_stack_create(cfg, sw.n_layers, sw.d_ff, dev, device=device)
    x = fill_prompt(w, device)
    y = torch.empty_like(x)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    for _ in range(3):
        M.mtla_stack_reset(s)
        torch.cuda.synchronize(device)
        ev0.record()
        M.mtla_stack_prefill(s, x, y)
        ev1.record()
        torch.cuda.synchronize(device)
        times.append(ev0.elapsed_time(ev1))
    M.mtla_stack_check(s)
    assert torch.isfinite(y[:, -1].float()).all()
    del x, y
    prefill_ms = float(np.median(times[1:]))
    dt = synth.torch_dtype(w.dtype)
    xs = [synth.decode_input(w, i).to(device) for i in range(8)]
    yd = torch.empty(w.batch, w.d_model, dtype=dt, device=device)
    for i in range(warmup):
        M.mtla_stack_decode_step(s, xs[i % 8], yd)
    torch.cuda.synchronize(device)
    l0 = M.mtla_stack_launch_count(s)
    slots0 = M.mtla_position(M.mtla_stack_layer(s, 0))[1]
    ev0.record()
    for i in range(steps):
        M.mtla_stack_decode_step(s, xs[i % 8], yd)
    ev1.record()
    torch.cuda.synchronize(device)
    ms = ev0.elapsed_time(ev1) / steps
    slots1 = M.mtla_position(M.mtla_stack_layer(s, 0))[1]
    M.mtla_stack_check(s)
    assert torch.isfinite(yd.float()).all()
    launches = (M.mtla_stack_launch_count(s) - l0) / steps
    cache_bytes = M.mtla_stack_cache_bytes(s)
    M.mtla_stack_destroy(s)
    peaks = measured_peaks()
    work = stack_work(sw, 0.5 * (slots0 + 1 + slots1))
    hbm_s = (work["weight_bytes"] + work["cache_bytes"]) / (peaks["hbm_gbs"] * 1e9)
    tensor_s = work["flop"] / (peaks["bf16_tflops_sustained"] * 1e12)
    return {"workload": sw.name, "n_layers": sw.n_layers, "d_ff": sw.d_ff, "batch": w.batch,
            "d_model": w.d_model, "stride": w.stride, "prompt_tokens": w.prefill_tokens,
            "prefill_ms": prefill_ms, "prefill_tokens_per_s": w.batch * w.prefill_tokens / (prefill_ms * 1e-3),
            "decode_tokens_per_s": w.batch / (ms * 1e-3), "us_per_step": ms * 1e3,
            "context_slots": [slots0, slots1], "launches_per_step": launches,
            "roofline_us": max(hbm_s, tensor_s) * 1e6,
            "step_roofline_frac": max(hbm_s, tensor_s) / (ms * 1e-3),
            "cache_bytes": cache_bytes,
            "note": "a step is one token per sequence through all layers; weights and caches of this "
                    "model fit L2, so the step is bound by kernel latency, not by HBM"}


def stack_cpu_baseline(sw: synth.StackWorkload, budget_s: float = 10.0) -> dict:
    """The decoder oracle's decode step, as it stands, on one sequence after the full prompt."""
    from oracle import decoder_oracle as D
    from tests import helpers as H
    from threadpoolctl import threadpool_info
    w = sw.layer
    sp = H.oracle_stack_params(sw, synth.make_stack_weights(sw))
    prompt = synth.stored(synth.normal(w.seed, "prompt/0", (w.prefill_tokens, w.d_model)), w.dtype)
    _, st = D.stack_forward_by_layers(sp, prompt.double().numpy(), rows=[])
    n, t0 = 0, time.perf_counter()
    while n < 64 and time.perf_counter() - t0 < budget_s:
        D.stack_decode_step(sp, st, synth.decode_input(w, n, batch=1)[0].double().numpy())
        n += 1
    el = time.perf_counter() - t0
    cores = max([int(i.get("num_threads", 1)) for i in threadpool_info()] + [1])
    return {"value": n / el, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"1 of {w.batch} sequences x {n} decode steps through {sw.n_layers} layers after a "
                      f"{w.prefill_tokens}-token prompt, {el:.1f} s"}


FP32_FMA_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # SMs x fp32 lanes x 2 FLOP x max SM clock


def time_training(device, batch: int = 8, tokens: int = 512, runs: int = 3,
                  cpu_baseline: bool = True) -> dict:
    """The training path on the paper's layer in fp32: mtla_prefill as the forward pass of the
    parallel form and mtla_train_backward as its reverse.  A step is forward + backward over
    `batch` sequences of `tokens` tokens; the roofline is plain fp32 FMA arithmetic (both passes
    run on the CUDA cores; TF32 would not hold the fp32 tolerance)."""
    from paper_2505_13544_b200 import binding as M
    w = synth.WORKLOADS["paper"].scaled(name="train_paper_fp32", dtype="fp32", batch=batch,
                                        prefill_tokens=tokens, decode_steps=2)
    Mx, h = build_layer(w, extra_steps=4, device=device)
    x = fill_prompt(w, device)
    dy = torch.randn(x.shape, device=device, generator=torch.Generator(device=device).manual_seed(w.seed))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    fwd, bwd = [], []
    launches = 0
    for _ in range(runs + 1):
        M.mtla_reset(h)
        torch.cuda.synchronize(device)
        l0 = M.mtla_launch_count(h)
        ev[0].record()
        M.mtla_prefill(h, x)
        ev[1].record()
        dx, grads = M.mtla_train_backward(h, x, dy)
        ev[2].record()
        torch.cuda.synchronize(device)
        launches = M.mtla_launch_count(h) - l0
        fwd.append(ev[0].elapsed_time(ev[1]))
        bwd.append(ev[1].elapsed_time(ev[2]))
    M.mtla_check(h)
    assert torch.isfinite(dx).all() and all(torch.isfinite(g).all() for g in grads.values())
    M.mtla_destroy(h)
    f_ms, b_ms = float(np.median(fwd[1:])), float(np.median(bwd[1:]))
    flop = prefill_flop(w)["total"]
    # The reverse pass costs two products per forward product; its attention works on dense
    # T x T matrices (all pairs, not only the s-th of them the mask admits).
    res = {"workload": w.name, "batch": batch, "tokens": tokens, "stride": w.stride, "dtype": "f32",
           "forward_ms": f_ms, "backward_ms": b_ms,
           "tokens_per_s": batch * tokens / ((f_ms + b_ms) * 1e-3),
           "algorithmic_tflop": 3 * flop / 1e12,
           "roofline": {"bound": "alu", "peak": FP32_FMA_TFLOPS, "unit": "TFLOP/s",
                        "peak_source": "148 SMs x 128 fp32 lanes x 2 x 1.965 GHz",
                        "achieved": 3 * flop / ((f_ms + b_ms) * 1e-3) / 1e12,
                        "frac": 3 * flop / ((f_ms + b_ms) * 1e-3) / 1e12 / FP32_FMA_TFLOPS},
           "gpu_launches": int(launches)}
    if cpu_baseline:
        from oracle import train_oracle as TR
        from tests import helpers as H
        p = H.oracle_params(w, synth.make_weights(w))
        xs = x[0].double().cpu().numpy()
        t0 = time.perf_counter()
        y, sv = TR.forward(p, xs)
        TR.backward(p, sv, dy[0].double().cpu().numpy())
        el = time.perf_counter() - t0
        res["cpu_baseline"] = {"value": tokens / el, "unit": "tokens/s", "kind": "oracle",
                               "sample": f"1 of {batch} sequences, forward + backward, {el:.1f} s"}
    return res


def run_other_configs(device, steps: int = 64, warmup: int = 8):
    """The other benchmark configurations, each for a fraction of a second: the parallel prefill
    of the long-context workload against the tensor roofline, and decode steps of every
    configuration at its full context."""
    prefill, configs = None, []
    for name in ("tiny", "paper", "sweep_s1", "sweep_s2", "sweep_s3", "sweep_s4", "longctx"):
        w = synth.WORKLOADS[name]
        M, h = build_layer(w, extra_steps=steps + warmup + 8, device=device)
        x = fill_prompt(w, device)
        pf = time_prefill(M, h, w, x, device, runs=3 if name == "longctx" else 1)
        del x
        torch.cuda.empty_cache()
        if name == "longctx":
            prefill = pf
        row = time_decode(M, h, w, device, steps, warmup)
        row["prefill_ms"] = pf["ms"]
        row["prefill_tokens_per_s"] = pf["tokens_per_s"]
        row["prefill_tensor_roofline_frac"] = pf["roofline"]["frac"] if w.dtype == "bf16" else None
        configs.append(row)
        M.mtla_destroy(h)
        del h
        torch.cuda.empty_cache()
    return prefill, configs


def run_sustained(M, h, w: synth.Workload, xs, y, local: int, device, seconds: float, step_ms: float,
                  max_steps: int):
    """The same decode loop for at least `seconds`, long enough for the board to settle under its
    power limit; clocks and power are sampled (never set) while it runs."""
    n = min(max_steps, int(math.ceil(seconds / (step_ms * 1e-3) * 1.1)))
    slots0 = M.mtla_position(h)[1]
    M.mtla_profile_begin_attention(h, n)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        torch.cuda.synchronize(device)
        ev0.record()
        for i in range(n):
            M.mtla_decode_step(h, xs[i % 8], y)
        ev1.record()
        torch.cuda.synchronize(device)
    ms = ev0.elapsed_time(ev1)
    attn_ms, attn_steps = M.mtla_profile_end(h)
    slots1 = M.mtla_position(h)[1]
    M.mtla_check(h)
    peaks = measured_peaks()
    work = algorithmic_work(w, 0.5 * (slots0 + 1 + slots1))
    attn_s = attn_ms * 1e-3 / max(attn_steps, 1)
    step_s = ms * 1e-3 / n
    hbm_s = (work["weight_bytes"] + work["cache_bytes"]) / (peaks["hbm_gbs"] * 1e9)
    return {"steps": n, "seconds": ms * 1e-3, "ms_per_step": ms / n,
            "tokens_per_s": w.batch * n / (ms * 1e-3), "context_slots": [slots0, slots1],
            "attention_us": attn_s * 1e6,
            "attention_gbs": work["cache_bytes"] / attn_s / 1e9,
            "attention_frac": work["cache_bytes"] / attn_s / 1e9 / peaks["hbm_gbs"],
            "attention_frac_of_nominal_8TBs": work["cache_bytes"] / attn_s / 1e9 / NOMINAL_HBM_GBS,
            "step_roofline_frac": hbm_s / step_s,
            "step_roofline_frac_of_nominal_8TBs":
                (work["weight_bytes"] + work["cache_bytes"]) / (NOMINAL_HBM_GBS * 1e9) / step_s,
            "clocks": clocks.summary()}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=256)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="large",
                    choices=sorted(synth.WORKLOADS) + sorted(synth.BEAM_WORKLOADS)
                    + sorted(synth.STACK_WORKLOADS) + ["train_paper_fp32"])
    ap.add_argument("--compare", action="store_true",
                    help="time MHA / GQA / MQA / MLA / MTLA at the workload's width, batch and one context")
    ap.add_argument("--paged", action="store_true",
                    help="keep the cache in 64-slot pages (mtla_create_paged) instead of contiguous rows")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch (profiling-sized variants)")
    ap.add_argument("--sustained-seconds", type=float, default=1.0,
                    help="length of the second, sustained timing loop (0 skips it)")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the prefill / other-configuration blocks of the default run")
    ap.add_argument("--context-tokens", type=int, default=0,
                    help="override the workload's imported context length")
    args = ap.parse_args()
    if args.impl == "reference":
        if (args.workload in synth.BEAM_WORKLOADS or args.workload in synth.STACK_WORKLOADS
                or args.workload == "train_paper_fp32"):
            raise SystemExit("--impl reference covers the decode workloads")
        run_reference(args)
        return

    import torch.distributed as dist
    from paper_2505_13544_b200 import replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier(device_ids=[local])
        torch.cuda.synchronize(device)

    if args.compare:
        if world > 1 or args.workload in synth.BEAM_WORKLOADS:
            raise SystemExit("--compare runs a decode workload on one GPU")
        run_compare(args, device, local)
        return
    if args.workload in synth.BEAM_WORKLOADS:
        if world > 1:
            raise SystemExit("the beam workloads run on one GPU")
        run_beam(args, synth.BEAM_WORKLOADS[args.workload], device, local)
        return
    if args.workload == "train_paper_fp32":
        # The training path alone (the `training` block of the default run): forward + backward.
        if world > 1:
            raise SystemExit("the training workload runs on one GPU")
        with ClockSampler(local) as clocks:
            res = time_training(device, runs=max(args.steps, 3) if args.steps < 16 else 3,
                                cpu_baseline=not args.no_cpu_baseline)
        ms = res["forward_ms"] + res["backward_ms"]
        print(json.dumps({"metric": "mtla_train_tokens_per_s", "value": res["tokens_per_s"], "unit": UNIT,
                          "n_gpus": 1, "steps": 3, "warmup": 1, "ms_per_step": ms, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                          "config": {"workload": res["workload"], "batch": res["batch"],
                                     "tokens": res["tokens"], "step": "forward + backward"},
                          "roofline": res["roofline"], "training": res,
                          "gpu_launches": res["gpu_launches"], "clocks": clocks.summary()}))
        return
    if args.workload in synth.STACK_WORKLOADS:
        if world > 1:
            raise SystemExit("the decoder-stack workload runs on one GPU")
        sw = synth.STACK_WORKLOADS[args.workload]
        with ClockSampler(local) as clocks:
            res = time_stack(sw, device, steps=args.steps, warmup=max(args.warmup, 3))
        line = {"metric": METRIC, "value": res["decode_tokens_per_s"], "unit": UNIT, "n_gpus": 1,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": res["us_per_step"] * 1e-3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if sw.layer.dtype == "bf16" else "f32", "data": "synthetic",
                "config": {"workload": sw.name, "batch": sw.layer.batch, "n_layers": sw.n_layers,
                           "d_model": sw.layer.d_model, "d_ff": sw.d_ff, "stride": sw.layer.stride,
                           "l2": "weights and caches fit L2: latency-bound, bandwidth figures are effective"},
                "decoder": res, "gpu_launches": int(round(res["launches_per_step"] * args.steps)),
                "clocks": clocks.summary()}
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = stack_cpu_baseline(sw)
        print(json.dumps(line))
        return
    w = pick_workload(args)
    K, W = args.steps, max(args.warmup, 3)
    # Room for the sustained loop: its step count follows the measured step time, bounded here by
    # the step's time at the nominal 8 TB/s (and by 4096 steps for the small configurations).
    floor_ms = algorithmic_work(w, (w.prefill_tokens + w.context_tokens) / w.stride)["cache_bytes"] / 8.0e9
    sustained_steps = 0
    if args.sustained_seconds > 0:
        sustained_steps = min(4096, int(args.sustained_seconds / max(floor_ms * 1e-3, 1e-5) * 1.1) + 8)
    M, h = build_layer(w, extra_steps=3 * (K + W) + sustained_steps, device=device, paged=args.paged)
    extras = fill_context(M, h, w, device)
    dt = synth.torch_dtype(w.dtype)
    xs = [synth.decode_input(w, i).to(device) for i in range(8)]
    y = torch.empty(w.batch, w.d_model, dtype=dt, device=device)

    # ---- device-resident timing: K decode steps, inputs already in HBM
    for i in range(W):
        M.mtla_decode_step(h, xs[i % 8], y)
    slots_begin = M.mtla_position(h)[1]
    launches0 = M.mtla_launch_count(h)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # Timed region: K steps with only the two events around the attention kernel.
    M.mtla_profile_begin_attention(h, K)
    with ClockSampler(local) as clocks:
        barrier()
        ev0.record()
        for i in range(K):
            M.mtla_decode_step(h, xs[i % 8], y)
        ev1.record()
        barrier()
    local_ms = ev0.elapsed_time(ev1)
    attn_ms, attn_steps = M.mtla_profile_end(h)
    launches = M.mtla_launch_count(h) - launches0
    slots_end = M.mtla_position(h)[1]
    M.mtla_check(h)
    value, ms = replicas.throughput(w.batch * K, local_ms, device)
    # The same K steps once more with an event between every pair of kernels: the breakdown.
    M.mtla_profile_begin(h, K)
    torch.cuda.synchronize(device)
    for i in range(K):
        M.mtla_decode_step(h, xs[i % 8], y)
    torch.cuda.synchronize(device)
    stage_ms, stage_steps = M.mtla_profile_end_stages(h)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    xh = [synth.decode_input(w, i).pin_memory() for i in range(8)]
    yh = torch.empty(w.batch, w.d_model, dtype=dt).pin_memory()
    for i in range(W):
        M.mtla_decode_step_host(h, xh[i % 8], yh)
    barrier()
    ev0.record()
    for i in range(K):
        M.mtla_decode_step_host(h, xh[i % 8], yh)
    ev1.record()
    barrier()
    e2e_value, _ = replicas.throughput(w.batch * K, ev0.elapsed_time(ev1), device)
    assert torch.isfinite(yh.float()).all()
    M.mtla_check(h)

    sustained = None
    if sustained_steps > 0:
        sustained = run_sustained(M, h, w, xs, y, local, device, args.sustained_seconds, local_ms / K,
                                  sustained_steps)

    if rank != 0:
        M.mtla_destroy(h)
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    n_slots = 0.5 * (slots_begin + 1 + slots_end)
    work = algorithmic_work(w, n_slots)
    attn_launch_s = attn_ms * 1e-3 / max(attn_steps, 1)
    achieved_gbs = work["cache_bytes"] / attn_launch_s / 1e9
    step_s = local_ms * 1e-3 / K
    hbm_time = (work["weight_bytes"] + work["cache_bytes"]) / (peaks["hbm_gbs"] * 1e9)
    tensor_time = (work["attn_flop"] + work["proj_flop"]) / (peaks["bf16_tflops_sustained"] * 1e12)
    # DRAM traffic of the attention kernel from the committed ncu capture, scaled by the cache
    # bytes of this launch; dropped once the kernel's source differs from the captured one.
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        t = json.load(open(tpath)).get(M.mtla_attention_variant(h), {})
        if t.get("dram_bytes_per_cache_byte") is not None and t.get("kernel_code_sha256") == kernel_code_hash():
            traffic = t["dram_bytes_per_cache_byte"] * work["cache_bytes"]

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "d_model": w.d_model,
                   "n_heads": w.n_heads, "head_dim": w.head_dim, "latent_rank": w.latent_rank,
                   "rope_dim": w.rope_dim, "stride": w.stride,
                   "context_slots": [slots_begin, slots_end],
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2: every step streams the whole cache "
                         f"({work['cache_bytes'] / 1e6:.0f} MB) and the weights"
                         if work["cache_bytes"] > 126e6 else
                         "cache smaller than L2: bandwidth figures are effective, not DRAM",
                   "storage": "paged, 64-slot pages" if args.paged else "contiguous",
                   "attention_variant": M.mtla_attention_variant(h)},
        "roofline": {"bound": "hbm", "kernel": "decode attention (a7)",
                     "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved_gbs / peaks["hbm_gbs"],
                     "peak_source": f"of {peaks['source']}",
                     "frac_of_nominal_8TBs": achieved_gbs / NOMINAL_HBM_GBS,
                     "launch_ms": attn_launch_s * 1e3, "traffic": traffic,
                     "note": "burst figure of the K-step region; the `sustained` block repeats it over "
                             "a loop of a second or more, under the board's power limit"},
        "step_roofline": {"hbm_time_ms": hbm_time * 1e3, "tensor_time_ms": tensor_time * 1e3,
                          "frac": max(hbm_time, tensor_time) / step_s,
                          "frac_of_nominal_8TBs": max(
                              (work["weight_bytes"] + work["cache_bytes"]) / (NOMINAL_HBM_GBS * 1e9),
                              tensor_time) / step_s},
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": w.batch * w.d_model * (2 if w.dtype == "bf16" else 4),
                "d2h_bytes_per_step": w.batch * w.d_model * (2 if w.dtype == "bf16" else 4)},
        "stage_us": {k: v * 1e3 / max(stage_steps, 1) for k, v in stage_ms.items()},
        "stage_us_note": "separate pass with an event between every pair of kernels (adds ~3 us each)",
        "gpu_launches": int(launches),
        "clocks": clocks.summary(),
    }
    if sustained:
        line["sustained"] = sustained
    if extras:
        line["prefill_of_this_workload"] = extras
    M.mtla_destroy(h)
    del h, xs, y
    torch.cuda.empty_cache()
    if world == 1 and args.workload == "large" and not args.no_other_configs and not args.batch:
        line["prefill"], line["configs"] = run_other_configs(device)
        line["decoder"] = time_stack(synth.STACK_WORKLOADS["decoder_paper"], device, steps=64, warmup=8)
        line["training"] = time_training(device, cpu_baseline=not args.no_cpu_baseline)
    if world == 1 and not args.no_cpu_baseline:
        n_seq = 1 if w.batch * w.latent_rank >= 8192 else min(w.batch, 4)
        res = oracle_decode_sample(w, n_seq, budget_s=12.0, max_steps=64)
        line["cpu_baseline"] = {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
