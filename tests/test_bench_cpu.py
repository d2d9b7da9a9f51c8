"""bench.py's bookkeeping, without a GPU: the algorithmic bytes behind the roofline figure and
the code hash that ties the committed DRAM-traffic capture to the kernel source."""
import importlib.util
import json
import os

from paper_2505_13544_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)


def test_algorithmic_bytes_per_slot_row():
    """(r + d_R) elements of 2 bytes per slot and sequence: 1152 B at the large layer, 576 B at
    the paper's (Section 4.3: 4.5 d_h elements per slot)."""
    big = synth.WORKLOADS["large"]
    assert bench.algorithmic_work(big, 1.0)["cache_bytes"] == big.batch * 1152
    small = synth.WORKLOADS["paper"]
    assert bench.algorithmic_work(small, 1.0)["cache_bytes"] == small.batch * 576
    assert small.slot_width == 4.5 * small.head_dim
    # Attention FLOP per slot and head: a score over r + d_R columns and a value update over r.
    assert bench.algorithmic_work(big, 1.0)["attn_flop"] == big.batch * big.n_heads * (2 * 576 + 2 * 512)


def test_traffic_capture_is_keyed_to_the_kernel_code():
    t = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))["tcgen05"]
    assert len(t["kernel_code_sha256"]) == 64 and 1.0 <= t["dram_bytes_per_cache_byte"] < 1.2
    assert bench.kernel_code_hash() == bench.kernel_code_hash()
    # bench.py reports the capture only while the hash matches (null otherwise): a comment-only
    # edit must not change it, a code edit must.
    text = "int a = 1;   // one\n\n  int b = 2;\n"
    assert bench.code_hash([text]) == bench.code_hash(["int a = 1;\nint b = 2; // two\n// three\n"])
    assert bench.code_hash([text]) != bench.code_hash([text + "int c = 3;\n"])


def test_prefill_flop_of_the_long_context_workload():
    """Allowed pairs B n_h sum_m ceil(m/s) at 2 (d_h + d_R) + 2 d_h FLOP each, plus the three
    projections: 2.90 TFLOP for 8 x 16384 tokens at s = 4."""
    f = bench.prefill_flop(synth.WORKLOADS["longctx"])
    assert abs(f["attention"] / 1e12 - 1.65) < 0.01
    assert abs(f["total"] / 1e12 - 2.90) < 0.01
    w = synth.WORKLOADS["tiny"].scaled(batch=1, prefill_tokens=5, stride=2)
    pairs = 1 + 1 + 2 + 2 + 3                      # ceil(m/2) for m = 1..5
    assert bench.prefill_flop(w)["attention"] == w.n_heads * pairs * (2 * (64 + 32) + 2 * 64)
