"""Host-side accounting of bench.py: the algorithmic work of a step and the DRAM traffic it reads from the
committed ncu summary of the gate/up projection."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2509_23094_b200 import inputs  # noqa: E402


def test_algorithmic_work_of_the_default_workload():
    """One LLaDA-8B-shaped layer, L = 1024, 835 selected rows of which 32 are masked: the figures quoted for it."""
    wl = inputs.WORKLOADS["llada1l_1024"]
    sh = wl.shape
    flops, byts = bench.algorithmic_work(sh, 1, 1024, [835], 32, 1)
    d, F, V, H, Dh = sh.d_model, sh.d_ffn, sh.vocab, sh.n_q_heads, sh.head_dim
    per_layer = d * (H + 2 * sh.n_kv_heads) * Dh + H * Dh * d + 3 * d * F
    assert sh.params_per_layer == per_layer
    assert flops == 2 * 835 * per_layer + 4 * H * Dh * 835 * 1024 + 2 * 32 * d * V
    assert 4.0e11 < flops < 4.2e11 and 1.50e9 < byts < 1.54e9
    # every weight byte once: the weights dominate the bytes
    assert byts > 2 * per_layer + 2 * d * V


def test_traffic_is_read_from_the_committed_summary():
    """The gate/up block of the committed capture: DRAM bytes within a few per cent of the algorithmic bytes of that
    launch (201.3 MB of weights + 6.8 MB in + 20.5 MB out), and a missing tag gives None with a reason."""
    t, src = bench.profiled_traffic("gate/up")
    assert t is not None and "profiles/" in src
    assert 0.98 * 228.7e6 < t < 1.15 * 228.7e6
    t2, why = bench.profiled_traffic("no such kernel")
    assert t2 is None and why
