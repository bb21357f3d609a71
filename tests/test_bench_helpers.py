"""Host-side logic of bench.py that needs no GPU: where the ncu DRAM-traffic figure of the bench line comes
from, and the algorithmic byte counts."""
import os
import re

import numpy as np

import bench
import csp_synth as synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_traffic_comes_from_the_committed_summary_of_that_kernel_workload_and_launch():
    found = 0
    for name in sorted(os.listdir(os.path.join(ROOT, "profiles"))):
        text = open(os.path.join(ROOT, "profiles", name)).read()
        m = re.search(r"^dram_bytes_per_launch:\s*([0-9.eE+]+)", text, re.M)
        mm = re.match(r"(score|select_compact|select|compact|decode_attn)[a-z_]*_(configs\d(?:_\d+pct)?)_(all_layers_one_call|one_layer_per_call)\.md$", name)
        if not (m and mm):
            continue
        got, src = bench.ncu_traffic(mm.group(1), mm.group(2), mm.group(3))
        assert got == float(m.group(1)) and src == os.path.join("profiles", name)
        found += 1
    assert found >= 1
    assert bench.ncu_traffic("score", "configs9", "all_layers_one_call") == (None, None)
    assert bench.ncu_traffic("score", "configs1", "some_other_launch") == (None, None)


def test_algorithmic_bytes_of_the_headline_workload():
    cfg = synth.config(1)
    ab = bench.algorithmic_bytes(cfg, cfg.seq_lens, 32 * 1027)
    k_bytes = 4096 * 32 * 128 * 2
    assert ab["score"] == k_bytes + 32 * 32 * 128 * 2 + 4096 + 2 * 4 * 4064 * 32
    assert ab["compact"] == 32 * 1027 * (4 + 2 * 2 * 256 + 2)
    assert ab["total"] == ab["score"] + ab["select"] + ab["compact"]
    assert ab["select_compact"] == ab["select"] + ab["compact"]
    assert abs(ab["total"] - 70.0e6) < 0.5e6


def test_launch_count_of_a_call():
    """Kernels per csp_prune_layer call as the bench line claims them: the ordering kernel for batches of sequences, one
    kernel for selection and compaction where at least an SM's worth of units hold 1 K - 4 K positions each (two per SM up to 8 K)."""
    class P:
        def __init__(self, batch, n_kv_heads, max_len, out_capacity=100, dtype=1):
            self.batch, self.n_kv_heads, self.max_len, self.out_capacity, self.dtype = batch, n_kv_heads, max_len, out_capacity, dtype
    assert bench.kernels_per_call(P(32, 32, 4096), 148) == 3        # order, score, selection + compaction
    assert bench.kernels_per_call(P(1, 32, 4096), 148) == 3         # one sequence: score, select, compact
    assert bench.kernels_per_call(P(32, 32, 16384), 148) == 4       # too long for one CTA's selection
    assert bench.kernels_per_call(P(32, 8, 8109), 148) == 4         # more than 4096 positions and fewer than two units per SM
    assert bench.kernels_per_call(P(32, 32, 8109, 811), 148) == 3   # 1024 units of up to 8109 positions, a tenth kept
    assert bench.kernels_per_call(P(32, 32, 8109, 405), 148) == 4   # too few rows to copy for the selection to hide
    assert bench.kernels_per_call(P(4, 32, 4096), 148) == 4         # 128 units: fewer than one per SM
    assert not bench.fused_select_compact(P(32, 32, 1024), 148) and bench.fused_select_compact(P(37, 4, 1025), 148)


def test_help_text_renders():
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--help"], capture_output=True, text=True)
    assert out.returncode == 0 and "--all-configs" in out.stdout
