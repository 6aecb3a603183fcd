"""Host-side helpers of bench.py that need no GPU: the table of ncu DRAM bytes it reads for `roofline.traffic`."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_dram_traffic_table_has_a_row_for_each_timed_kernel():
    """One row per kernel and expert shape: the single-CTA kernel on C2-shaped and C3-shaped experts (the default
    launches of the bench workloads), the CTA-pair kernel on C2-shaped experts (--pairs on)."""
    pair = bench.dram_traffic_per_expert("expert_ffn_pair_kernel<false>", 4096, 14336)
    dense = bench.dram_traffic_per_expert("expert_ffn_kernel<false>", 4096, 14336)
    small = bench.dram_traffic_per_expert("expert_ffn_kernel<false>", 7168, 2048)
    assert pair is not None and dense is not None and small is not None
    # per expert: gate + up weights once (2 F H bf16) plus that expert's rows; never below the weights alone
    for v in (pair, dense):
        assert v >= 2 * 14336 * 4096 * 2 and v < 1.2 * (2 * 14336 * 4096 * 2 + 2048 * (4096 + 14336) * 2)
    assert small >= 2 * 2048 * 7168 * 2 and small < 1.1 * (2 * 2048 * 7168 * 2) + 2e6
    assert bench.dram_traffic_per_expert("no_such_kernel", 4096, 14336) is None
    assert bench.dram_traffic_per_expert("expert_ffn_kernel<false>", 1, 1) is None


def test_workload_config_names_the_workload_and_the_l2_policy():
    cfg = bench.gen.CONFIGS["C2"]
    c = bench.workload_config(cfg, 2)
    assert c["workload"].startswith("C2: T=8192") and c["global_tokens"] == 2 * 8192
    assert "larger than L2" in c["l2_policy"] and "model" not in c
