"""The FLOP / byte model the bench reports against, pinned to the paper's Table 1 (LA MACs per layer)
and to the state size it prints (1.0 MiB per layer = 16 heads x 128 x 128 x fp32)."""
import json
import os

from paper_2609_32114_b200 import synth


def test_table1_mac_column(golden_dir):
    with open(os.path.join(golden_dir, "table1_la_macs.json")) as f:
        t = json.load(f)
    per_chunk_head = synth.macs_per_chunk_head(t["chunk"], t["head_dim"])
    assert per_chunk_head == 5898240
    for tokens, gmac in zip(t["tokens"], t["gmac"]):
        ours = per_chunk_head * (tokens // t["chunk"]) * t["heads"] / 1e9
        assert abs(ours - gmac) <= 0.0051, (tokens, ours, gmac)      # the table prints two decimals
    assert t["heads"] * t["head_dim"] ** 2 * 4 / 2 ** 20 == t["state_mib"]


def test_algorithmic_work_of_the_headline_workload():
    w = synth.WORKLOADS["gdn_layer_4k"]
    assert synth.algorithmic_flops(w, 4096) == 2 * 5898240 * 64 * 16          # 12.08 GFLOP
    assert synth.algorithmic_bytes(w, 4096, 1) == 4096 * 16512 + 16 * 128 * 128 * 4   # 68.68 MB
    k = synth.WORKLOADS["kda_8k"]
    assert synth.algorithmic_bytes(k, 8192, 1) == 8192 * 32 * 1540 + 32 * 128 * 128 * 4


def test_traffic_table_is_rebuilt_from_the_committed_summaries():
    """profiles/traffic.json (what bench.py reports as `roofline.traffic`) is exactly what the summary tool derives
    from the ncu summaries beside it: no hand-copied constants."""
    import json
    import os

    from paper_2609_32114_b200 import ncu_summary

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with open(os.path.join(root, "profiles", "traffic.json")) as f:
        stored = json.load(f)
    assert stored == json.loads(json.dumps(ncu_summary.traffic()))
    chain = stored["gdn_layer_4k"]["tc_chain"]
    assert chain["dram_read"] > 0 and chain["source"].endswith(".md")
