"""Host logic of bench.py that needs no GPU: which measured peak a timed region is held against, and how the
DRAM traffic of a kernel is taken from the committed ncu summaries (scaled by the batch, dropped once the
kernel's sources have changed since the capture)."""
import re
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))

import bench  # noqa: E402

PEAKS = {"hbm_gbs": 6455.6, "bf16_tflops": 1691.3, "bf16_tflops_sustained": 1444.3, "source": "measured"}


def test_peak_follows_the_timed_region():
    short_full_clock = {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": []}
    peak, why = bench.pick_tensor_peak(PEAKS, short_full_clock, 0.05)
    assert peak == 1691.3 and "burst" in why
    peak, why = bench.pick_tensor_peak(PEAKS, short_full_clock, 2.0)          # seconds long
    assert peak == 1444.3 and "sustained" in why
    capped = {"sm_mhz": 1485.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"]}
    peak, why = bench.pick_tensor_peak(PEAKS, capped, 0.5)                    # short, but against the power cap
    assert peak == 1444.3 and "power cap" in why
    low_clock_no_reason = {"sm_mhz": 1200.0, "sm_max_mhz": 1965.0, "reasons": []}
    assert bench.pick_tensor_peak(PEAKS, low_clock_no_reason, 0.5)[0] == 1444.3
    assert bench.pick_tensor_peak(PEAKS, {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}, 0.5)[0] == 1691.3


def test_traffic_comes_from_the_committed_summary_and_scales_with_the_batch(monkeypatch):
    summary = ROOT / "profiles" / "attn_bwd_fused_sm100_kernel_train_batch.md"
    text = summary.read_text()
    per_launch = float(re.search(r"DRAM traffic per launch = ([0-9.eE+]+) bytes", text).group(1))
    recorded = re.search(r"kernel sources sha256: ([0-9a-f]+)", text).group(1)
    assert re.search(r"captured batch: 1\b", text)
    # sources as they were at the capture: the batch-1 figure times the batch
    monkeypatch.setattr(bench, "kernel_source_digest", lambda kernel: recorded)
    got, note = bench.ncu_traffic("attn_bwd_fused_sm100_kernel", "train_batch", 4)
    assert got == 4 * per_launch and "scaled x4" in note
    # a kernel that changed since: no figure, and the reason is given
    monkeypatch.setattr(bench, "kernel_source_digest", lambda kernel: "0" * 16)
    got, note = bench.ncu_traffic("attn_bwd_fused_sm100_kernel", "train_batch", 4)
    assert got is None and "changed" in note
    got, note = bench.ncu_traffic("attn_bwd_fused_sm100_kernel", "no_such_workload", 1)
    assert got is None and "no ncu capture" in note


def test_source_digest_covers_the_kernels_files():
    d = bench.kernel_source_digest("attn_fwd_sm100_kernel")
    assert re.fullmatch(r"[0-9a-f]{16}", d)
    assert d != bench.kernel_source_digest("decode_split_kernel")
    for files in bench.KERNEL_SOURCES.values():
        for f in files:
            assert (ROOT / "paper_2509_15763_b200" / "csrc" / f).exists(), f
