"""Host-side logic of bench.py that needs no GPU: which measured peak a tensor fraction is quoted against, and the
description of the workload in the bench line."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))

import bench  # noqa: E402
from paper_2412_04757_b200 import inputs  # noqa: E402

PEAKS = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6400.0, "source": "measured"}


def test_burst_peak_only_at_full_clock_without_a_power_cap():
    # the burst figure when the sampled SM clock stayed at >= 95 % of its maximum and no power cap was active while
    # the kernels ran, the sustained one otherwise; every other denominator is always reported beside it
    at_max = bench.tensor_roofline(800.0, PEAKS, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": []})
    assert at_max["peak"] == 1600.0 and abs(at_max["frac"] - 0.5) < 1e-12 and "burst" in at_max["of"]
    capped = bench.tensor_roofline(800.0, PEAKS, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": ["sw_power_cap"]})
    assert capped["peak"] == 1400.0 and "sustained" in capped["of"]
    slow = bench.tensor_roofline(800.0, PEAKS, {"sm_mhz": 1800.0, "sm_max_mhz": 1965.0, "reasons": []})
    assert slow["peak"] == 1400.0
    unknown = bench.tensor_roofline(800.0, PEAKS, {})
    assert unknown["peak"] == 1400.0                       # no clock record: the cautious denominator
    for r in (at_max, capped, slow, unknown):
        assert abs(r["frac_burst"] - 0.5) < 1e-12 and abs(r["frac_sustained"] - 800.0 / 1400.0) < 1e-12
        assert abs(r["frac_nominal"] - 800.0 / bench.NOMINAL_BF16_TFLOPS) < 1e-12
    assert bench.tensor_roofline(None, PEAKS, {})["frac"] is None


def test_workload_description_names_the_configuration():
    cfg = inputs.config(2)
    w = bench.workload_config(cfg, world=1, nseq=1)
    assert w["workload"].startswith(cfg.name) and w["parallelism"] == "single GPU"
    assert bench.workload_config(cfg, world=4, nseq=1)["parallelism"] == "replicas only"
    assert (w["layers"], w["q_heads"], w["kv_heads"], w["context"], w["chunk"], w["window"], w["sink"], w["top_k"]) == (
        cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.context, cfg.chunk, cfg.window, cfg.n_sink, cfg.top_k)
    assert "model" not in w
    # algorithmic keys of the local part per row: sink + local window + the causal half of the call
    assert bench.local_keys(cfg, t0=cfg.context - cfg.chunk, n=cfg.chunk, E=cfg.context - cfg.chunk - cfg.window) == (
        cfg.n_sink + cfg.window + (cfg.chunk + 1) / 2.0)
