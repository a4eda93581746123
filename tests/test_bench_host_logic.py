"""Host-side arithmetic of bench.py that the JSON line depends on (no GPU): the roofline floors, the scaling of a
bounded oracle sample to whole batches, the staleness rule of the captured DRAM traffic."""
import importlib.util
import sys
from pathlib import Path
from types import SimpleNamespace

import torch

ROOT = Path(__file__).resolve().parent.parent
spec = importlib.util.spec_from_file_location("bench_module", ROOT / "bench.py")
bench = importlib.util.module_from_spec(spec)
sys.modules["bench_module"] = bench
spec.loader.exec_module(bench)

from paper_2401_15077_b200 import workloads as W  # noqa: E402


def test_floors_and_binding_bound():
    pk = {"hbm": 6550.4, "tc_burst": 1627.0, "tc_sustained": 1356.9, "sm_max_mhz": 1965.0}
    # a 70B-like launch: 76 MB, 32.7 Gflop -> the tensor pipe binds at the burst peak
    ctx = SimpleNamespace(alg_bytes=76_000_000, alg_flops=32_700_000_000, alg_exps=32_700_000_000 // 512)
    r = bench.bounds(ctx, 0.043, pk, long_run=False)
    assert r["bound"] == "tensor"
    assert abs(r["t_hbm_ms"] - 76e6 / 6550.4e9 * 1e3) < 1e-9 and abs(r["t_mma_ms"] - 32.7e9 / 1627e12 * 1e3) < 1e-9
    assert abs(r["frac_of_binding_bound"] - r["t_mma_ms"] / 0.043) < 1e-12
    assert abs(r["hbm_frac"] - 76e6 / 0.043e-3 / 1e9 / 6550.4) < 1e-12
    assert abs(r["hbm_frac_nominal"] / r["hbm_frac"] - 6550.4 / 8000.0) < 1e-12
    assert abs(r["t_exp_ms"] - (32.7e9 // 512) / (148 * 16 * 1965e6) * 1e3) < 1e-6
    # a long run is held against the sustained tensor peak
    assert bench.bounds(ctx, 0.043, pk, long_run=True)["tensor_peak"] == 1356.9
    # an HBM-bound launch
    ctx2 = SimpleNamespace(alg_bytes=1_170_000_000, alg_flops=170_000_000_000, alg_exps=170_000_000_000 // 512)
    assert bench.bounds(ctx2, 0.218, pk, long_run=False)["bound"] == "hbm"


def test_sample_is_scaled_by_its_share_of_the_work():
    cfg = W.scaled(W.CONFIGS["tiny"], batch=4, prefix=(100, 100), tree=(8, 8))
    attn = SimpleNamespace(cfg=cfg, seq_lens=torch.tensor([100, 300, 100, 500]), tree_sizes=torch.tensor([8, 8, 8, 8]))
    work = [(100 + 8) * 8, (300 + 8) * 8, (100 + 8) * 8, (500 + 8) * 8]
    v, share = bench.scaled_steps_per_s(attn, 2, 4.0)
    assert abs(share - (work[0] + work[1]) / sum(work)) < 1e-12 and abs(v - share / 4.0) < 1e-12
    v_all, share_all = bench.scaled_steps_per_s(attn, 4, 10.0)
    assert share_all == 1.0 and v_all == 0.1


def test_captured_traffic_is_null_when_the_kernel_source_changed(monkeypatch):
    cfg = W.CONFIGS["serving_mix"]
    value, note = bench.ncu_traffic(cfg)
    # the committed constant belongs to the committed kernel source
    assert value is not None and 1.15e9 < value < 1.25e9 and "ncu capture" in note
    monkeypatch.setitem(bench.NCU_TRAFFIC, "attn_cu_sha256", "0" * 64)
    value, note = bench.ncu_traffic(cfg)
    assert value is None and note.startswith("stale")
    assert bench.ncu_traffic(W.CONFIGS["tiny"])[0] is None
