"""Host-side arithmetic of bench.py (no GPU): the bytes -> latency view of the paper's memory model
(Sec. 6 and the hardware-simulation appendix: DRAM 60 GB/s, Flash 1 GB/s, compute ignored), the
algorithmic byte counts behind the roofline, and the keep-count / capacity conventions they use."""
import importlib.util
import os

import pytest

import dip_inputs as di

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_mod", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_simulator_view_on_hand_worked_counters(bench):
    """Two layers, three tokens, d_model 256 / d_ff 512, INT4 (half a byte per weight).
    A gate/up column is 2 * 512 * 0.5 = 512 B, a down column 256 * 0.5 = 128 B.
    Counters summed over layers: gate/up 60 hits + 36 misses, down 150 hits + 90 misses; six updates
    per cache kind = 2 layers x 3 tokens.
      DRAM bytes per token  = ((60 + 36) * 512 + (150 + 90) * 128) / 3 = (49152 + 30720) / 3 = 26624
      Flash bytes per token = (36 * 512 + 90 * 128) / 3 = (18432 + 11520) / 3 = 9984
      time per token = 26624 / 60e9 + 9984 / 1e9 = 4.437333e-7 + 9.984e-6 = 1.04277333e-5 s"""
    w = di.WORKLOADS["phi3_mini"].scaled(d_model=256, d_ff=512)
    meta_gu = [0, 6, 60, 36, 0, 0, 0, 0]
    meta_d = [0, 6, 150, 90, 0, 0, 0, 0]
    v = bench.simulator_view(w, 2, meta_gu, meta_d)
    assert v["dram_bytes_per_token"] == pytest.approx(26624.0, rel=1e-12)
    assert v["flash_bytes_per_token"] == pytest.approx(9984.0, rel=1e-12)
    assert v["mlp_tokens_per_s"] == pytest.approx(1.0 / 1.04277333333e-5, rel=1e-9)
    assert v["dense_mlp_bytes_per_token"] == 2 * 3 * 256 * 512 * 0.5
    # no misses: DRAM only; only misses: every used byte also crosses the Flash link once
    v = bench.simulator_view(w, 2, [0, 6, 96, 0, 0, 0, 0, 0], [0, 6, 240, 0, 0, 0, 0, 0])
    assert v["flash_bytes_per_token"] == 0 and v["mlp_tokens_per_s"] == pytest.approx(60e9 / 26624.0, rel=1e-12)
    v = bench.simulator_view(w, 2, [0, 6, 0, 96, 0, 0, 0, 0], [0, 6, 0, 240, 0, 0, 0, 0])
    assert v["flash_bytes_per_token"] == v["dram_bytes_per_token"] == pytest.approx(26624.0)
    assert v["mlp_tokens_per_s"] == pytest.approx(1.0 / (26624.0 / 60e9 + 26624.0 / 1e9), rel=1e-12)
    # a slower Flash link scales the miss term alone
    v2 = bench.simulator_view(w, 2, meta_gu, meta_d, flash_gbs=0.5)
    assert 1.0 / v2["mlp_tokens_per_s"] == pytest.approx(26624.0 / 60e9 + 9984.0 / 0.5e9, rel=1e-12)


def test_algorithmic_bytes_phi3_medium(bench):
    """Kept-column bytes of one MLP-step at 5120 / 17920, bf16, keep ratio 0.25 with caches:
    gate/up 1280 * 2 * 17920 * 2 + 4 * (5120 + 1280 + 17920); down 4480 * 5120 * 2 + 4 * (17920 + 4480 + 5120)."""
    w = di.WORKLOADS["phi3_medium"]
    assert (w.k_x, w.k_h, w.cap_gu, w.cap_d) == (1280, 4480, 2560, 8960)
    b = bench.algorithmic_bytes(w, w.k_x, w.k_h, True)
    assert b["gate_up"] == 91_750_400 + 97_280 == 91_847_680
    assert b["down"] == 45_875_200 + 110_080 == 45_985_280
    assert b["step"] == b["gate_up"] + b["down"] + 4 * (5120 + 17920) + 4 * (1280 + 4480) + 8 * (5120 + 17920)
    # INT4: half a byte per weight plus the binary16 scale rows of the groups touched
    w4 = di.WORKLOADS["llama3_8b_int4"]
    b4 = bench.algorithmic_bytes(w4, w4.k_x, w4.k_h, True)
    assert b4["gate_up"] == 1024 * 2 * 14336 // 2 + 4 * (4096 + 1024 + 14336) + 32 * 2 * 14336 * 2
    assert b4["down"] == 3584 * 4096 // 2 + 4 * (14336 + 3584 + 4096) + 112 * 4096 * 2


def test_whole_job_rate_and_median(bench):
    assert bench.whole_job_rate(40 * 20, 4, 10.0) == pytest.approx(320000.0)
    assert bench.median_repeat([3.0, 1.0, 2.0]) == 2.0
    assert bench.median_repeat([4.0, 1.0, 2.0, 3.0]) == 3.0      # upper median: an actual repeat
