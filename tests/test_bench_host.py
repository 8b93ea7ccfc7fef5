"""Host logic of bench.py that needs no GPU: the byte accounting of a decode step (exactness-aware trimming), the
table of profiler traffic figures it reads, the measured-peaks lookup and the clock-sample parser."""
import importlib.util
import json
import os

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_evaluated_layers_follow_the_exactness_counter(bench):
    """Sweep k of a decode step (prefix 0, h0 initialisation) evaluates blocks k..L-1: the states 0..k are exact after
    k sweeps (finite-step exactness), so re-evaluating the blocks before them would reproduce stored outputs."""
    for L in (1, 3, 20, 32):
        for K in range(0, L + 4):
            exact, want = 0, []
            for _ in range(K):
                b0 = min(exact, L)
                want.append(L - b0)
                exact += 1
            assert bench.evaluated_layers(L, K) == want
    assert bench.evaluated_layers(20, 2) == [20, 19]


def test_d20_step_bytes(bench):
    """d20, batch 1, ctx 2048, K = 2: (20 + 19) / 20 of one sweep's weights and keys/values plus the LM head."""
    cfg = bench.d20()
    w, kv, lm = bench.alg_bytes(cfg, 1, 2048)
    assert w == {"qkv": 196608000, "out_proj": 65536000, "mlp_up": 262144000, "mlp_down": 262144000}
    assert kv == 20 * 2 * 2048 * 1280 * 2 and lm == 65536 * 1280 * 2
    layers = bench.evaluated_layers(cfg.n_layer, 2)
    step = sum(layers) / cfg.n_layer * (sum(w.values()) + kv) + lm
    assert step == 2110259200                 # 2.11 GB moved per step from a cache of exactly 2048 positions
    untrimmed = 2 * (sum(w.values()) + kv) + lm
    assert untrimmed == 2160066560            # the untrimmed figure quoted beside it
    assert kv % 8 == 0 and bench.alg_bytes(cfg, 8, 2048)[1] == 8 * kv


def test_profiler_traffic_table_is_close_to_the_algorithmic_bytes(bench):
    """roofline.traffic comes from the table kept beside the ncu summary; every class the benchmark can name as its
    dominant kernel is there, and no launch moves more than a few per cent above its algorithmic bytes."""
    cfg = bench.d20()
    w, _, _ = bench.alg_bytes(cfg, 1, 2048)
    want = dict(w)
    want["chain"] = w["out_proj"] + w["mlp_up"] + w["mlp_down"]
    for cls, alg in want.items():
        t = bench.ncu_traffic(cls)
        assert t is not None, cls
        assert alg <= t <= 1.04 * alg, (cls, t, alg)
    assert bench.ncu_traffic("no_such_class") is None


def test_peaks_come_from_the_measured_file_or_the_stated_fallback(bench):
    value, source = bench.peaks()
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        assert value == pytest.approx(json.load(open(path))["hbm_gbs"])
        assert "measured" in source
    else:
        assert value == pytest.approx(6650.0) and "fallback" in source
    assert bench.HBM_NOMINAL_GBS == 8000


def test_clock_sampler_parses_samples_and_reasons(bench, tmp_path):
    s = bench.ClockSampler(0)

    class Done:
        def terminate(self): pass
        def wait(self, timeout=None): return 0
        def kill(self): pass
    s.proc = Done()
    s.path = str(tmp_path / "clocks.csv")
    open(s.path, "w").write("1965, 1965, Not Active, Not Active, Not Active, Not Active\n"
                            "1800, 1965, Not Active, Not Active, Not Active, Active\n"
                            "1700, 1965, Not Active, Not Active, Not Active, Active\n"
                            "garbage line\n")
    got = s.stop()
    assert got["sm_mhz"] == 1800 and got["sm_max_mhz"] == 1965 and got["samples"] == 3
    assert got["reasons"] == ["sw_power_cap"]
    assert bench.ClockSampler(0).stop()["reasons"] == ["nvidia-smi unavailable"]


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` times the CPU oracle on the benchmark's point and prints one JSON line with the
    same metric, unit and workload as the CUDA arm, marked as the reference, with no device traffic."""
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "tokens/s" and d["higher_is_better"] is True
    assert d["metric"].startswith("d20 decode tokens/s") and "d20 decode" in d["config"]["workload"]
    assert d["dtype"] == "f64" and d["data"] == "synthetic" and d["vs_baseline"] is None and d["n_gpus"] == 1
    assert d["value"] > 0 and d["ms_per_step"] == pytest.approx(1000.0 / d["value"], rel=1e-6)
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and "oracle" in cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
