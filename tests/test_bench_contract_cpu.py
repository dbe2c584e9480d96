"""The benchmark's reference arm (the CPU oracle on the host cores) prints one JSON line with the agreed keys, and both
arms describe the workload with the same `config`.  Runs without a GPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "1", "--steps", "1",
                          "--warmup", "1"], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "wnw_decode_tokens_per_s_at_20pct_audio_budget" and d["unit"] == "tokens/s"
    assert d["n_gpus"] == 1 and d["steps"] == 1 and d["warmup"] == 1 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["vs_baseline"] is None and d["dtype"] == "f64" and d["data"] == "synthetic"
    assert d["value"] > 0 and abs(d["value"] * d["ms_per_step"] * 1e-3 - d["config"]["batch"]) < 1e-6
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and "layers" in cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    cfg = d["config"]
    assert cfg["workload"] == "cfg1_voxtral3b_4min" and cfg["layers"] == 30 and cfg["layer_issue"] == "chained"
    assert (cfg["q_heads"], cfg["kv_heads"], cfg["head_dim"], cfg["batch"], cfg["audio_budget"]) == (32, 8, 128, 1, 0.2)


def test_both_arms_use_the_same_config_keys():
    sys.path.insert(0, ROOT)
    import bench
    w = bench.make_workload("cfg1", 4, 0)
    ours = bench.method_config(w, 1, 0, 0, False)
    assert ours == bench.method_config(w)
    assert isinstance(ours["layers"], int) and ours["tidal_kv"] == "bf16" and ours["score_scope"] == "per layer"
    assert bench.method_config(w, 3, 1, 1, True)["layer_issue"] == "all_layers_together"
