"""The reference arm of the benchmark (the CPU oracle timed on the host cores) runs without a GPU: its JSON line must
carry the contract's keys, the metric and unit of the GPU arm, and a `config` that names the same workload."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags, env=None):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", *flags], cwd=ROOT,
                       capture_output=True, text=True, timeout=600, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    return r.stdout.strip()


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    out = _run("--config", "1", "--steps", "2", "--warmup", "1")
    assert len(out.splitlines()) == 1
    d = json.loads(out)
    assert d["impl"] == "reference" and d["metric"].startswith("routed tokens/sec") and d["unit"] == "tokens/s"
    for key in ("value", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline", "dtype",
                "data", "config", "cpu_baseline", "e2e", "sample_tokens_per_step"):
        assert key in d, key
    assert d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and d["ms_per_step"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    # the workload is named by the same keys the GPU arm prints (no key of the sample inside `config`)
    cfg = d["config"]
    assert cfg["T"] == 4096 and cfg["H"] == 1024 and cfg["E"] == 8 and "sample_tokens_per_step" not in cfg
    assert d["sample_tokens_per_step"] == 4096          # the tiny configuration is timed whole


def test_reference_arm_other_ranks_print_nothing():
    assert _run("--config", "1", "--steps", "1", "--warmup", "0", env=dict(os.environ, RANK="1", WORLD_SIZE="2")) == ""
