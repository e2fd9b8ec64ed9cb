"""The benchmark's reference arm (the float64 oracle timed on the host cores) needs no GPU:
run it on the tiny workload and check the JSON line it prints, and the byte model behind
`value`."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "c1", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 1 and d["steps"] == 1
    assert d["unit"] == "GB/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and d["ms_per_step"] > 0
    assert d["config"]["workload"] == "c1"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == dict(value=d["value"], unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0)


def test_algorithmic_bytes_of_the_headline_workload():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_33746_b200.workload import named_config
    cfg = named_config("c3_b8_r1")
    b = bench.algorithmic_bytes(cfg, list(cfg.seq_lens), cfg.budget_ppm)
    assert b["total"] == b["lut"] + b["scan"] + b["select"] + b["attend"]
    units = cfg.n_kv_heads * sum(cfg.seq_lens)
    # per (token, KV head): 32 code bytes + norm 4 + list id 2 + one fp32 score per query head
    # of the group written by the scan ...
    assert b["scan"] >= units * (32 + 4 + 2 + 4 * cfg.group)
    # ... and read once by the top-k
    assert b["select"] >= units * 4 * cfg.group
    # about 104 B per unit in all, a fifth of what dense bf16 attention reads (512 B)
    assert 95 <= b["total"] / units <= 115
    assert bench.dense_attention_bytes(cfg, list(cfg.seq_lens)) == units * 512
