"""Host-side checks of bench.py that need no GPU: the workload parser, the algorithmic byte count the
roofline uses, and the reference arm (the oracle on the host cores) printing one well-formed JSON line."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_workload_strings_and_algorithmic_bytes():
    from paper_2601_09212_b200 import workloads as W
    kw = bench.workload_kwargs("C3")
    assert (kw["B"], kw["gamma"], kw["V"], kw["top_k"], kw["cfg"]) == (64, 8, 16384, 1000, True) and kw["dtype"] == W.BF16
    # every stored logit once: 2 models x 2 arrays x B x gamma x V x 2 bytes, plus tokens, uniforms, schedule, outputs
    logits = 2 * 2 * 64 * 8 * 16384 * 2
    assert logits <= bench.algorithmic_bytes(kw) <= logits + 64 * 1024
    kw = bench.workload_kwargs("B=3,gamma=5,V=4100,dtype=fp32,top_k=7,cfg=1,cfg_scale=2.5,law=student3")
    assert kw == dict(rho=0.9, B=3, gamma=5, V=4100, dtype=W.F32, top_k=7, cfg=True, cfg_scale=2.5, law="student3")
    assert bench.algorithmic_bytes(kw) >= 2 * 2 * 3 * 5 * 4100 * 4
    with pytest.raises(SystemExit):
        bench.workload_kwargs("B=3,gamma=5")
    with pytest.raises(SystemExit):
        bench.workload_kwargs("B=3,gamma=5,V=64,colour=red")
    d = bench.describe("C4", bench.workload_kwargs("C4"), "s")
    assert d["workload"] == "C4" and d["logits"] == "bf16" and d["law"] == "student3" and d["top_k"] == 0


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                          "--workload", "B=4,gamma=4,V=2048,dtype=bf16,cfg=1,top_k=100"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "verified_draft_tokens_per_sec" and d["higher_is_better"] is True
    assert d["steps"] == 2 and d["warmup"] == 1 and d["value"] > 0 and d["n_gpus"] == 1
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"] and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("B=4") and d["config"]["top_k"] == 100 and d["vs_baseline"] is None
