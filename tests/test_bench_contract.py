"""The reference arm of bench.py runs on the CPU: its JSON line must carry the keys the contract names."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "llama7b_attn_4096x4096_s50_a50"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 1 and d["steps"] == 1
    for key in ("metric", "value", "unit", "ms_per_step", "higher_is_better", "scaling", "vs_baseline", "dtype", "data",
                "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["config"]["workload"] and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_format_study_matches_the_closed_form():
    """Section 3.2: a stored entry costs 2.5 bytes against 2 dense, and a gap of more than 15 rows costs one
    padding entry per 16 rows.  On Bernoulli masks of density d = 1 - s that is 1.25 * d * (1 + rho) of the dense
    size with rho = s^16 / (1 - s^16); the host encoder's entry counts must land on it (sampling noise only)."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--sweep", "format"], capture_output=True,
                         text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads([l for l in out.stdout.splitlines() if l.strip()][-1])
    assert d["sweep"] == "format" and len(d["points"]) >= 9
    for pt in d["points"]:
        s = pt["weight_sparsity"]
        want = 1.25 * pt["realised_density"] * (1.0 + s ** 16 / (1.0 - s ** 16))
        assert abs(pt["column"]["entries_over_dense"] - want) < 0.004 * max(want, 0.25), pt
        # the lane-tile image pays for headers and for filling each lane's last group of 8
        assert pt["lane_tile"]["image_over_dense"] > pt["lane_tile"]["entries_over_dense"]
    half = [pt for pt in d["points"] if pt["weight_sparsity"] == 0.5][0]
    assert abs(half["column"]["entries_over_dense"] - 0.625) < 0.002          # "about 63 %" at 50 % sparsity
    # other run widths: the library's entry counts sit on the closed form, width 4 is the encoder's own count, and
    # 4 bits are the smallest format in the range the paper prunes to (70 - 80 %), 3 bits at 50 - 60 %
    for pt in d["points"]:
        for n, v in pt["run_width"].items():
            # (the rows after a column's last kept row store nothing, which the closed form ignores: up to half a
            # per cent fewer padding entries at 2 bits and 95 % sparsity with 4096 rows)
            assert abs(v["entries_over_dense"] - v["closed_form"]) < 0.008 * max(v["closed_form"], 0.25), (pt, n)
        assert abs(pt["run_width"]["4"]["entries_over_dense"] - pt["column"]["entries_over_dense"]) < 1e-12
    best = {pt["weight_sparsity"]: pt["best_run_width"] for pt in d["points"]}
    assert best[0.7] == "4" and best[0.8] == "4" and best[0.5] == "3" and best[0.3] == "2" and best[0.95] == "6"
