"""The benchmark's command-line contract, as far as it can be checked without a GPU: the reference
arm (the oracle timed on the host cores) prints one JSON line with the agreed keys, and the product
arm refuses to run without a device instead of falling back to anything."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                          timeout=600, env=env, cwd=ROOT)


def test_reference_arm_prints_one_json_line_with_the_agreed_keys():
    r = run_bench("--impl", "reference", "--workload", "c1", "--steps", "2", "--warmup", "1")
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference"
    assert d["metric"] == "denoise-step attention us/layer" and d["unit"] == "us/layer-step"
    assert d["higher_is_better"] is False and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["n_gpus"] == 1 and d["steps"] == 2 and d["warmup"] >= 3 and d["data"] == "synthetic"
    assert d["value"] > 0 and abs(d["ms_per_step"] * 1e3 - d["value"]) < 1e-6 * d["value"]
    assert d["config"]["workload"].startswith("c1")
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["gpu_launches"] == 0


def test_product_arm_needs_a_gpu():
    r = run_bench("--workload", "c1", "--steps", "4", "--warmup", "3")
    assert r.returncode != 0
    assert not [ln for ln in r.stdout.splitlines() if ln.startswith("{")]      # no result line of any kind


def test_timed_walk_always_holds_losa_steps_in_block_proportion():
    """The K timed layer-steps are cut into ceil(K / T) dense first steps and the rest LoSA steps,
    whatever K the caller asks for: the walk of the driver's short run (20 steps), of the default
    run (4 blocks of 36 layers) and of a single-layer run."""
    sys.path.insert(0, ROOT)
    import bench
    for K, T, L, want_layers in ((20, 8, 36, 3), (1152, 8, 36, 36), (16, 8, 1, 1), (7, 16, 1, 1), (100, 8, 36, 13)):
        L_eff, sweeps = bench.schedule(K, T, L)
        assert L_eff == want_layers
        assert sum(n for _, _, n in sweeps) == K
        dense = sum(n for _, t, n in sweeps if t == 0)
        assert dense == -(-K // T) and dense < K
        assert all(n == L_eff for _, _, n in sweeps[:-1]) and 1 <= sweeps[-1][2] <= L_eff
        # model order from a block boundary: consecutive sweeps are consecutive denoising steps
        assert [(b * T + t) for b, t, _ in sweeps] == list(range(len(sweeps)))
    L_eff, sweeps = bench.schedule(20, 8, 36)
    assert [(t, n) for _, t, n in sweeps] == [(0, 3), (1, 3), (2, 3), (3, 3), (4, 3), (5, 3), (6, 2)]


def test_both_arms_name_the_workload_identically():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2604_12056_b200 import workloads as wl
    src = open(os.path.join(ROOT, "bench.py")).read()
    assert src.count("workload_name(") == 3          # the definition and one use per arm, nothing appended to the reference arm's
    assert "36 layer(s)" in bench.workload_name(wl.config("c5"), 36)
