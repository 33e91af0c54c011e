"""bench.py without a GPU: the reference arm (the oracle on the host cores) prints the agreed JSON
line, --gpus N plans one rank per GPU, and the byte accounting matches the stated formulas."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "1", "--workload", "dense150m"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "merged_params_per_sec" and d["unit"] == "params/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["gpu_launches"] == 0
    assert d["value"] > 0 and d["steps"] == 1 and d["config"]["workload"] == "dense150m"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "params/s", "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1"], capture_output=True, text=True,
                         timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_dry_launch_plans_one_rank_per_gpu():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "7",
                          "--dry-launch"], capture_output=True, text=True, timeout=120, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    plan = json.loads(out.stdout)
    assert [item["rank"] for item in plan] == [0, 1, 2, 3]
    ports = {item["env"]["MASTER_PORT"] for item in plan}
    assert len(ports) == 1 and 1024 < int(ports.pop()) < 65536
    for r, item in enumerate(plan):
        env = item["env"]
        assert env["RANK"] == env["LOCAL_RANK"] == str(r)
        assert env["WORLD_SIZE"] == env["LOCAL_WORLD_SIZE"] == "4" and env["MASTER_ADDR"] == "127.0.0.1"
        assert item["argv"][1].endswith("bench.py") and item["argv"][2:] == ["--gpus", "4", "--steps", "7"]


def test_spawned_ranks_run_with_their_environment(tmp_path):
    # the launcher itself, with a stand-in for the ranks' work: every rank of the reference arm but
    # rank 0 exits silently, rank 0 prints the line -- so one line comes back from N processes
    sys.path.insert(0, ROOT)
    import bench
    args = bench.parse_args(["--gpus", "3", "--impl", "reference", "--steps", "1", "--warmup", "0",
                             "--workload", "tiny"])
    script = tmp_path / "run.py"
    # (the launcher refuses to start more ranks than there are GPUs: none are needed for this arm)
    script.write_text("import sys\nsys.path.insert(0, %r)\nimport bench, torch\n"
                      "torch.cuda.device_count = lambda: 3\n"
                      "sys.exit(bench.spawn_ranks(bench.parse_args(%r), %r))\n"
                      % (ROOT, ["--gpus", "3"], ["--gpus", "3", "--impl", "reference", "--steps", "1",
                                                 "--warmup", "0", "--workload", "tiny"]))
    out = subprocess.run([sys.executable, str(script)], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 3 and args.gpus == 3


def test_byte_accounting_follows_the_stated_formulas():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2604_21428_b200 import synth
    w = synth.workload("scale500m")
    assert bench.participants(w, 0) == 24
    assert bench.algorithmic_bytes(w) == 500_000_000 * (24 * 2 + 16)
    assert bench.algorithmic_bytes(w, out_bf16=True) == 500_000_000 * (24 * 2 + 18)
    assert bench.algorithmic_bytes(w, "int4") == int(500_000_000 * (24 * (0.5 + 4 / 128) + 16))
    assert abs(bench.write_share(w) - 8 / 64) < 1e-12
    # radial-directional: three launches above 8 participants, two (through the Gram matrix) up to 8
    assert bench.algorithmic_bytes(w, "rda") == 500_000_000 * (2 * (24 * 2 + 4) + 24) and bench.rda_launches(w) == 3
    d6 = synth.workload("dense150m")
    assert bench.algorithmic_bytes(d6, "rda") == d6.total_params * (2 * 6 * 2 + 20) and bench.rda_launches(d6) == 2
    assert bench.algorithmic_bytes(d6, "rda", rda_three_pass=True) == d6.total_params * (2 * (6 * 2 + 4) + 24)
    t = synth.workload("tiny")
    assert bench.algorithmic_bytes(t) == (1 << 20) * (2 * 4 + 16)
    d = synth.workload("dense150m")
    assert [bench.participants(d, p) for p in range(d.P)] == [6] * 4
    # no interference: all reads at the read ceiling, all writes at the write ceiling
    assert abs(bench.blend_ceiling(7000.0, 7000.0, 0.3) - 7000.0) < 1e-9
    assert abs(bench.blend_ceiling(8000.0, 4000.0, 0.5) - 1 / (0.5 / 8000 + 0.5 / 4000)) < 1e-9
