"""bench.py's contract that can be checked without a GPU: the reference arm prints one JSON line with the agreed keys,
non-zero ranks stay silent, and the recorded profiler traffic belongs to the step kernel as it stands in the tree."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, env=None):
    e = dict(os.environ)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, capture_output=True, text=True,
                          env=e, cwd=ROOT, timeout=600)


def test_reference_arm_prints_one_json_line():
    r = _run(["--impl", "reference", "--gpus", "1", "--steps", "6", "--warmup", "3"])
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "replica_param_updates_per_s" and d["unit"] == "param-updates/s"
    assert d["higher_is_better"] is True and d["steps"] == 6 and d["warmup"] == 3 and d["n_gpus"] == 1
    assert d["value"] > 0 and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in d["config"] and "model" not in d["config"]


def test_reference_arm_is_silent_on_other_ranks():
    r = _run(["--impl", "reference", "--gpus", "2", "--steps", "3", "--warmup", "3"], env={"RANK": "1", "WORLD_SIZE": "2"})
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_recorded_traffic_matches_the_kernel_source():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.step_source_hash() == bench.NCU_TRAFFIC["step_source_sha256"], \
        "the step kernel changed since the ncu capture: re-capture and update NCU_TRAFFIC (bench.py reports null meanwhile)"
    w_adamw = type("W", (), {"opt": "adamw", "K": 16})
    w_sgdm = type("W", (), {"opt": "sgdm", "K": 16})
    assert bench.step_bytes_per_update(w_adamw) == 24.5 and bench.step_bytes_per_update(w_sgdm) == 16.5
    for opt, algo in (("adamw", 24.5), ("sgdm", 16.5)):
        measured = bench.NCU_TRAFFIC["bytes_per_update"][opt]
        assert 0.95 * algo <= measured <= 1.02 * algo     # no re-reads: traffic ~ algorithmic bytes


def test_recorded_instruction_counts_match_the_resident_kernel_source():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.resident_source_hash() == bench.NCU_RESIDENT_INSTR["source_sha256"], \
        "the resident-steps kernel changed since the ncu capture: re-capture and update NCU_RESIDENT_INSTR"
    # the ALU peak: 148 SMs x 4 schedulers x 32 lanes per clock
    assert bench.SM_COUNT * bench.LANES_PER_SM_CLK == 18944
    assert 35 < bench.NCU_RESIDENT_INSTR["adamw"] < bench.NCU_RESIDENT_INSTR["sgdm"] < 45       # issued (packed fp32)
    assert 45 < bench.NCU_RESIDENT_INSTR["scalar_equivalent"]["sgdm"] < bench.NCU_RESIDENT_INSTR["scalar_equivalent"]["adamw"] < 55
