"""Host-side checks of bench.py that need no GPU: the workload table against the byte counts
the hot-path definition gives, the spread helper, and the reference arm end to end (it times
the CPU oracle, so it runs anywhere)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def load_bench():
    sys.path.insert(0, ROOT)
    import bench
    return bench


def test_workload_table_matches_the_definition_of_the_bytes():
    bench = load_bench()
    assert set(bench.DEFAULT_STEPS) == set(bench.WORKLOADS)
    for key, w in bench.WORKLOADS.items():
        if w.get("env") == "policy":
            continue
        if w.get("env") == "cartpole":
            want = 16 + 4 + 1 + 48.0 / w["T"]                  # obs + reward + done, 24-byte state in and out
        elif w["obs_mode"] == 1:
            want = 84 * 84 + 4 + 1 + 64.0 / w["T"]             # one frame + reward + done, 32-byte state in and out
        elif key == "step4096":
            want = 1 + 32 + 32 + 24 + 4 + 1                    # action, state in, state out, obs, reward, done
        else:
            want = 24 + 4 + 1 + 64.0 / w["T"]
        assert abs(w["bytes"] - want) < 1e-9, key
        assert w["n"] >= 1 and w["T"] >= 1 and w["frameskip"] in (1, 4)
    assert bench.WORKLOADS["rollout65k"]["n"] == 65536 and bench.WORKLOADS["rollout65k"]["T"] == 128
    assert bench.WORKLOADS["rollout1m"]["mode"] == 1 and bench.WORKLOADS["pixels16k"]["frameskip"] == 4


def test_spread():
    bench = load_bench()
    s = bench.spread([2.0, 4.0, 4.0, 4.0, 5.0, 5.0, 7.0, 9.0])
    assert s["n"] == 8 and s["mean"] == 5.0 and s["std"] == 2.0 and s["cv"] == 0.4
    assert bench.spread([3.0])["std"] == 0.0


def test_reference_arm_prints_one_line_of_the_contract():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, check=True, cwd=ROOT)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["higher_is_better"] is True and line["steps"] == 2
    assert line["unit"] == "env-steps/s" and line["value"] > 1e6
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0,
                           "d2h_bytes_per_step": 0}
    assert "65536" in line["config"]["workload"]
    # the other ranks of a multi-rank launch print nothing and exit 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, check=True, cwd=ROOT, env=env)
    assert out.stdout.strip() == ""
