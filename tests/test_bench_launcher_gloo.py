"""`python bench.py --gpus 2` starts its own ranks and runs the slab-sharded layer (Algorithm 1) across them.
Here, without GPUs, the same launcher runs two CPU ranks over gloo with the test stand-in for the CUDA steps
(tests/gloo_ops.py); what is checked is the launch, the rendezvous, the exchange and the printed line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_gpus_2_spawns_two_ranks_and_prints_one_line():
    env = dict(os.environ)
    env["PYTHONPATH"] = os.path.join(ROOT, "tests") + os.pathsep + env.get("PYTHONPATH", "")
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo",
                          "--ops-module", "gloo_ops:make_ops", "--config", "cfg1_2d_64", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, env=env, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["scaling"] == "strong" and line["steps"] == 2
    assert line["backend"] == "gloo" and line["data_path"].startswith("stand-in")
    assert line["config"]["slab_per_rank"] == [32, 64] and line["config"]["modes_per_rank"] == 64
    assert set(line["phases_ms"]) >= {"F_local", "all_reduce_X", "mix", "all_gather_Y", "I_local"}
    assert line["collective_payload_bytes_per_step"]["all_reduce"] == 8 * 1 * 128 * (4 + 4)
    assert line["ms_per_step"] > 0 and line["value"] > 0


def test_bench_refuses_the_gloo_backend_without_a_stand_in():
    env = dict(os.environ)
    env.update(WORLD_SIZE="2", RANK="0", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo",
                          "--config", "cfg1_2d_64"], capture_output=True, text=True, env=env, timeout=300, cwd=ROOT)
    assert res.returncode != 0 and "no CPU path" in res.stderr
