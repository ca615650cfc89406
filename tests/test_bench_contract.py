"""CPU-only checks of the benchmark's reference arm (the fp64 oracle timed on the host cores) and of
how it behaves when launched as several ranks: rank 0 alone works and prints the JSON line, the
other ranks exit 0 without output."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_rank(rank, world):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", CUDA_VISIBLE_DEVICES="")
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", str(world),
                           "--workload", "cfg1", "--steps", "2", "--warmup", "1"],
                          env=env, capture_output=True, text=True, timeout=600)


def test_reference_arm_two_ranks():
    procs = [run_rank(r, 2) for r in range(2)]
    assert all(p.returncode == 0 for p in procs), [p.stderr[-500:] for p in procs]
    assert procs[1].stdout.strip() == ""
    line = json.loads(procs[0].stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["steps"] == 2
    assert line["unit"] == "us/step" and line["higher_is_better"] is False and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["cpu_baseline"]["value"] == line["value"] and line["cpu_baseline"]["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"] == "7b-layer-16k" and line["vs_baseline"] is None


def test_rank_plumbing_two_ranks_gloo():
    """Two CPU ranks over gloo: the job's time is the slowest rank's, the whole-job value divides by the replicas,
    and rank 0 alone prints."""
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29541",
                   CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py"), "--selftest-ranks"], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-500:] for o in outs]
    assert outs[1][0].strip() == ""
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line == {"max_ms": 20.0, "world": 2, "us_per_step": 20.0 / 5 * 1e3 / 2}
