"""The N > 1 path of bench.py on CPU: two gloo ranks.  Sequences are independent, so ranks run replicas with
their own seeds and no data-path collective; the only exchanges are the barrier and the max-over-ranks time."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, n=2):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_two_ranks_get_distinct_replicas_and_the_slowest_time(tmp_path):
    r = _torchrun([os.path.join(ROOT, "tests", "_rank_worker.py"), str(tmp_path)])
    assert r.returncode == 0, r.stderr[-2000:]
    out = [json.load(open(tmp_path / f"rank{k}.json")) for k in range(2)]
    assert [o["rank"] for o in out] == [0, 1] and all(o["world"] == 2 for o in out)
    assert out[0]["seed"] != out[1]["seed"] and out[0]["ids"] != out[1]["ids"]      # own replica per rank
    assert out[0]["max_ms"] == out[1]["max_ms"] == 15.0                               # max over ranks, on every rank


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--workload", "c1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` started as a plain command (no WORLD_SIZE in the environment) launches two ranks
    itself; with the gloo backend the launch path runs here without a GPU: two ranks meet, agree on the slowest
    rank's time, and rank 0 alone prints the line, with n_gpus 2 and a global batch of two replicas."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env.update(CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo", "--workload", "c2"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["launch_check"] and d["n_gpus"] == 2 and d["slowest_ms"] == 2.0
    assert d["config"]["global_batch"] == 2 * 1
