"""World-size-2 CPU (gloo) checks of the multi-process plumbing bench.py uses: the path has no collective on its
data (replicas only), so what has to work across ranks is the barrier, the max over ranks of the timed interval,
and the rule that only rank 0 prints the result line."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["RIVER_REPO"])
import bench
rank, world = bench.dist_setup(int(os.environ["WORLD_SIZE"]))
bench.dist_barrier()
mx = bench.dist_max(10.0 + rank)          # slowest rank decides the timed interval
sm = bench.dist_sum(float(rank + 1))
bench.dist_barrier()
print(json.dumps({"rank": rank, "world": world, "max": mx, "sum": sm}), flush=True)
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(world, argv, extra_env=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RIVER_REPO=ROOT, CUDA_VISIBLE_DEVICES="",
                   OMP_NUM_THREADS="2")
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable] + argv, cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            out, err = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            for q in procs:
                q.kill()
            raise
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_barrier_max_sum_over_two_gloo_ranks():
    outs = _spawn(2, ["-c", WORKER])
    recs = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda r: r["rank"])
    assert [r["rank"] for r in recs] == [0, 1]
    for r in recs:
        assert r["world"] == 2
        assert r["max"] == 11.0      # max over ranks, seen by every rank
        assert r["sum"] == 3.0


def test_single_process_helpers_are_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.dist_max(3.5) == 3.5 and bench.dist_sum(2.0) == 2.0
    bench.dist_barrier()


def test_reference_arm_prints_one_line_from_rank_zero_only():
    outs = _spawn(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--workload", "tiny", "--steps", "2",
                      "--warmup", "3"])
    lines = [[l for l in o.splitlines() if l.startswith("{")] for o in outs]
    assert len(lines[0]) == 1 and len(lines[1]) == 0
    j = json.loads(lines[0][0])
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["cpu_baseline"]["kind"] == "oracle"
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["e2e"]["value"] == j["value"] > 0


def test_our_arm_fails_loudly_without_a_gpu():
    """The product path has no CPU fallback: without CUDA the bench must exit non-zero, not time something else."""
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, "bench.py", "--workload", "tiny", "--steps", "1"], cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=240)
    assert p.returncode != 0
    assert not [l for l in p.stdout.splitlines() if l.startswith("{")]
