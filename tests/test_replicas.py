"""The N > 1 path of the benchmark on CPU: two gloo ranks go through the replica plumbing (barrier, MAX over
ranks of the timed region, whole-job throughput) and through `bench.py --impl reference`, where rank 0 alone
prints the line."""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def torchrun(args, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port())] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_take_the_max_and_sum_the_work(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import sys
        sys.path.insert(0, {ROOT!r})
        from paper_2601_21109_b200 import replicas
        rank, local_rank, world = replicas.world_from_env()
        replicas.init("gloo", local_rank, world)
        replicas.barrier(world, cuda=False)
        mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        slowest = replicas.max_over_ranks(mine, world, device="cpu")
        assert slowest == 15.0, slowest
        value = replicas.job_throughput(2048, 7, world, slowest)
        assert abs(value - 2048 * 7 * 2 / 15e-3) < 1e-6
        replicas.barrier(world, cuda=False)
        if rank == 0:
            print("RESULT", world, slowest, value)
        replicas.finish(world)
    """))
    r = torchrun([str(script)])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("RESULT")]
    assert len(lines) == 1 and lines[0].split()[1] == "2"


def test_single_process_is_a_world_of_one():
    from paper_2601_21109_b200 import replicas
    env = {k: os.environ.pop(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE") if k in os.environ}
    try:
        assert replicas.world_from_env() == (0, 0, 1)
        assert replicas.max_over_ranks(3.5, 1) == 3.5
        assert replicas.job_throughput(100, 2, 1, 10.0) == 100 * 2 / 10e-3
    finally:
        os.environ.update(env)


def test_reference_arm_under_two_ranks_prints_one_line():
    r = torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "cfg1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2


def test_bench_starts_its_own_ranks_when_no_launcher_is_around():
    # plain `python bench.py --gpus 2`: the script re-launches itself as two ranks; one line, n_gpus = 2
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    env["OMP_NUM_THREADS"] = "2"
    r = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                        "--workload", "cfg1"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["impl"] == "reference"
    assert line["config"]["parallelism"] == "replicas only"
