"""The N>1 plumbing on CPU: two gloo ranks, max-over-ranks timing, per-rank token seeds."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent("""
    import sys, json
    sys.path.insert(0, %r)
    from paper_2511_17885_b200 import dist as D
    rank, local, world = D.init("gloo")
    D.barrier()
    thr, t = D.aggregate_throughput(100.0 * (rank + 1), 1.0 + rank)
    seeds = D.token_seed_for_rank(5, rank)
    if rank == 0:
        print(json.dumps({"thr": thr, "t": t, "world": world, "seed": seeds}))
    D.barrier()
    D.shutdown()
""" % ROOT)


def test_two_gloo_ranks_aggregate(tmp_path):
    f = tmp_path / "w.py"
    f.write_text(SCRIPT)
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                        "--master-addr", "127.0.0.1", "--master-port", "29533", str(f)],
                       capture_output=True, text=True, timeout=180)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2 and abs(d["t"] - 2.0) < 1e-12 and abs(d["thr"] - 150.0) < 1e-9


def test_rank_seeds_differ():
    from paper_2511_17885_b200 import dist as D
    assert len({D.token_seed_for_rank(3, r) for r in range(8)}) == 8


def test_bench_reference_arm_runs_on_cpu():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "C0"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    d = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert d["impl"] == "reference" and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
