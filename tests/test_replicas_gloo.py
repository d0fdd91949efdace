"""The N > 1 path of the benchmark is "replicas only": no data-path collective, only barrier + max-over-ranks
timing and a sum of the work.  Covered here with two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    from paper_2411_09317_b200.replicas import Replicas
    r = Replicas("gloo")
    assert r.world == 2
    r.barrier()
    ms = 10.0 if r.rank == 0 else 25.0          # rank 1 is the slow replica
    units = 100.0 * (r.rank + 1)                # rank 0 did 100 units, rank 1 did 200
    thr, worst = r.aggregate_throughput(units, ms)
    assert worst == 25.0, worst
    assert abs(thr - 300.0 / 0.025) < 1e-6, thr
    assert r.max_over_ranks(float(r.rank)) == 1.0 and r.sum_over_ranks(1.0) == 2.0
    r.barrier()
    if r.rank == 0:
        print(json.dumps({"ok": True, "throughput": thr}))
    r.close()
""") % ROOT


def test_two_gloo_ranks_aggregate_by_max_time_and_sum_of_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29653", str(script)],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    assert '"ok": true' in out.stdout


def test_single_rank_is_identity():
    from paper_2411_09317_b200.replicas import Replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    r = Replicas("gloo")
    thr, ms = r.aggregate_throughput(50.0, 5.0)
    assert (thr, ms) == (50.0 / 0.005, 5.0)
