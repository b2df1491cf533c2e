"""The N>1 benchmark plumbing on CPU: two gloo ranks, max-over-ranks time, summed units."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    from paper_2512_00956_b200 import dist as D
    rank, local, world = D.init(backend="gloo")
    D.barrier()
    rate, t = D.whole_job_rate(units_this_rank=100.0 * (rank + 1), seconds_this_rank=1.0 + rank)
    assert world == 2 and abs(t - 2.0) < 1e-12 and abs(rate - 150.0) < 1e-9, (rate, t)
    assert D.max_over_ranks(float(rank)) == 1.0
    D.barrier(); D.shutdown()
    print("rank", rank, "ok")
""") % ROOT


def test_two_rank_gloo_aggregation(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29533", CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "ok" in out
