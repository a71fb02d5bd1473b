"""The multi-rank plumbing of the benchmark on CPU: two gloo ranks, barrier + MAX of the times + SUM of the units."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys, time
    sys.path.insert(0, %r)
    from paper_2605_13915_b200.ranks import Ranks
    r = Ranks("gloo")
    assert r.world == 2
    if r.rank == 1:
        time.sleep(0.3)          # a slow rank: the barrier must hold the fast one back
    t0 = time.time()
    r.barrier()
    waited = time.time() - t0
    ms = 10.0 if r.rank == 0 else 25.0
    thr, job_ms = r.job_throughput(1000.0 * (r.rank + 1), ms)
    out = {"rank": r.rank, "root": r.is_root, "waited": waited, "max": r.max_over_ranks(ms),
           "sum": r.sum_over_ranks(ms), "thr": thr, "job_ms": job_ms}
    r.barrier()
    r.close()
    print(json.dumps(out))
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_combine_times_and_units():
    import json
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=120)
        assert p.returncode == 0, se[-2000:]
        outs.append(json.loads(so.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["root"] and not outs[1]["root"]
    assert outs[0]["waited"] > 0.2                     # rank 0 waited at the barrier for the slow rank
    for o in outs:
        assert o["max"] == 25.0 and o["sum"] == 35.0
        assert o["job_ms"] == 25.0
        assert abs(o["thr"] - 3000.0 / 25e-3) < 1e-6   # all units over the slowest rank's time


def test_single_rank_needs_no_process_group(monkeypatch):
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    sys.path.insert(0, ROOT)
    from paper_2605_13915_b200.ranks import Ranks
    r = Ranks("gloo")
    assert r.world == 1 and r.is_root
    r.barrier()
    assert r.max_over_ranks(3.5) == 3.5
    thr, ms = r.job_throughput(70.0, 3.5)
    assert ms == 3.5 and abs(thr - 20000.0) < 1e-9


def test_bench_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher re-executes itself under torch.distributed.run with two ranks.  The CPU
    arm (--impl reference) exercises that path here: rank 0 prints the one JSON line, rank 1 exits 0 without work."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                       # one line for the whole job
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["value"] > 0
