"""The N > 1 path of the benchmark is N independent replicas; what the processes share is the
measurement protocol (barrier, slowest time, summed work).  Two gloo ranks on CPU exercise it."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys, json
    sys.path.insert(0, %r)
    from paper_2203_17063_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    rep.barrier()
    ms = 10.0 if rep.rank == 0 else 25.0            # the second replica is slower
    rate, slowest = rep.whole_job_rate(1000.0 * (rep.rank + 1), ms)
    rep.barrier()
    print(json.dumps({"rank": rep.rank, "world": rep.world, "rate": rate, "slowest": slowest,
                      "max": rep.max(rep.rank), "sum": rep.sum(rep.rank + 1)}))
    rep.close()
""") % ROOT


def test_two_replicas_report_sum_over_slowest():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(eval(out.strip().splitlines()[-1].replace("true", "True")))
    for o in outs:
        assert o["world"] == 2
        assert o["slowest"] == 25.0                       # max over ranks
        assert abs(o["rate"] - 3000.0 / 25e-3) < 1e-6     # all replicas' work over the slowest time
        assert o["max"] == 1.0 and o["sum"] == 3.0


def test_single_process_is_a_no_op():
    sys.path.insert(0, ROOT)
    from paper_2203_17063_b200.replicas import Replicas

    env_backup = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        rep = Replicas()
        assert (rep.rank, rep.world, rep.active) == (0, 1, False)
        rep.barrier()
        assert rep.whole_job_rate(500.0, 10.0) == (50000.0, 10.0)
        rep.close()
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v
