"""The N > 1 path of the benchmark (independent replicas; ranks meet only at a
barrier and for the maximum of their timings), on two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2608_26965_b200 import replicas
    rank, local, size = replicas.world()
    assert replicas.init("gloo")
    replicas.barrier()
    # rank r pretends its replica took 10 + 5 r ms for 100 units
    agg = replicas.aggregate_throughput(100.0, 10.0 + 5.0 * rank)
    replicas.barrier()
    print(json.dumps({"rank": rank, "size": size, **agg}))
    replicas.shutdown()
""") % ROOT


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(out.strip().splitlines()[-1])
    import json
    res = [json.loads(o) for o in outs]
    for r in res:
        assert r["size"] == 2 and r["n"] == 2
        assert abs(r["ms"] - 15.0) < 1e-9                      # the slower rank
        assert abs(r["value"] - 2 * 100.0 / 15e-3) < 1e-6      # both ranks' units over that time


def test_single_process_needs_no_group():
    from paper_2608_26965_b200 import replicas
    env_backup = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        assert replicas.init("gloo") is False
        assert replicas.max_over_ranks(3.5) == 3.5
        assert replicas.aggregate_throughput(10.0, 2.0)["value"] == 10.0 / 2e-3
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v
