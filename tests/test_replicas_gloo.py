"""The several-GPU path of bench.py is "replicas only": no data-path collective, a barrier and a
maximum over ranks around the timed region.  Checked here with two gloo processes on the CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    from workloads import replicas
    rank, local_rank, world = replicas.dist_env()
    dist.init_process_group("gloo")
    ms_local = 2.0 + 3.0 * rank                       # rank 1 is the slow replica
    dist.barrier()
    ms = replicas.max_over_ranks(ms_local, world)
    value = replicas.job_throughput(1024, ms, world)
    seed = replicas.replica_seed(1002, rank)
    print(json.dumps({{"rank": rank, "local_rank": local_rank, "world": world, "ms": ms, "value": value, "seed": seed}}))
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_report_the_slowest_time_and_the_summed_throughput(tmp_path):
    import json
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert [d["world"] for d in outs] == [2, 2] and [d["local_rank"] for d in outs] == [0, 1]
    assert outs[0]["ms"] == outs[1]["ms"] == 5.0                 # the slowest replica's time, on every rank
    assert outs[0]["value"] == 2 * 1024 / 5e-3                   # work of both replicas over that time
    assert outs[0]["seed"] != outs[1]["seed"]                    # replicas draw different inputs


def test_single_process_defaults():
    from workloads import replicas
    env = {k: os.environ.pop(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE") if k in os.environ}
    try:
        assert replicas.dist_env() == (0, 0, 1)
        assert replicas.max_over_ranks(3.5, 1) == 3.5
        assert replicas.job_throughput(1024, 1.0, 1) == 1024 / 1e-3
    finally:
        os.environ.update(env)
