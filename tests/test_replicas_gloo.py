"""The multi-GPU path is N independent replicas: the only cross-rank steps are a barrier and
the maximum of the ranks' elapsed times.  Both are exercised here with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, sys.argv[1])
    import torch.distributed as dist
    from paper_2410_09615_b200 import replicas
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    assert replicas.world_size() == world == 2
    replicas.barrier()
    elapsed_ms = 10.0 + 5.0 * rank            # rank 1 is the slow replica
    worst = replicas.max_over_ranks(elapsed_ms)
    value = replicas.whole_job_us_per_call(worst / 4, 14, world)
    replicas.barrier()
    if rank == 0:
        print(json.dumps({"worst_ms": worst, "value": value, "n_gpus": world}))
    dist.destroy_process_group()
""")


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_take_the_slowest_time_and_only_rank0_prints(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    import json
    line = json.loads(outs[0][0].strip())
    assert outs[1][0].strip() == ""                       # rank 1 prints nothing
    assert line["worst_ms"] == 15.0                       # maximum over ranks
    # 15 ms over 4 steps of 14 calls on each of 2 replicas
    assert abs(line["value"] - 1e3 * (15.0 / 4) / (14 * 2)) < 1e-9


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    from paper_2410_09615_b200 import replicas
    assert replicas.world_size() == 1
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_us_per_call(0.21, 14, 1) == 1e3 * 0.21 / 14
