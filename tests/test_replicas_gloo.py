"""The N > 1 path of the bench ("replicas only"): two CPU ranks over gloo run the host-side logic that
the GPU ranks run over NCCL - rendezvous from the launcher's environment, the barrier on both sides of
the timed region, the max-over-ranks step time and the whole-job figure made from it."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_PROGRAM = r"""
import json, sys, time
sys.path.insert(0, {root!r})
import torch
from paper_2609_05255_b200 import replicas
rank, world, local = replicas.rank_env()
dist = replicas.init_process_group("gloo", world)
dev = torch.device("cpu")
replicas.barrier(dist)
t0 = time.perf_counter()
time.sleep(0.05 * (rank + 1))                 # rank 1 is the slow one
mine = (time.perf_counter() - t0) * 1e3
replicas.barrier(dist)
slowest = replicas.max_over_ranks(mine, dist, dev)
total = replicas.sum_over_ranks(1000 + rank, dist, dev)
print(json.dumps(dict(rank=rank, world=world, local=local, mine=mine, slowest=slowest, total=total,
                      value=replicas.job_ms_per_iteration(slowest, 1, world))))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(rank, world, port, argv):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), GLOO_SOCKET_IFNAME="lo")
    return subprocess.Popen([sys.executable] + argv, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)


def test_two_gloo_ranks_agree_on_the_slowest_time():
    port = _free_port()
    procs = [_launch(r, 2, port, ["-c", RANK_PROGRAM.format(root=ROOT)]) for r in range(2)]
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert [d["rank"] for d in outs] == [0, 1] and all(d["world"] == 2 for d in outs)
    assert outs[0]["slowest"] == outs[1]["slowest"] == max(d["mine"] for d in outs)
    assert outs[1]["mine"] > outs[0]["mine"]
    assert outs[0]["total"] == outs[1]["total"] == 2001
    # two replicas finish two iterations in the slowest rank's time
    assert outs[0]["value"] == outs[0]["slowest"] / 2


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2609_05255_b200 import replicas
    assert replicas.init_process_group("gloo", 1) is None
    replicas.barrier(None)
    assert replicas.max_over_ranks(3.5, None, None) == 3.5
    assert replicas.sum_over_ranks(2, None, None) == 2.0
    assert replicas.job_ms_per_iteration(12.0, 1, 4) == 3.0


def test_reference_arm_runs_on_rank_zero_only():
    """Under a multi-rank launch every rank but 0 leaves the reference arm at once, printing nothing."""
    p = _launch(1, 2, _free_port(), [os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                                     "--steps", "1", "--warmup", "0"])
    o, e = p.communicate(timeout=120)
    assert p.returncode == 0, e[-2000:]
    assert o.strip() == ""
