"""Host-side plumbing for several GPUs, exercised with two gloo ranks on the CPU.

The path has no data-path collective (sequences are independent, every rank runs its own
replicas), so what is checked is the rendezvous, the partition of sequence ids, the barrier and
the max-over-ranks / whole-job arithmetic that the benchmark reports."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2601_07353_b200 import dist
    info = dist.env_rank_info()
    dist.init(info, "gloo")
    dist.barrier(info)
    ids = dist.rank_sequence_ids(info, sets=3, batch=4)
    slow = dist.max_over_ranks(1.0 + info.rank, info)          # rank 1 is the slow one
    total = dist.sum_over_ranks(10.0, info)
    rate = dist.whole_job_rate(100, slow, info)
    dist.barrier(info)
    print(json.dumps(dict(rank=info.rank, world=info.world, main=info.is_main, ids=ids, slow=slow, total=total, rate=rate)))
    dist.shutdown()
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_gloo_ranks_partition_and_reduce():
    import json
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert [o["main"] for o in outs] == [True, False]
    flat = [i for o in outs for s in o["ids"] for i in s]
    assert sorted(flat) == list(range(2 * 3 * 4))              # ranks and sets never share a sequence id
    assert outs[0]["ids"][0] == [0, 1, 2, 3] and outs[1]["ids"][0] == [12, 13, 14, 15]
    for o in outs:
        assert o["slow"] == 2.0 and o["total"] == 20.0
        assert o["rate"] == 100 * 2 / 2.0                        # units of all ranks over the slowest rank's time


def test_single_process_needs_no_group():
    from paper_2601_07353_b200 import dist
    info = dist.RankInfo(0, 1, 0)
    dist.barrier(info)
    assert dist.max_over_ranks(3.5, info) == 3.5
    assert dist.whole_job_rate(10, 2.0, info) == 5.0
    assert dist.rank_sequence_ids(info, 2, 3) == [[0, 1, 2], [3, 4, 5]]


def test_reference_arm_runs_on_rank_zero_only():
    """`bench.py --impl reference` under a 2-rank launch: rank 1 exits 0 without printing."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
