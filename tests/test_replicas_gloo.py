"""The multi-GPU plumbing of bench.py on CPU: two gloo ranks.  The decode path has no exchange step
(one GPU per replica, no sharding), so all that crosses ranks is the timing protocol: barrier, the
maximum of the measured time over the ranks, and the whole-job throughput derived from it."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_PROGRAM = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import bench
    rep = bench.Replicas("gloo")
    assert rep.world == 2 and rep.rank == int(os.environ["RANK"])
    seeds = rep.seed_for(1001)
    rep.barrier()
    local_ms = 2.0 if rep.rank == 0 else 5.0          # rank 1 is the slow one
    worst = rep.max_over_ranks(local_ms)
    value = rep.job_value(8, worst)                   # 8 sequences per replica
    rep.barrier()
    print(json.dumps({"rank": rep.rank, "seed": seeds, "worst": worst, "value": value}))
    rep.close()
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_agree_on_the_slowest_rank_and_the_job_throughput():
    import json
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", RANK_PROGRAM], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    assert outs[0]["seed"] != outs[1]["seed"]                  # each replica draws its own batch
    for o in outs:
        assert o["worst"] == 5.0                               # the maximum over ranks, on every rank
        assert abs(o["value"] - 2 * 8 / 5.0e-3) < 1e-6         # both replicas' sequences over the slowest time


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    env_backup = {k: os.environ.pop(k, None) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    try:
        rep = bench.Replicas("gloo")
        assert rep.world == 1 and rep.dist is None
        assert rep.max_over_ranks(3.5) == 3.5 and rep.job_value(8, 2.0) == 4000.0
        rep.barrier(); rep.close()
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v
