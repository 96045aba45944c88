"""The multi-GPU path of the benchmark is N independent replicas; its host logic (rank-specific
batches, MAX-over-ranks timing, whole-job rate) is exercised here as two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import numpy as np
import torch.distributed as dist
from paper_2504_01337_b200 import inputs as G
from paper_2504_01337_b200 import replicas as R
rank, local, world = R.env_rank()
dist.init_process_group("gloo", rank=rank, world_size=world)
wl = G.Workload("t", N=64, d=32, E=8, I=16, K=2, T=3, P=2, seed=5)
wr = R.rank_workload(wl, rank)
x = G.hidden(wr)
wg, _ = G.gate_weights(wl)
my_ms = 2.0 + 3.0 * rank            # rank 1 is the slow one
R.barrier()
worst = R.max_over_ranks(my_ms)
out = dict(rank=rank, world=world, worst=worst, rate=R.whole_job_rate(wl.N, world, worst),
           x_sum=float(np.abs(x).sum()), wg_sum=float(np.abs(wg).sum()))
print("RESULT " + json.dumps(out), flush=True)
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_like_the_benchmark(tmp_path):
    import json
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    res = {}
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        line = [ln for ln in out.splitlines() if ln.startswith("RESULT ")][0]
        d = json.loads(line[7:])
        res[d["rank"]] = d
    assert res[0]["world"] == res[1]["world"] == 2
    # both ranks agree on the slowest rank's time, and the job rate counts both ranks' tokens
    assert res[0]["worst"] == res[1]["worst"] == 5.0
    assert np.isclose(res[0]["rate"], 2 * 64 / 5e-3)
    # same parameters on both ranks, different batches
    assert res[0]["wg_sum"] == res[1]["wg_sum"]
    assert res[0]["x_sum"] != res[1]["x_sum"]


def test_single_process_is_identity():
    from paper_2504_01337_b200 import replicas as R
    assert R.max_over_ranks(3.5) == 3.5
    assert R.whole_job_rate(100, 1, 10.0) == 100 / 10e-3
    R.barrier()
