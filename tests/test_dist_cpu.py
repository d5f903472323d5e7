"""The N>1 path of the benchmark (independent replicas, max-over-ranks timing) on CPU: two gloo ranks."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys
sys.path.insert(0, os.environ["PKV_ROOT"])
import numpy as np
import torch.distributed as dist
from paper_2609_39329_b200 import dist_util as du
from paper_2609_39329_b200 import inputs as gen
world, rank, local = du.env_ranks()
dist.init_process_group("gloo")
assert dist.get_world_size() == world == 2
cfg = gen.scaled_config(gen.benchmark_config(2), d=64, Hq=2, Hkv=1, hd=32, F=64, L=128, N=8, window=4, budget=16,
                        n_obs=4, seed=du.rank_seed(0, rank))
lay = gen.gen_layer(cfg, 0)
digest = float(np.abs(lay["K"]).sum())            # replicas work on different contexts
ms = 10.0 + 5.0 * rank                            # pretend rank 1 is slower
dist.barrier()
mx = du.max_over_ranks(ms)
other = du.max_over_ranks(digest)
dist.barrier()
if rank == 0:
    print("RESULT %.3f %.3f %d" % (mx, du.whole_job_value(mx, world), int(other != digest or True)))
open(os.path.join(os.environ["PKV_OUT"], "digest_%d.txt" % rank), "w").write("%.6f" % digest)
dist.destroy_process_group()
'''


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_gloo_ranks_take_the_max_and_draw_different_contexts(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, PKV_ROOT=ROOT, PKV_OUT=str(tmp_path), OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stdout + r.stderr
    out = r.stdout
    res = [l for l in out.splitlines() if l.startswith("RESULT")]
    assert len(res) == 1                                   # rank 0 alone reports
    mx, value = float(res[0].split()[1]), float(res[0].split()[2])
    assert mx == 15.0 and value == 7.5                     # slowest rank; two contexts in that time
    dig = [(tmp_path / ("digest_%d.txt" % r_)).read_text() for r_ in range(2)]
    assert dig[0] != dig[1]                                # seed + rank: different contexts


def test_helpers_without_a_process_group():
    from paper_2609_39329_b200 import dist_util as du
    assert du.max_over_ranks(3.5) == 3.5
    assert du.whole_job_value(8.0, 4) == 2.0
    assert du.rank_seed(7, 3) == 10
