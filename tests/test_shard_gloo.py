"""The multi-rank path on CPU: two gloo ranks own disjoint env ranges, reproduce the global
population without exchanging data, and agree on the timing reduction the bench uses."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2207_07736_b200 import shard

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %(root)r)
import numpy as np
import oracle
from paper_2207_07736_b200 import shard
rank, local_rank, world = shard.dist_env()
dist = shard.init_process_group("gloo")
off, n = shard.env_range(rank, world, 24)
sim = oracle.OracleSim(oracle.CARTPOLE, seed=7, env_ids=np.arange(off, off + n, dtype=np.uint32))
out = sim.rollout(40)
np.save(os.path.join(%(tmp)r, "obs%%d.npy" %% rank), out["obs"])
np.save(os.path.join(%(tmp)r, "done%%d.npy" %% rank), out["done"])
dist.barrier()
ms, units = shard.reduce_timing(dist, 10.0 * (rank + 1), float(n * 40))
if rank == 0:
    print(json.dumps({"ms": ms, "units": units, "world": world}))
dist.barrier()
dist.destroy_process_group()
"""


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_env_range():
    assert shard.env_range(0, 1, 100) == (0, 100)
    assert shard.env_range(3, 8, 65536) == (3 * 65536, 65536)
    with pytest.raises(ValueError):
        shard.env_range(2, 2, 10)
    with pytest.raises(ValueError):
        shard.env_range(0, 8, 1 << 30)                    # 2^33 envs do not fit the counter word
    assert shard.reduce_timing(None, 3.0, 5.0) == (3.0, 5.0)


def test_two_gloo_ranks_reproduce_the_global_population(tmp_path):
    port = free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER % {"root": ROOT, "tmp": str(tmp_path)})
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (so, se) in zip(procs, outs):
        assert p.returncode == 0, se
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line == {"ms": 20.0, "units": 2 * 24 * 40.0, "world": 2}        # max over ranks, sum of units
    ref = oracle.OracleSim(oracle.CARTPOLE, 48, seed=7).rollout(40)
    obs = np.concatenate([np.load(tmp_path / "obs0.npy"), np.load(tmp_path / "obs1.npy")], axis=1)
    done = np.concatenate([np.load(tmp_path / "done0.npy"), np.load(tmp_path / "done1.npy")], axis=1)
    assert np.array_equal(obs, ref["obs"]) and np.array_equal(done, ref["done"])
