"""The multi-GPU path shards one call by heads with no collective on the data path.  What can be
checked without GPUs: the partition covers every (batch, head) pair exactly once for any world size,
and two real ranks (gloo, CPU) that each generate only their own heads hold, together, exactly the
inputs of the unsharded call and agree on the global result of a max-over-ranks timing reduction."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import WORKLOADS
from paper_2607_24027_b200.shard import head_partition

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("heads", [1, 2, 7, 24, 40])
@pytest.mark.parametrize("world", [1, 2, 3, 4, 8, 64])
def test_partition_covers_every_head_once(heads, world):
    seen = []
    for r in range(world):
        s = head_partition(heads, world, r)
        seen.extend(range(heads)[s])
    assert seen == list(range(heads))
    sizes = [len(range(heads)[head_partition(heads, world, r)]) for r in range(world)]
    assert max(sizes) - min(sizes) <= 1


def test_partition_rejects_bad_requests():
    for args in [(-1, 2, 0), (4, 0, 0), (4, 2, 2), (4, 2, -1)]:
        with pytest.raises(ValueError):
            head_partition(*args)


_RANK_SCRIPT = r"""
import os, sys, hashlib
import numpy as np
import torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
from paper_2607_24027_b200 import synth
from paper_2607_24027_b200.configs import WORKLOADS
from paper_2607_24027_b200.shard import head_partition
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
wl = WORKLOADS["tiny"]
mine = head_partition(wl.batch * wl.heads, world, rank)
q, k, v = synth.generate(wl, heads=mine)                 # only this rank's heads are materialised
digest = [int.from_bytes(hashlib.sha256(np.ascontiguousarray(x[i]).tobytes()).digest()[:7], "big")
          for i in range(q.shape[0]) for x in (q, k, v)]
owned = torch.zeros(wl.batch * wl.heads, dtype=torch.int64)
owned[mine] = 1
dist.all_reduce(owned)                                    # bookkeeping only: the data path has no collective
sums = torch.zeros(wl.batch * wl.heads, 3, dtype=torch.int64)
if digest:
    sums[mine] = torch.tensor(digest, dtype=torch.int64).view(-1, 3)
dist.all_reduce(sums)
t = torch.tensor([1.0 + rank])                           # stands in for a rank's device time
dist.all_reduce(t, op=dist.ReduceOp.MAX)
if rank == 0:
    print("OWNED", owned.tolist())
    print("SUMS", sums.flatten().tolist())
    print("TMAX", float(t))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_own_disjoint_heads_and_see_the_same_bits(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script), ROOT]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = {l.split(" ", 1)[0]: l.split(" ", 1)[1] for l in out.stdout.splitlines() if l[:4] in ("OWNE", "SUMS", "TMAX")}
    wl = WORKLOADS["tiny"]
    assert eval(lines["OWNED"]) == [1] * (wl.batch * wl.heads)          # every head owned exactly once
    import hashlib
    q, k, v = synth.generate(wl)
    want = [int.from_bytes(hashlib.sha256(np.ascontiguousarray(x[0, h]).tobytes()).digest()[:7], "big")
            for h in range(wl.heads) for x in (q, k, v)]
    assert eval(lines["SUMS"]) == want                                   # the shards are the unsharded inputs
    assert float(lines["TMAX"]) == 2.0
