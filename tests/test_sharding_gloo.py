"""Multi-GPU path of the benchmark on CPU: independent requests are sharded over ranks with no
data-path collective; only the timing reduction (MAX over ranks) uses the process group.  Runs
world_size = 2 with the gloo backend."""
import os
import subprocess
import sys

import bench

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
mine = bench.shard_requests(5, 2, rank)
# every request is owned by exactly one rank
owned = [torch.zeros(5, dtype=torch.int64) for _ in range(2)]
mask = torch.zeros(5, dtype=torch.int64); mask[mine] = 1
dist.all_gather(owned, mask)
assert torch.equal(owned[0] + owned[1], torch.ones(5, dtype=torch.int64)), owned
# the reported time is the maximum over ranks
t = torch.tensor([1.0 + rank], dtype=torch.float64)
dist.all_reduce(t, op=dist.ReduceOp.MAX)
assert float(t) == 2.0
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok", mine)
"""


def test_shard_requests_partitions_without_overlap():
    for total in (0, 1, 4, 5, 17):
        for world in (1, 2, 3, 8):
            parts = [bench.shard_requests(total, world, r) for r in range(world)]
            flat = [i for p in parts for i in p]
            assert flat == list(range(total))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def test_two_gloo_ranks_shard_requests_and_reduce_time(tmp_path):
    port = 29500 + os.getpid() % 2000
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
    assert "rank 0 ok [0, 1, 2]" in outs[0] and "rank 1 ok [3, 4]" in outs[1]
