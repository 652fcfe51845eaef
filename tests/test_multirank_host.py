"""Host-side logic of the multi-GPU benchmark path on CPU: two gloo ranks. The layer shards as
independent replicas (no collective on the data path), so what N > 1 adds is the barrier, the
maximum over ranks of the timed region and the aggregate throughput; the reference arm runs on
rank 0 only."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo", rank=rank, world_size=int(os.environ["WORLD_SIZE"]))
mine = [10.0 + 5.0 * rank, 3.0 - rank]      # rank 1 is slower on the first, faster on the second
dist.barrier()
got = bench.max_over_ranks(mine, dist, "cpu")
dist.barrier()
dist.destroy_process_group()
print(json.dumps(got))
"""


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    import json
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29733")
        procs.append(subprocess.Popen([sys.executable, "-c", _WORKER, ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    assert outs[0] == outs[1] == [15.0, 3.0]
    sys.path.insert(0, ROOT)
    import bench
    v1 = bench.aggregate_value(1, 437e9, 0.6)
    v2 = bench.aggregate_value(2, 437e9, 0.6)
    assert abs(v2 / v1 - 2.0) < 1e-12           # weak scaling: same work per rank, slowest rank sets the time
    assert bench.max_over_ranks([1.5, 2.5], None, "cpu") == [1.5, 2.5]


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
