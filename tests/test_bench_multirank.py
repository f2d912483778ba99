"""Host-side logic of the multi-rank benchmark path on CPU: two gloo ranks, the max-over-ranks
timing reduction and the work totals (no GPU, no data-path collective)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    ms, graphs, edges, nodes = bench.reduce_over_ranks(10.0 + 5.0 * rank, 100 + rank, 1000, 500, dist, "cpu")
    if rank == 0:
        print(json.dumps({"ms": ms, "graphs": graphs, "edges": edges, "nodes": nodes}))
    dist.destroy_process_group()
""") % ROOT


def test_two_rank_reduction_with_gloo(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(SCRIPT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29611", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300,
                       env=dict(os.environ, CUDA_VISIBLE_DEVICES=""))
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    import json
    out = json.loads(line)
    assert out["ms"] == 15.0                      # the slowest rank sets the time
    assert out["graphs"] == 201 and out["edges"] == 2000 and out["nodes"] == 1000


def test_rank_seeds_differ():
    import bench
    assert bench.rank_seed(4, 0) != bench.rank_seed(4, 1)
