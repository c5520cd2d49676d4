"""world_size-2 gloo test of the N>1 plumbing (replicas only: barrier, max time, summed units)."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
from paper_2502_18394_b200 import replicas as R
R.init("gloo")
rank, _, ws = R.world()
R.barrier()
t, u = R.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1))
assert ws == 2 and t == 15.0 and u == 300.0, (t, u)
R.barrier()
R.finish()
sys.stdout.write("rank" + str(rank) + "ok\n"); sys.stdout.flush()
""" % ROOT


def test_two_rank_aggregate_gloo(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)]
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240, env=env)
    assert res.returncode == 0, res.stdout + res.stderr
    out = res.stdout + res.stderr
    assert "rank0ok" in out and "rank1ok" in out


def test_single_process_aggregate_is_identity():
    from paper_2502_18394_b200 import replicas as R
    assert R.aggregate(3.0, 7.0) == (3.0, 7.0)
