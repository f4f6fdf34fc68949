"""The multi-process path of bench.py on CPU: two gloo ranks (replicas only, no data-path collective);
the whole-job value is all ranks' units over the max-over-ranks time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent('''
    import os, sys, json
    sys.path.insert(0, os.environ["EORA_ROOT"])
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    bench._DIST["on"] = True
    rank = dist.get_rank()
    bench.barrier()
    value, ms = bench.aggregate(10.0 if rank == 0 else 25.0, 3, dist.get_world_size())
    if rank == 0:
        print(json.dumps({"value": value, "ms": ms}))
    dist.barrier()
    dist.destroy_process_group()
''')


def test_two_rank_aggregation_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, EORA_ROOT=ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    import json
    d = json.loads(line)
    assert d["ms"] == 25.0                         # the slower rank sets the time
    assert abs(d["value"] - 2 * 3 / 0.025) < 1e-9  # both ranks' units over that time


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
