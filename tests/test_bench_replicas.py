"""The multi-GPU arm of bench.py runs independent replicas; only its reporting step talks between ranks.  That
step is checked here with two gloo ranks on the CPU: tokens add up, the slowest rank sets the time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_aggregate_single_rank():
    sys.path.insert(0, ROOT)
    import bench
    v, e, ms = bench.aggregate_replicas(200.0, 0.5, 100.0, 2, 1)
    assert abs(v - 500.0) < 1e-9 and abs(e - 200.0) < 1e-9 and abs(ms - 100.0) < 1e-9


def test_aggregate_two_gloo_ranks(tmp_path):
    script = tmp_path / "agg.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        r = dist.get_rank()
        # rank 0: 100 tokens in 200 ms (0.5 s end to end); rank 1: 100 tokens in 250 ms (0.4 s end to end)
        out = bench.aggregate_replicas(200.0 + 50.0 * r, 0.5 - 0.1 * r, 100.0, 2, 2)
        if r == 0:
            print(json.dumps(out))
        dist.barrier()
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)],
                         capture_output=True, text=True, timeout=240, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    import json
    line = [l for l in res.stdout.splitlines() if l.startswith("[")][-1]
    v, e, ms = json.loads(line)
    assert abs(v - 200.0 / 0.25) < 1e-6          # 200 tokens over the slower rank's 250 ms
    assert abs(e - 200.0 / 0.5) < 1e-6           # end to end: the slower rank took 0.5 s
    assert abs(ms - 125.0) < 1e-6
