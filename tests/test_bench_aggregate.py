"""bench.py's whole-job aggregation over ranks (time = max, units = sum), on 2 gloo ranks."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_rank_gloo_aggregation(tmp_path):
    script = tmp_path / "agg.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        r = dist.get_rank()
        ms, units = bench.aggregate(dist, 10.0 + 5.0 * r, 1000.0 * (r + 1))
        assert ms == 15.0 and units == 3000.0, (ms, units)
        one_ms, one_units = bench.aggregate(None, 7.0, 11.0)
        assert (one_ms, one_units) == (7.0, 11.0)
        dist.barrier(); dist.destroy_process_group()
        print("rank", r, "ok")
    """))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stdout + out.stderr
    assert out.stdout.count("ok") == 2
