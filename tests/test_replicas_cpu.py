"""The multi-GPU path is "replicas only": every rank decodes its own sequence and the only cross-rank step
is the max-over-ranks of the step time.  This runs that step on two gloo ranks on the CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_max_over_ranks_and_job_value_two_gloo_ranks(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        local = 100.0 + 50.0 * rank                 # rank 1 is the slow one
        worst = bench.max_over_ranks(local)
        assert worst == 150.0, worst
        assert bench.job_value(worst, world) == 75.0
        dist.barrier()
        if rank == 0:
            print("OK", worst, bench.job_value(worst, world))
        dist.destroy_process_group()
    """))
    port = _free_port()
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                        "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
                       capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "OK 150.0 75.0" in r.stdout


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5) == 12.5
    assert bench.job_value(12.5, 1) == 12.5
