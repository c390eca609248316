"""The N > 1 plumbing on CPU: two gloo ranks, max-over-ranks timing and the whole-job throughput formula."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2607_08782_b200.multirank import Ranks
    r = Ranks(backend="gloo")
    assert r.world == 2
    r.barrier()
    local_seconds = 1.0 + r.rank            # rank 0: 1 s, rank 1: 2 s
    slowest = r.max_over_ranks(local_seconds)
    rate = r.whole_job_rate(1000.0, local_seconds)
    r.barrier()
    open(sys.argv[1] + "/rank%%d.txt" %% r.rank, "w").write("%%r %%r" %% (slowest, rate))
    r.close()
""")


def test_two_gloo_ranks_take_the_max_time_and_aggregate_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    out = None
    for _ in range(2):                                  # a port picked as free can still be taken: try twice
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
               "--master-addr", "127.0.0.1", "--master-port", str(port), str(script), str(tmp_path)]
        out = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
        if out.returncode == 0:
            break
    assert out.returncode == 0, out.stderr[-2000:]
    for rank in range(2):
        slowest, rate = (tmp_path / f"rank{rank}.txt").read_text().split()
        assert float(slowest) == 2.0                 # the slower replica defines the step time
        assert float(rate) == 2 * 1000.0 / 2.0       # all ranks' units over that time


def test_single_process_is_a_no_op():
    from paper_2607_08782_b200.multirank import Ranks
    env = {k: os.environ.pop(k) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK") if k in os.environ}
    try:
        r = Ranks(backend="gloo")
        assert r.world == 1 and r.max_over_ranks(3.5) == 3.5 and r.whole_job_rate(10, 2.0) == 5.0
        r.barrier()
        r.close()
    finally:
        os.environ.update(env)
