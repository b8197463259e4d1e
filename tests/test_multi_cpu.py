"""The multi-rank plumbing of the benchmark on CPU: two gloo ranks, the same reductions bench.py uses."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

from paper_2608_30830_b200.multi import Group, fit_requests, job_throughput

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_fit_requests_scale_rule():
    lens = np.array([8192] * 32)
    bpt = 131072
    assert fit_requests(lens, bpt, 200 << 30, 1) == 32                  # 32 GiB of images fit in 60% of 200 GiB
    assert fit_requests(lens, bpt, 200 << 30, 8) == 13                  # 15 GiB per rank -> 13 GiB of images + slack
    assert fit_requests(lens, bpt, 1 << 30, 8) == 1                     # never below one request
    n = fit_requests(lens, bpt, 200 << 30, 4)
    assert n * 8192 * bpt + (2 << 30) <= 0.6 * (200 << 30) / 4 < (n + 1) * 8192 * bpt + (2 << 30)


def test_single_rank_group_is_a_no_op():
    g = Group("gloo")
    assert (g.rank, g.world) == (0, 1)
    assert g.max([1.5, 2.0]) == [1.5, 2.0] and g.sum([3]) == [3.0]
    assert job_throughput(10.0, 2.0, g) == (5.0, 10.0, 2.0)
    g.barrier()
    g.close()


WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2608_30830_b200.multi import Group, job_throughput
    g = Group("gloo")
    g.barrier()
    # rank r moved (r + 1) GB in (r + 1) * 0.5 s: the job moved 3 GB in 1.0 s
    rate, total, slowest = job_throughput((g.rank + 1) * 1e9, (g.rank + 1) * 0.5, g)
    mx = g.max([g.rank, 10 - g.rank])
    assert (total, slowest, rate) == (3e9, 1.0, 3e9), (total, slowest, rate)
    assert mx == [1.0, 10.0], mx
    if g.rank == 0:
        print("RESULT", rate, g.world)
    g.close()
""")


def test_two_gloo_ranks_reduce_like_the_benchmark(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "RESULT 3000000000.0 2" in out.stdout
