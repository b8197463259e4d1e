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


TP_WORKER = textwrap.dedent("""
    import hashlib, sys
    sys.path.insert(0, %r); sys.path.insert(0, %r)
    import numpy as np
    from common import random_script, run_script
    from paper_2608_30830_b200 import kvr
    from paper_2608_30830_b200.multi import Group
    g = Group("gloo")
    # tensor parallel: every rank holds kv_heads / world heads of every token, in its own pool with its own host tier
    heads = 8 // g.world
    order = np.random.default_rng(5).permutation(64).astype(np.int32)
    pool = kvr.Pool(4, heads, 128, 2, 16, 64, 40 * 4096 * heads, initial_free_order=order, flags=kvr.METADATA_ONLY)
    log = run_script(pool, random_script(5, 300, max_tokens=200))
    # what must agree across ranks: every status, every block table, the free queue, which requests are where
    view = [(op, st, per, {k: (v if isinstance(v, int) else (v[0], v[1], v[2], v[5])) for k, v in snap[0].items()}, snap[1])
            for op, st, per, snap in log]
    digest = int.from_bytes(hashlib.sha256(repr(view).encode()).digest()[:6], "big")
    hi, lo = g.max([digest])[0], -g.max([-digest])[0]
    assert hi == lo == digest, (hi, lo, digest)
    if g.rank == 0:
        print("AGREE", g.world, len(log))
    g.close()
""")


def test_tensor_parallel_ranks_take_identical_decisions(tmp_path):
    """The bookkeeping is deterministic, so ranks that shard the KV heads and issue the same calls admit, reject and
    place every request identically without exchanging a byte; the test compares digests over two gloo ranks."""
    script = tmp_path / "tp_worker.py"
    script.write_text(TP_WORKER % (ROOT, os.path.join(ROOT, "tests")))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "AGREE 2 300" in out.stdout
