"""bench.py's reference arm runs on CPU: check the JSON line it prints against the benchmark contract."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "1", "--workload", "tiny"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [x for x in out.stdout.splitlines() if x.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline", "impl"):
        assert key in d, key
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["config"]["workload"] == "tiny" and d["data"] == "synthetic" and d["dtype"] == "u8"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1 and d["cpu_baseline"]["value"] == d["value"] > 0
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_other_ranks_of_the_reference_arm_stay_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "1"], capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_plain_launch_with_gpus_2_starts_two_ranks_and_prints_one_line():
    """`python bench.py --gpus 2` with no launcher in the environment must start the ranks itself.  Checked without a
    GPU through --dry-run: metadata-only pools, gloo ranks, the same barriers and reductions, one line from rank 0."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "2",
                          "--warmup", "1", "--workload", "paper_shape"], capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [x for x in out.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["dry_run"] is True and d["value"] is None and d["scaling"] == "weak"
    # 32 contexts of 8,400 tokens sharing 337 whole blocks (5,392 tokens): 3,008 private tokens each, on both ranks
    assert d["bookkeeping"]["bytes_suspended_per_step_all_ranks"] == 2 * 32 * 3008 * 80 * 2 * 128 * 2 * 2


import pytest  # noqa: E402


@pytest.mark.gpu
def test_our_arm_prints_one_contract_line_on_a_gpu():
    """`python bench.py` on a B200 (here the small configuration): one JSON line with the base keys, the roofline
    and CPU-baseline objects, an end-to-end figure whose bytes really crossed the link, and kernels of our own."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny", "--steps", "2", "--warmup", "3",
                          "--no-extras"], capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [x for x in out.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 2 and d["warmup"] == 3 and d["unit"] == "GB/s" and d["dtype"] == "u8"
    assert d["config"]["workload"] == "tiny" and d["config"]["staging"]["library_default"] is True
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 1000 and 0.2 < r["frac"] == pytest.approx(r["achieved"] / r["peak"])
    assert r["traffic"] is not None and 0 < r["traffic"] <= r["algorithmic_bytes_per_launch"]
    payload = d["config"]["payload_bytes_per_direction"]
    assert d["e2e"]["d2h_bytes_per_step"] >= payload and d["e2e"]["h2d_bytes_per_step"] >= payload     # the bytes crossed the link
    assert 0 < d["e2e"]["value"] <= d["value"] * 1.05 and d["gpu_launches"] >= 4
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1 and d["cpu_baseline"]["value"] > 0
    assert d["host_link"]["suspend_frac_of_d2h_peak"] > 0.5 and d["host_link"]["resume_frac_of_h2d_peak"] > 0.5


@pytest.mark.gpu
def test_the_movers_alone_keep_up_with_a_plain_device_copy():
    """`python bench.py --alone-by-size`: the paged gather and scatter, one launch each, beside torch's copy_ of the
    same number of contiguous bytes.  With work handed out through the launch's counter the bulk mover is at least as
    fast as the plain copy from 64 MiB on; the bound here is loose (shared machine), the fixed-share kernel failed it."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    if torch.cuda.mem_get_info()[0] < (44 << 30):
        pytest.skip("needs 44 GiB of free device memory")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--alone-by-size"], capture_output=True, text=True,
                         timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [x for x in out.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    rows = json.loads(lines[0])["rows"]
    assert [r["launch_mib"] for r in rows] == [16, 64, 256, 1024, 2048, 4096]
    for r in rows[3:]:
        assert r["gather_vs_copy"] > 0.97 and r["scatter_vs_copy"] > 0.97, r
        assert r["gather_frac_of_peak"] > 0.93 and r["scatter_frac_of_peak"] > 0.93, r
