"""The C-ABI library without a GPU: it loads, exports what include/kvr.h declares, and its bookkeeping
(metadata-only pools: no CUDA calls) gives the same statuses, block tables, arena offsets and counters as
the oracle on seeded call scripts."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle as orc
from common import check_invariants, random_script, run_script
from paper_2608_30830_b200 import kvr

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "kvr.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(kvr_[a-z_]+)\s*\(", header))
    assert declared == set(kvr.EXPORTS)
    L = kvr.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_struct_layouts_match_the_header():
    # sizes the C compiler gives for the header's structs, via a tiny C program
    import subprocess
    import tempfile
    src = '#include <stdio.h>\n#include "kvr.h"\nint main(){printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(kvr_geometry), sizeof(kvr_config), sizeof(kvr_stats), sizeof(kvr_prices), sizeof(kvr_controller_config), sizeof(kvr_controller_stats));return 0;}\n'
    with tempfile.TemporaryDirectory() as d:
        open(os.path.join(d, "t.c"), "w").write(src)
        subprocess.check_call(["gcc", "-std=c11", "-I", os.path.join(ROOT, "include"), "-o", os.path.join(d, "t"), os.path.join(d, "t.c")])
        out = subprocess.check_output([os.path.join(d, "t")]).split()
    assert [int(x) for x in out] == [C.sizeof(kvr.Geometry), C.sizeof(kvr.Config), C.sizeof(kvr.Stats), C.sizeof(kvr.Prices),
                                     C.sizeof(kvr.ControllerConfig), C.sizeof(kvr.ControllerStats)]


def test_bytes_per_token(golden):
    assert kvr.bytes_per_token(80, 8, 128, 2) == int(golden["bpt_llama31_70b"][0])
    for L, kib in [(8, 32), (32, 128), (64, 256)]:
        assert kvr.bytes_per_token(L, 8, 128, 2) == kib * 1024 == orc.bytes_per_token(L, 8, 128, 2)
    assert kvr.bytes_per_token(0, 8, 128, 2) == 0
    assert kvr.bytes_per_token(8, 8, 128, 3) == 0      # dtype_bytes must be 1, 2 or 4
    assert kvr.bytes_per_token(8, 1, 4, 2) == 0        # 8-byte rows cannot be moved in 16-byte vectors


def test_create_rejects_bad_configs():
    for kw, status in [(dict(num_blocks=0), kvr.ERR_INVALID_ARG), (dict(head_dim=3), kvr.ERR_GEOMETRY),
                       (dict(route=7), kvr.ERR_INVALID_ARG), (dict(chunk_bytes=1000), kvr.ERR_INVALID_ARG),
                       (dict(initial_free_order=[0, 0, 1, 2]), kvr.ERR_INVALID_ARG)]:
        args = dict(layers=2, kv_heads=2, head_dim=4, dtype_bytes=2, block_size=4, num_blocks=4,
                    host_capacity_bytes=1 << 16, flags=kvr.METADATA_ONLY)
        args.update(kw)
        with pytest.raises(kvr.KvrError) as e:
            kvr.Pool(**args)
        assert e.value.status == status and str(e.value)


GEOM = (2, 2, 4, 2, 4)


def pair(NB, cap, seed):
    order = np.random.default_rng(seed).permutation(NB).astype(np.int32)
    a = orc.OrcPool(*GEOM, NB, cap, initial_free_order=order, with_data=False)
    b = kvr.Pool(*GEOM, NB, cap, initial_free_order=order, flags=kvr.METADATA_ONLY)
    return a, b


@pytest.mark.parametrize("seed", range(12))
def test_bookkeeping_matches_oracle_on_random_scripts(seed):
    # small host tier and small pool so HOST_FULL and HBM_FULL both occur
    NB, cap = 24, 6 * 4096
    a, b = pair(NB, cap, seed)
    ops = random_script(seed, 400, max_tokens=40)
    la = run_script(a, ops)
    lb = run_script(b, ops, after_each=lambda op, st: check_invariants(b, range(12)))
    seen = set()
    for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(la, lb):
        assert (sa, pa) == (sb, pb), op
        assert snap_a == snap_b, op
        seen.add(sa)
        seen.update(pa if isinstance(pa, list) and op[0] != "admit" else [])
    assert {orc.OK, orc.ERR_BAD_STATE, orc.ERR_UNKNOWN_REQUEST} <= seen


def test_scripts_reach_every_outcome():
    seen = set()
    for seed in range(12):
        a, _ = pair(24, 6 * 4096, seed)
        for op, st, per, _ in run_script(a, random_script(seed, 400, max_tokens=40)):
            seen.add(st)
            if isinstance(per, list) and op[0] != "admit":
                seen.update(per)
    assert {orc.OK, orc.RESIDENT, orc.RECOMPUTE, orc.HOST_FULL, orc.HBM_FULL, orc.ERR_BAD_STATE,
            orc.ERR_UNKNOWN_REQUEST, orc.ERR_INVALID_ARG} <= seen


def test_paper_pool_occupancy_in_the_library(golden):
    NB = int(golden["pool_tokens"][0]) // 16
    p = kvr.Pool(80, 8, 128, 2, 16, NB, 0, flags=kvr.METADATA_ONLY)
    n = 0
    while p.admit(n, int(golden["context_tokens"][0]))[0] == kvr.OK:
        n += 1
    assert n == int(golden["fill_contexts"][0]) and p.stats()["hbm_full_rejects"] == 1
    assert p.stats()["blocks_free"] == NB - 81 * 525


def test_metadata_only_pool_refuses_data_calls():
    p = kvr.Pool(*GEOM, 8, 1 << 16, flags=kvr.METADATA_ONLY)
    p.admit(1, 4)
    st, _ = p.export_to_device([1], 256, 1 << 20)
    assert st == kvr.ERR_BAD_STATE and "metadata-only" in kvr.last_error()
    assert p.wait() == kvr.OK and p.device_ptr is None


def test_concurrent_callers_are_serialised():
    """Four threads work on one pool at once (ctypes drops the GIL during a call), each on its own requests.
    Every call must see consistent bookkeeping: conservation and disjointness hold at the end and nothing is lost."""
    import threading
    NB = 4096
    p = kvr.Pool(*GEOM, NB, 64 * 4096, flags=kvr.METADATA_ONLY)
    errors = []

    def worker(base):
        rng = np.random.default_rng(base)
        try:
            for it in range(400):
                rid = base + int(rng.integers(8))
                kind = int(rng.integers(6))
                if kind == 0:
                    p.admit(rid, int(rng.integers(1, 60)))
                elif kind == 1:
                    p.suspend_to_host([rid])
                elif kind == 2:
                    p.resume_from_host([rid])
                elif kind == 3:
                    p.expire([rid])
                elif kind == 4:
                    p.retain_in_hbm([rid])
                else:
                    p.release(rid)
                if it % 50 == 0:
                    s = p.stats()
                    assert s["blocks_free"] + s["blocks_active"] + s["blocks_pinned"] == NB
        except Exception as e:        # surfaced below: an assertion in a thread would otherwise vanish
            errors.append(e)
    threads = [threading.Thread(target=worker, args=(100 * k,)) for k in range(1, 5)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    ids = [100 * k + i for k in range(1, 5) for i in range(8)]
    check_invariants(p, ids)


def test_a_plain_c_program_can_drive_the_library(tmp_path):
    """The boundary is a C ABI: compile a C11 program against include/kvr.h, link libkvr.so, run a bookkeeping flow."""
    import subprocess
    src = r'''
    #include <stdio.h>
    #include <math.h>
    #include "kvr.h"
    int main(void) {
      kvr_config cfg = {0};
      cfg.g = (kvr_geometry){ .layers = 2, .kv_heads = 2, .head_dim = 4, .dtype_bytes = 2, .block_size = 4 };
      cfg.num_blocks = 8; cfg.host_capacity_bytes = 1 << 16; cfg.flags = KVR_METADATA_ONLY;
      kvr_pool *pool = NULL;
      if (kvr_pool_create(&cfg, &pool) != KVR_OK) { printf("create: %s\n", kvr_last_error()); return 1; }
      int32_t blocks[3] = {5, 2, 7}, got[3];
      uint64_t req = 42;
      if (kvr_request_admit_into(pool, req, 9, blocks, 3) != KVR_OK) return 2;
      if (kvr_suspend_to_host(pool, &req, 1, KVR_SYNC, NULL) != KVR_OK) return 3;
      if (kvr_expire(pool, &req, 1, NULL) != KVR_OK) return 4;
      if (kvr_resume_from_host(pool, &req, 1, 0, NULL) != KVR_RECOMPUTE) return 5;
      if (kvr_request_admit(pool, req, 9, got, 3) != KVR_OK) return 6;
      kvr_stats st;
      kvr_pool_stats(pool, &st);
      kvr_prices pr = {0.0176, 0.02, 1.91};
      double t1, ts, t2;
      kvr_policy_break_evens(&pr, &t1, &ts);
      kvr_policy_host_ttl(&pr, 2 * 425.0 / 1800.0, 425.0, 1800.0, NULL, &t2);
      printf("%lld %lld %d %d %d %.3f %.1f %.1f %llu\n", (long long)st.blocks_free, (long long)st.recompute_marked,
             got[0], got[1], got[2], t1, ts, t2, (unsigned long long)kvr_bytes_per_token(&cfg.g));
      return kvr_pool_destroy(pool);
    }
    '''
    c = tmp_path / "t.c"
    c.write_text(src)
    exe = tmp_path / "t"
    pkg = os.path.join(ROOT, "paper_2608_30830_b200")
    kvr.lib()
    subprocess.check_call(["gcc", "-std=c11", "-I", os.path.join(ROOT, "include"), str(c), "-o", str(exe),
                           "-L", pkg, "-l:libkvr.so", "-Wl,-rpath," + pkg, "-lm"])
    out = subprocess.check_output([str(exe)], text=True).split()
    # free queue after the flow: 0 1 3 4 6 5 2 7 -> admit takes 0 1 3; five blocks stay free
    assert out == ["5", "1", "0", "1", "3", "1.136", "108.5", "1781.2", "64"]
