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


# ---- shared prefixes, reference counts ------------------------------------------------------

@pytest.mark.parametrize("seed", range(8))
def test_sharing_scripts_match_the_oracle(seed):
    """Scripts whose admissions name donors and shared-prefix lengths (legal and illegal): statuses, tables, kept
    prefixes, reference counts, arena offsets, free-queue order and counters equal the oracle's after every call."""
    NB, cap = 32, 8 * 4096
    a, b = pair(NB, cap, seed)
    ops = random_script(500 + seed, 500, max_tokens=40, sharing=True)
    la = run_script(a, ops)
    lb = run_script(b, ops, after_each=lambda op, st: check_invariants(b, range(12)))
    shared_admissions = 0
    for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(la, lb):
        assert (sa, pa) == (sb, pb), op
        assert snap_a == snap_b, op
        shared_admissions += op[0] == "admit_sharing" and sa == orc.OK and op[4] > 0
    assert shared_admissions > 0


def test_paper_context_split_in_the_library(golden):
    """Section 2 / Appendix B: an 8,400-token context whose 5,400-token system prefix is shared moves 3,000 tokens =
    983,040,000 bytes (0.98 GB), not 2.75 GB; the prefix stays resident while any referrer waits on the host."""
    L, H, D, e = (int(x) for x in golden["bpt_factors"])
    p = kvr.Pool(L, H, D, e, 8, 4096, 8 << 30, flags=kvr.METADATA_ONLY)
    ctx, shared = int(golden["context_tokens"][0]), int(golden["shared_prefix_tokens"][0])
    assert p.admit(0, shared)[0] == kvr.OK
    for rid in (1, 2, 3):
        assert p.admit_sharing(rid, ctx, 0, shared // 8)[0] == kvr.OK
    assert p.release(0) == kvr.OK                                           # the prefix outlives the request that made it
    assert p.suspend_to_host([1, 2, 3])[0] == kvr.OK
    s = p.stats()
    assert s["bytes_suspended"] == 3 * 983_040_000 and s["blocks_pinned"] == 675 and s["blocks_free"] == 4096 - 675
    assert p.refcount(int(p.sharing(1)[1][0])) == 3
    assert p.expire([1])[0] == kvr.OK and p.release(2) == kvr.OK
    assert p.stats()["blocks_pinned"] == 675                                # request 3 still refers to it
    assert p.resume_from_host([3])[0] == kvr.OK and p.info(3)[1]["nb"] == 1050
    assert p.release(3) == kvr.OK and p.stats()["blocks_free"] == 4096      # freed with the last referrer


# ---- a move that cannot be enqueued leaves everything unchanged (host-made failures) -----------

def full_snapshot(p, ids):
    from common import snapshot
    return snapshot(p, ids)


def test_injected_allocation_failures_leave_a_metadata_pool_unchanged():
    NB, cap = 32, 8 * 4096
    order = np.random.default_rng(3).permutation(NB).astype(np.int32)

    def fresh():
        o = orc.OrcPool(*GEOM, NB, cap, initial_free_order=order, with_data=False)
        g = kvr.Pool(*GEOM, NB, cap, initial_free_order=order, flags=kvr.METADATA_ONLY)
        for pool in (o, g):
            assert pool.admit(1, 13)[0] == 0 and pool.admit_sharing(2, 17, 1, 2)[0] == 0 and pool.admit(3, 5)[0] == 0
            assert pool.retain_in_hbm([3])[0] == 0
        return o, g
    for call in ("suspend", "resume", "resume_into"):
        o, g = fresh()
        if call != "suspend":
            assert o.suspend_to_host([1, 2, 3])[0] == g.suspend_to_host([1, 2, 3])[0] == kvr.OK
        pick = g.free_queue()[[5, 2, 9]].astype(np.int32)                    # request 2's private part: 3 blocks
        do = {"suspend": lambda pool: pool.suspend_to_host([1, 9, 2, 3])[0],
              "resume": lambda pool: pool.resume_from_host([2, 1, 9, 3])[0],
              "resume_into": lambda pool: pool.resume_from_host_into(2, pick)}[call]
        # how many allocation points does the call pass?  (armed far away, then read the counter)
        probe = fresh()[1]
        if call != "suspend":
            probe.suspend_to_host([1, 2, 3])
        assert probe.test_fail_nth(kvr.FAIL_ALLOC, 10**9) == kvr.OK
        do(probe)
        n_points = probe.test_points(kvr.FAIL_ALLOC)
        assert n_points >= 2
        for k in range(1, n_points + 1):
            before = full_snapshot(g, range(12))
            assert g.test_fail_nth(kvr.FAIL_ALLOC, k) == kvr.OK
            st = do(g)
            assert st == kvr.ERR_NOMEM, (call, k, st)
            assert g.test_fail_nth(kvr.FAIL_ALLOC, 0) == kvr.OK
            assert full_snapshot(g, range(12)) == before, (call, k)
            check_invariants(g, range(12))
        # disarmed, the same call goes through, and the pool keeps agreeing with the oracle afterwards
        assert do(g) == do(o)
        ops = random_script(77, 50, max_tokens=40, sharing=True)
        for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(run_script(o, ops), run_script(g, ops)):
            assert (sa, pa) == (sb, pb) and snap_a == snap_b, (call, op)


# ---- free queue: named blocks leave in O(1) -------------------------------------------------------

def test_named_admission_costs_microseconds_at_the_largest_pool():
    """Appendix A: pinning removes blocks from the doubly linked free queue in O(1).  At the long-context
    configuration's 147,456 blocks a named admission of 64 blocks must not scan the queue."""
    import time
    NB = 147456
    p = kvr.Pool(32, 8, 128, 2, 8, NB, 0, flags=kvr.METADATA_ONLY)
    rng = np.random.default_rng(0)
    picks = rng.permutation(NB - 64)[:64 * 200].astype(np.int32).reshape(200, 64)
    p.admit_into(10**6, 64 * 8, np.arange(NB - 64, NB, dtype=np.int32))     # warm-up
    t0 = time.perf_counter()
    for i in range(200):
        assert p.admit_into(i, 64 * 8, picks[i]) == kvr.OK
    per_call = (time.perf_counter() - t0) / 200
    assert per_call < 200e-6, per_call            # ctypes marshalling included; a queue scan would cost ~1 ms
    fq = p.free_queue()
    named = set(picks.reshape(-1).tolist())
    assert len(fq) == NB - 64 * 201 and not (set(fq.tolist()) & named)
    assert fq.tolist() == [b for b in range(NB - 64) if b not in named]      # the other ids kept their order


# ---- NUMA placement: sysfs parsing against a fake tree -------------------------------------------

def test_numa_lookup_against_a_fake_sysfs_tree(tmp_path):
    dev = tmp_path / "bus" / "pci" / "devices" / "0000:1b:00.0"
    dev.mkdir(parents=True)
    (dev / "numa_node").write_text("1\n")
    node1 = tmp_path / "devices" / "system" / "node" / "node1"
    node1.mkdir(parents=True)
    (node1 / "cpulist").write_text("16-31,48-50,63\n")
    node, cpus = kvr.numa_lookup(tmp_path, "0000:1B:00.0")                   # CUDA prints the bus id in upper case
    assert node == 1 and cpus == list(range(16, 32)) + [48, 49, 50, 63]
    # a platform that does not say (-1), a device that is not there, a malformed list
    (dev / "numa_node").write_text("-1\n")
    assert kvr.numa_lookup(tmp_path, "0000:1b:00.0") == (-1, [])
    assert kvr.numa_lookup(tmp_path, "0000:ff:00.0") == (-1, [])
    (dev / "numa_node").write_text("1\n")
    (node1 / "cpulist").write_text("3-1\n")
    assert kvr.numa_lookup(tmp_path, "0000:1b:00.0") == (1, [])
    assert kvr.Pool(*GEOM, 8, 1 << 16, flags=kvr.METADATA_ONLY).numa_node == -1
