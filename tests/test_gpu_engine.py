"""GPU tests of the transfer engine's plumbing, byte for byte against the oracle through the C ABI:
staging rings whose launches span several slots and wrap around the ring's end, shared prefixes with data, moves
that fail while being enqueued (host-made failures: nothing here faults the GPU), caller-owned staging memory and
streams, the automatic route."""
import numpy as np
import pytest
import torch

import oracle as orc
from common import check_invariants, random_script, run_script, snapshot
from paper_2608_30830_b200 import kvr

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

from gpu_common import Twin  # noqa: E402

SMALL = (3, 2, 16, 2, 8)          # L, H, D, e, BS: 64-byte rows, 512-byte tiles, 384 bytes per token

RINGS = [
    pytest.param(dict(chunk_bytes=4096, staging_slots=3), id="3x4K"),
    pytest.param(dict(chunk_bytes=4096, staging_slots=5, suspend_single_bytes=8192, resume_single_bytes=8192), id="5x4K-single8K"),
    pytest.param(dict(chunk_bytes=8192, staging_slots=16, suspend_single_bytes=4096, resume_single_bytes=4096, copy_piece_bytes=4096), id="16x8K-piece4K"),
    pytest.param(dict(chunk_bytes=4096, staging_slots=7, copy_piece_bytes=12288), id="7x4K-piece12K"),
    pytest.param(dict(chunk_bytes=12288, staging_slots=4, kernel=kvr.KERNEL_WARP), id="4x12K-warp"),
]


@pytest.mark.parametrize("ring", RINGS)
@pytest.mark.parametrize("seed", [0, 1])
def test_rings_with_launches_that_span_slots_and_wrap(ring, seed):
    """Slot sizes that are not multiples of a request's plane size, so runs of tiles end at arbitrary offsets, the
    ring wraps inside launches (leaving a gap before its end) and copies are cut at slot and piece boundaries."""
    NB, cap = 64, 14 * 4096
    t = Twin(SMALL, NB, cap, seed=seed, **ring)
    ops = random_script(300 + seed, 300, max_tokens=110)
    la = run_script(t.o, ops)
    lb = run_script(t.g, ops)
    for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(la, lb):
        assert (sa, pa) == (sb, pb) and snap_a == snap_b, op
    t.assert_same_images(range(12))
    t.assert_same_pool()
    s = t.g.stats()
    assert s["gather_bytes"] == s["bytes_suspended"] and s["scatter_bytes"] == s["bytes_resumed"] > 0
    t.close()


def test_one_large_batch_through_a_small_ring():
    """One batched suspend and resume of 40 ragged requests through a 6-slot ring: launches of up to five slots,
    dozens of wraps, every image and the whole pool against the oracle."""
    geom = (2, 8, 128, 2, 16)                     # 2 KiB rows, 32 KiB tiles, 8 KiB per token
    t = Twin(geom, 2048, 160 << 20, seed=4, chunk_bytes=1 << 20, staging_slots=6, suspend_single_bytes=2 << 20, resume_single_bytes=2 << 20)
    rng = np.random.default_rng(4)
    lens = [int(x) for x in rng.integers(1, 700, size=40)]
    ids = list(range(40))
    for rid, n in zip(ids, lens):
        a, b = t.both("admit", rid, n)
        assert a[0] == b[0] == orc.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b and a[0] == orc.OK
    t.assert_same_images(ids)
    t.assert_same_pool()
    a, b = t.both("resume_from_host", ids[::-1])
    assert a == b and a[0] == orc.OK
    t.assert_same_pool()
    s = t.g.stats()
    total = sum(lens) * 8192
    assert s["gather_bytes"] == s["scatter_bytes"] == total
    assert s["gather_launches"] <= total // (4 << 20) + 4              # launches of several slots, not one per slot
    t.close()


@pytest.mark.parametrize("mode", [dict(route=kvr.ROUTE_STAGED, kernel=kvr.KERNEL_BULK, chunk_bytes=4096, staging_slots=4),
                                  dict(route=kvr.ROUTE_MAPPED, kernel=kvr.KERNEL_WARP),
                                  dict(route=kvr.ROUTE_DMA2D)], ids=["staged", "mapped", "dma2d"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sharing_scripts_with_data(mode, seed):
    """Scripts with shared-prefix admissions: only private suffixes move; prefixes stay where they are, referenced;
    statuses, tables, counts, every image and the final pool equal the oracle's."""
    NB, cap = 64, 12 * 4096
    t = Twin(SMALL, NB, cap, seed=seed, **mode)
    ops = random_script(700 + seed, 350, max_tokens=90, sharing=True)
    la = run_script(t.o, ops)
    lb = run_script(t.g, ops)
    shared = 0
    for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(la, lb):
        assert (sa, pa) == (sb, pb) and snap_a == snap_b, op
        shared += op[0] == "admit_sharing" and sa == orc.OK and op[4] > 0
    assert shared > 0
    t.assert_same_images(range(12))
    t.assert_same_pool()
    check_invariants(t.g, range(12))
    t.close()


def test_shared_prefix_round_trip_moves_the_suffix_only():
    geom = (4, 8, 128, 2, 16)
    bpt = kvr.bytes_per_token(*geom[:4])
    t = Twin(geom, 512, 64 << 20, seed=9)
    a, b = t.both("admit", 0, 1600)                                          # the prefix: 100 full blocks
    assert a[0] == b[0] == orc.OK and a[1].tolist() == b[1].tolist()
    for rid, n in ((1, 1600 + 900), (2, 1600 + 37), (3, 1600)):
        a, b = t.both("admit_sharing", rid, n, 0, 100)
        assert a[0] == b[0] == orc.OK and a[1].tolist() == b[1].tolist()
    whole = {rid: orc.gather(t.o.data, *geom, 512, t.o.info(rid)[1]["blocks"], t.o.info(rid)[1]["n_tokens"]) for rid in (1, 2, 3)}
    assert t.both("release", 0) == (orc.OK, orc.OK)
    a, b = t.both("suspend_to_host", [1, 2, 3])
    assert a == b and a[0] == orc.OK
    t.assert_same_images([1, 2, 3])
    assert t.g.stats()["bytes_suspended"] == (900 + 37) * bpt == t.g.stats()["gather_bytes"]
    assert t.g.stats()["blocks_pinned"] == 100 and t.g.refcount(int(t.g.sharing(1)[1][0])) == 3
    a, b = t.both("resume_from_host", [3, 2, 1])
    assert a == b and a[0] == orc.OK
    t.assert_same_pool()
    got = t.pool_bytes()
    for rid in (1, 2, 3):                                                    # logical content of the whole context is back
        d = t.g.info(rid)[1]
        assert np.array_equal(orc.gather(got, *geom, 512, d["blocks"], d["n_tokens"]), whole[rid])
    t.close()


# ---- moves that fail while being enqueued -------------------------------------------------------

@pytest.mark.parametrize("kind", [kvr.FAIL_CUDA, kvr.FAIL_ALLOC], ids=["cuda-call", "host-alloc"])
@pytest.mark.parametrize("mode", [dict(route=kvr.ROUTE_STAGED, chunk_bytes=4096, staging_slots=3),
                                  dict(route=kvr.ROUTE_MAPPED), dict(route=kvr.ROUTE_DMA2D)], ids=["staged", "mapped", "dma2d"])
def test_a_move_that_cannot_be_enqueued_changes_nothing(mode, kind):
    """The n-th CUDA call (or host allocation) of a suspend, a resume and a named resume reports failure without
    being issued, for every n the call reaches.  Each time: the status is the error, every observable piece of
    bookkeeping is what it was, the pool bytes and the resident images are untouched, and once disarmed the same
    call succeeds and the pool keeps agreeing with the oracle."""
    NB = 64
    want_status = kvr.ERR_CUDA if kind == kvr.FAIL_CUDA else kvr.ERR_NOMEM
    for call in ("suspend", "resume", "resume_into"):
        # 15 granules hold all four images; with 14 the batched suspend also meets a full tier (request 3), whose
        # rejection must be taken back too when the call fails
        cap = (14 if call == "suspend" else 16) * 4096
        t = Twin(SMALL, NB, cap, seed=11, flags=kvr.PROFILE, **mode)
        for pool in (t.o, t.g):
            assert pool.admit(1, 61)[0] == 0 and pool.admit_sharing(2, 75, 1, 3)[0] == 0 and pool.admit(3, 9)[0] == 0
            assert pool.admit(4, 30)[0] == 0 and pool.suspend_to_host([4])[0] == 0          # one resident image throughout
        if call != "suspend":
            assert t.o.suspend_to_host([1, 2, 3])[0] == t.g.suspend_to_host([1, 2, 3], kvr.SYNC)[0] == kvr.OK
        pick = t.g.free_queue()[[7, 1, 4, 12, 3, 9, 0]].astype(np.int32)     # request 2's private part: 7 blocks
        do = {"suspend": lambda pool: pool.suspend_to_host([1, 9, 2, 3])[0],
              "resume": lambda pool: pool.resume_from_host([2, 1, 9, 3])[0],
              "resume_into": lambda pool: pool.resume_from_host_into(2, pick)}[call]
        assert t.g.wait() == kvr.OK
        image4 = t.g.host_image(4).copy()
        k = 0
        while True:
            k += 1
            before = snapshot(t.g, range(12))
            bytes_before = t.pool_bytes()
            assert t.g.test_fail_nth(kind, k) == kvr.OK
            st = do(t.g)
            reached = t.g.test_points(kind)
            assert t.g.test_fail_nth(kind, 0) == kvr.OK
            if reached < k:                                                  # the call has fewer such points: it went through
                assert st == do(t.o), (call, k)
                break
            assert st == want_status, (call, k, st, kvr.last_error())
            assert snapshot(t.g, range(12)) == before, (call, k)
            # nothing landed in live data: every block some request refers to holds what it held (blocks of the free
            # queue have no owner and no defined content: a resume abandoned half-way may have written into them)
            L, H, D, e, BS = SMALL
            now_bytes = t.pool_bytes().reshape(2 * L, NB, BS * H * D * e)
            live = sorted({int(b) for rid in range(12) if t.g.info(rid)[0] == kvr.OK
                           for b in (t.g.info(rid)[1]["blocks"] if t.g.info(rid)[1]["blocks"] is not None else t.g.sharing(rid)[1])})
            assert live and np.array_equal(now_bytes[:, live], bytes_before.reshape(now_bytes.shape)[:, live]), (call, k)
            assert np.array_equal(t.g.host_image(4), image4)
            check_invariants(t.g, range(12))
            assert k < 400
        assert k > 3, (call, k)
        assert t.g.wait() == kvr.OK, kvr.last_error()
        ops = random_script(91, 60, max_tokens=70, sharing=True)
        for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(run_script(t.o, ops), run_script(t.g, ops)):
            assert (sa, pa) == (sb, pb) and snap_a == snap_b, (call, op)
        t.assert_same_images(range(12))
        t.assert_same_pool()
        t.close()


# ---- resources the caller owns ------------------------------------------------------------------------

def test_caller_owned_staging_and_streams():
    geom = (2, 8, 128, 2, 16)
    slots, slot = 4, 1 << 20
    staging = torch.full((2 * slots * slot + 512,), 0x5A, dtype=torch.uint8, device="cuda")
    base = (staging.data_ptr() + 255) // 256 * 256
    streams = [torch.cuda.Stream() for _ in range(4)]
    t = Twin(geom, 512, 64 << 20, seed=6, chunk_bytes=slot, staging_slots=slots, device_staging=base,
             streams=[s.cuda_stream for s in streams])
    ids = list(range(6))
    for rid, n in zip(ids, (700, 33, 1, 512, 250, 90)):
        a, b = t.both("admit", rid, n)
        assert a[0] == b[0] == orc.OK and a[1].tolist() == b[1].tolist()
    a, b = t.both("suspend_to_host", ids)
    assert a == b
    t.assert_same_images(ids)
    a, b = t.both("resume_from_host", ids)
    assert a == b
    t.assert_same_pool()
    for s in streams:
        s.synchronize()
    off = base - staging.data_ptr()
    st = staging.cpu().numpy()
    assert (st[:off] == 0x5A).all() and (st[off + 2 * slots * slot:] == 0x5A).all()     # nothing outside the caller's range
    assert (st[off:off + 2 * slots * slot] != 0x5A).any()                               # and the range was used
    t.close()
    with pytest.raises(kvr.KvrError):                                       # the same stream twice
        kvr.Pool(*geom, 64, 1 << 20, streams=[streams[0].cuda_stream] * 4)
    with pytest.raises(kvr.KvrError):                                       # misaligned staging
        kvr.Pool(*geom, 64, 1 << 20, device_staging=base + 16, chunk_bytes=slot, staging_slots=slots)


def test_more_moves_in_flight_than_descriptor_buffers():
    """max_moves_in_flight = 2: the third un-synchronised move waits for a buffer instead of allocating one."""
    geom = (2, 8, 128, 2, 16)
    t = Twin(geom, 2048, 256 << 20, seed=3, max_moves_in_flight=2, chunk_bytes=4 << 20, staging_slots=4)
    ids = list(range(10))
    for rid in ids:
        a, b = t.both("admit", rid, 1500 + 37 * rid)
        assert a[0] == b[0] == orc.OK and a[1].tolist() == b[1].tolist()
    for rid in ids:                                                          # ten moves, no waits in between
        assert t.both("suspend_to_host", [rid]) == ((orc.OK, [orc.OK]), (kvr.OK, [kvr.OK]))
    t.assert_same_images(ids)
    for rid in ids[::-1]:
        assert t.both("resume_from_host", [rid]) == ((orc.OK, [orc.OK]), (kvr.OK, [kvr.OK]))
    t.assert_same_pool()
    t.close()


def test_a_plain_c_program_moves_data_over_staging_and_streams_it_owns(tmp_path):
    """The boundary is a C ABI: a C11 program allocates the pool, the arena, the staging memory and the four
    streams itself, hands them over in kvr_config, suspends and resumes one request, and checks the image against
    image[plane][t] = pool[plane][table[t / BS]][t % BS] computed in the program."""
    import os
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = r'''
    #include <stdio.h>
    #include <stdlib.h>
    #include <string.h>
    #include <cuda_runtime_api.h>
    #include "kvr.h"
    #define CK(x) do { if ((x) != cudaSuccess) { printf("cuda error line %d\n", __LINE__); return 10; } } while (0)
    int main(void) {
      enum { L = 2, H = 2, D = 64, E = 2, BS = 4, NB = 64, N = 61 };
      const size_t row = H * D * E, tile = BS * row, pool_bytes = (size_t)2 * L * NB * tile;
      const size_t slot = 8192, slots = 3, arena_bytes = 1 << 20;
      unsigned char *hpool = malloc(pool_bytes), *dpool, *stg, *arena;
      for (size_t i = 0; i < pool_bytes; ++i) hpool[i] = (unsigned char)((i * 2654435761u) >> 13);
      CK(cudaMalloc((void **)&dpool, pool_bytes));
      CK(cudaMalloc((void **)&stg, 2 * slots * slot));
      CK(cudaHostAlloc((void **)&arena, arena_bytes, cudaHostAllocMapped));
      CK(cudaMemcpy(dpool, hpool, pool_bytes, cudaMemcpyHostToDevice));
      cudaStream_t st[4];
      for (int i = 0; i < 4; ++i) CK(cudaStreamCreateWithFlags(&st[i], cudaStreamNonBlocking));
      kvr_config cfg = {0};
      cfg.g = (kvr_geometry){ .layers = L, .kv_heads = H, .head_dim = D, .dtype_bytes = E, .block_size = BS };
      cfg.num_blocks = NB; cfg.host_capacity_bytes = arena_bytes; cfg.chunk_bytes = slot; cfg.staging_slots = slots;
      cfg.route = KVR_ROUTE_STAGED; cfg.device_pool = dpool; cfg.host_arena = arena; cfg.device_staging = stg;
      for (int i = 0; i < 4; ++i) cfg.streams[i] = st[i];
      cfg.max_moves_in_flight = 2;
      kvr_pool *pool = NULL;
      if (kvr_pool_create(&cfg, &pool) != KVR_OK) { printf("create: %s\n", kvr_last_error()); return 1; }
      int32_t table[16] = {9, 40, 3, 63, 17, 5, 22, 31, 8, 50, 11, 2, 60, 33, 1, 47};
      uint64_t req = 7;
      if (kvr_request_admit_into(pool, req, N, table, 16) != KVR_OK) return 2;
      if (kvr_suspend_to_host(pool, &req, 1, KVR_SYNC, NULL) != KVR_OK) { printf("suspend: %s\n", kvr_last_error()); return 3; }
      const void *img = NULL; uint64_t img_bytes = 0;
      if (kvr_request_info(pool, req, NULL, NULL, NULL, NULL, 0, &img, &img_bytes, NULL) != KVR_OK) return 4;
      if (img_bytes != (uint64_t)N * 2 * L * row) return 5;
      const unsigned char *im = img;
      for (int plane = 0; plane < 2 * L; ++plane)
        for (int t = 0; t < N; ++t)
          if (memcmp(im + ((size_t)plane * N + t) * row, hpool + (((size_t)plane * NB + table[t / BS]) * BS + t % BS) * row, row)) return 6;
      int32_t fresh[16] = {12, 13, 14, 15, 16, 18, 19, 20, 21, 23, 24, 25, 26, 27, 28, 29};
      if (kvr_resume_from_host_into(pool, req, fresh, 16, KVR_SYNC) != KVR_OK) return 7;
      unsigned char *back = malloc(pool_bytes);
      CK(cudaMemcpy(back, dpool, pool_bytes, cudaMemcpyDeviceToHost));
      for (int plane = 0; plane < 2 * L; ++plane)
        for (int t = 0; t < N; ++t)
          if (memcmp(back + (((size_t)plane * NB + fresh[t / BS]) * BS + t % BS) * row,
                     hpool + (((size_t)plane * NB + table[t / BS]) * BS + t % BS) * row, row)) return 8;
      kvr_stats s;
      kvr_pool_stats(pool, &s);
      printf("%llu %lld %lld\n", (unsigned long long)s.bytes_suspended, (long long)s.gather_launches, (long long)s.d2h_copies);
      return kvr_pool_destroy(pool);
    }
    '''
    c = tmp_path / "t.c"
    c.write_text(src)
    exe = tmp_path / "t"
    pkg = os.path.join(root, "paper_2608_30830_b200")
    kvr.lib()
    subprocess.check_call(["gcc", "-std=c11", "-I", os.path.join(root, "include"), "-I", "/usr/local/cuda/include", str(c),
                           "-o", str(exe), "-L", pkg, "-l:libkvr.so", "-Wl,-rpath," + pkg,
                           "-L", "/usr/local/cuda/lib64", "-lcudart", "-Wl,-rpath,/usr/local/cuda/lib64"])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stdout)
    nbytes, launches, copies = (int(x) for x in out.stdout.split())
    assert nbytes == 61 * 2 * 2 * 256 and launches >= 3 and copies >= launches      # 62,464 bytes through 8 KiB slots


def test_a_synchronous_move_does_not_hold_the_pool_against_other_threads():
    """One thread keeps making KVR_SYNC moves of ~190 MiB (about 3.5 ms each on the link); meanwhile a second thread
    does bookkeeping calls on the same pool.  The lock is given up while a call sleeps on GPU work, so the second
    thread's calls must take microseconds, not the length of a move; and every request comes back whole."""
    import threading
    import time
    geom = (8, 8, 128, 2, 16)                      # 32 KiB per token
    bpt = kvr.bytes_per_token(*geom[:4])
    NB, n = 2048, 6000
    dev = torch.empty(NB * 16 * bpt, dtype=torch.uint8, device="cuda")
    dev.view(torch.bfloat16).normal_(generator=torch.Generator(device="cuda").manual_seed(21))
    tiles = dev.view(2 * 8, NB, 16 * 2048)

    def logical(blocks):
        idx = torch.from_numpy(np.asarray(blocks).astype(np.int64)).cuda()
        return tiles.index_select(1, idx).reshape(16, len(blocks) * 16, 2048)[:, :n].cpu().numpy()
    with kvr.Pool(*geom, NB, 3 * n * bpt, device_pool=dev.data_ptr()) as g:
        want = {rid: logical(g.admit(rid, n)[1]) for rid in (1, 2)}
        torch.cuda.synchronize()
        stop, errors, slow = threading.Event(), [], []

        def mover():
            try:
                for _ in range(12):
                    assert g.suspend_to_host([1, 2], kvr.SYNC)[0] == kvr.OK
                    assert g.resume_from_host([2, 1], kvr.SYNC)[0] == kvr.OK
            except Exception as e:
                errors.append(e)
            stop.set()

        def bystander():
            try:
                k = 0
                while not stop.is_set():
                    t0 = time.perf_counter()
                    assert g.admit(100 + k, 40)[0] == kvr.OK
                    assert g.retain_in_hbm([100 + k])[0] == kvr.OK
                    assert g.release(100 + k) == kvr.OK
                    g.stats()
                    slow.append(time.perf_counter() - t0)
                    k += 1
                    time.sleep(0.0002)
            except Exception as e:
                errors.append(e)
        ts = [threading.Thread(target=mover), threading.Thread(target=bystander)]
        for t in ts:
            t.start()
        for t in ts:
            t.join()
        assert not errors, errors
        assert len(slow) > 50
        assert float(np.median(slow)) < 1e-3, np.median(slow)       # a held lock would make every round ~3.5 ms
        assert g.wait() == kvr.OK
        for rid in (1, 2):
            assert np.array_equal(logical(g.info(rid)[1]["blocks"]), want[rid]), rid
        check_invariants(g, [1, 2])


@pytest.mark.parametrize("kernel", [kvr.KERNEL_WARP, kvr.KERNEL_BULK], ids=["warp", "bulk"])
def test_a_table_entry_out_of_range_is_skipped_and_reported(kernel):
    """The movers check every table entry against the pool's block count.  The self-test makes the check fire
    safely (the entry is outside the block count given to the kernel, yet inside the real pool): the tile is skipped,
    the error word says 3, kvr_wait reports it, and after clearing the pool moves data as before."""
    geom = (4, 2, 64, 2, 16)
    t = Twin(geom, 64, 1 << 21, seed=31, kernel=kernel, chunk_bytes=8192, staging_slots=3)
    assert t.g.selftest_block_check() == kvr.OK and t.g.wait() == kvr.OK
    assert t.g.selftest_block_check(leave_error_set=True) == kvr.OK
    assert t.g.wait() == kvr.ERR_CUDA and "status 3" in kvr.last_error()
    assert t.g.clear_device_error() == kvr.OK and t.g.wait() == kvr.OK
    t.both("admit", 1, 300)
    a, b = t.both("suspend_to_host", [1])
    assert a == b
    t.assert_same_images([1])
    a, b = t.both("resume_from_host", [1])
    assert a == b
    t.assert_same_pool()
    t.close()
