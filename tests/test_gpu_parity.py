"""GPU parity: the CUDA library against the CPU oracle, byte for byte, through the C ABI.

Small cases compare every host image and the whole pool; they span several tiles, ragged tails, empty
requests, chunk boundaries that cut requests, more requests than one launch holds, both routes and both
kernels, and un-synchronised call sequences whose hazards the library must order itself."""
import numpy as np
import pytest
import torch

import oracle as orc
from common import check_invariants, random_script, run_script
from kvr_synth import CONFIGS, context_lengths, free_order
from paper_2608_30830_b200 import kvr

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

from gpu_common import Twin  # noqa: E402

MODES = [
    pytest.param(dict(route=kvr.ROUTE_STAGED, kernel=kvr.KERNEL_WARP), id="staged-warp"),
    pytest.param(dict(route=kvr.ROUTE_STAGED, kernel=kvr.KERNEL_BULK), id="staged-bulk"),
    pytest.param(dict(route=kvr.ROUTE_MAPPED, kernel=kvr.KERNEL_WARP), id="mapped-warp"),
    pytest.param(dict(route=kvr.ROUTE_MAPPED, kernel=kvr.KERNEL_BULK), id="mapped-bulk"),
    pytest.param(dict(route=kvr.ROUTE_STAGED, kernel=kvr.KERNEL_BULK, layout=kvr.BLOCK_MAJOR), id="staged-bulk-blockmajor"),
    pytest.param(dict(route=kvr.ROUTE_MAPPED, kernel=kvr.KERNEL_WARP, layout=kvr.BLOCK_MAJOR), id="mapped-warp-blockmajor"),
    pytest.param(dict(route=kvr.ROUTE_DMA2D), id="dma2d"),
    pytest.param(dict(route=kvr.ROUTE_DMA2D, layout=kvr.BLOCK_MAJOR), id="dma2d-blockmajor"),
]
SMALL = (3, 2, 16, 2, 8)          # L, H, D, e, BS: 64-byte rows, 512-byte tiles, 384 bytes per token
LENGTHS = [0, 1, 7, 8, 9, 64, 67, 200, 3, 16]


@pytest.mark.parametrize("mode", MODES)
def test_suspend_then_resume_small(mode):
    t = Twin(SMALL, 128, 1 << 22, seed=1, chunk_bytes=4096, staging_slots=2, **mode)
    ids = list(range(len(LENGTHS)))
    for rid, n in zip(ids, LENGTHS):
        a, b = t.both("admit", rid, n)
        assert a[0] == b[0] == orc.OK and a[1].tolist() == b[1].tolist()
    a, b = t.both("suspend_to_host", ids)
    assert a == b
    t.assert_same_images(ids)
    t.assert_same_pool()                                  # a suspend does not touch the pool
    a, b = t.both("resume_from_host", ids)
    assert a == b
    for rid in ids:
        assert t.o.info(rid)[1]["blocks"].tolist() == t.g.info(rid)[1]["blocks"].tolist()
    t.assert_same_pool()                                  # only valid slots of the new blocks changed
    check_invariants(t.g, ids)
    s = t.g.stats()
    if mode.get("route") == kvr.ROUTE_DMA2D:
        assert s["gather_launches"] == s["scatter_launches"] == 0 and s["d2h_bytes"] == s["h2d_bytes"] == sum(LENGTHS) * 384
    else:
        assert s["gather_launches"] >= 1 and s["scatter_launches"] >= 1
        assert s["gather_bytes"] == s["scatter_bytes"] == sum(LENGTHS) * 384
    t.close()


@pytest.mark.parametrize("mode", MODES[:2] + MODES[4:5])
def test_export_import_kernels_alone(mode):
    """gather and scatter kernels HBM to HBM, against the oracle's per-element loops."""
    t = Twin(SMALL, 96, 0, seed=2, **mode)
    L, H, D, e, BS = SMALL
    ids = list(range(len(LENGTHS)))
    tables = {}
    for rid, n in zip(ids, LENGTHS):
        tables[rid] = t.g.admit(rid, n)[1]
        t.o.admit(rid, n)
    cap = sum(-(-n * 384 // 256) * 256 for n in LENGTHS) + 256
    buf = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    st, offs = t.g.export_to_device(ids, buf.data_ptr(), cap, kvr.SYNC)
    assert st == kvr.OK, kvr.last_error()
    host = buf.cpu().numpy()
    for rid, n, off in zip(ids, LENGTHS, offs):
        want = orc.gather(t.o.data, L, H, D, e, BS, t.NB, tables[rid], n, layout=t.layout)
        assert off % 256 == 0 and np.array_equal(host[int(off):int(off) + want.size], want)
    # scatter new content back through the same tables
    new = np.random.default_rng(5).integers(0, 256, size=cap, dtype=np.uint8)
    buf.copy_(torch.from_numpy(new))
    torch.cuda.synchronize()
    st, offs2 = t.g.import_from_device(ids, buf.data_ptr(), cap, kvr.SYNC)
    assert st == kvr.OK and offs2.tolist() == offs.tolist()
    for rid, n, off in zip(ids, LENGTHS, offs):
        orc.scatter(t.o.data, new[int(off):int(off) + n * 384], L, H, D, e, BS, t.NB, tables[rid], n, layout=t.layout)
    t.assert_same_pool()
    assert t.g.export_to_device(ids, buf.data_ptr(), 100)[0] == kvr.ERR_INVALID_ARG
    t.close()


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_random_scripts_with_data(mode, seed):
    """Seeded call scripts (legal and illegal calls, HOST_FULL, HBM_FULL, relabelling) with no waits between
    calls: statuses, tables, offsets, every host image at the end and the final pool must equal the oracle's."""
    NB, cap = 48, 10 * 4096
    t = Twin(SMALL, NB, cap, seed=seed, chunk_bytes=4096, staging_slots=2, **mode)
    ops = random_script(100 + seed, 300, max_tokens=70)
    la = run_script(t.o, ops)
    lb = run_script(t.g, ops)
    for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(la, lb):
        assert (sa, pa) == (sb, pb) and snap_a == snap_b, op
    t.assert_same_images(range(12))
    t.assert_same_pool()
    check_invariants(t.g, range(12))
    t.close()


@pytest.mark.parametrize("mode", MODES[:2])
def test_images_checked_after_every_move(mode):
    NB, cap = 48, 12 * 4096
    t = Twin(SMALL, NB, cap, seed=7, chunk_bytes=8192, staging_slots=3, **mode)
    ops = random_script(7, 120, max_tokens=70)

    def after(op, st):
        if op[0] in ("suspend", "resume", "resume_into"):
            t.assert_same_images(range(12))
    # run the oracle one call ahead of the library so images can be compared after each library call
    lo = []
    for op in ops:
        lo += run_script(t.o, [op])
        lg = run_script(t.g, [op], after_each=after)
        assert lo[-1][1:] == lg[-1][1:], op
    t.assert_same_pool()
    t.close()


@pytest.mark.parametrize("kernel", [kvr.KERNEL_WARP, kvr.KERNEL_BULK])
def test_more_requests_than_one_launch_holds(kernel):
    geom = (1, 1, 16, 1, 2)                                # 16-byte rows, 32-byte tiles
    n_req = 1100 * 2 + 7
    t = Twin(geom, 8192, 1 << 24, seed=3, kernel=kernel, chunk_bytes=1 << 20)
    rng = np.random.default_rng(3)
    ids = list(range(n_req))
    for rid in ids:
        n = int(rng.integers(0, 6))
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b
    t.assert_same_images(ids)
    a, b = t.both("resume_from_host", ids)
    assert a == b
    t.assert_same_pool()
    t.close()


def test_hazards_without_waiting():
    """Blocks freed by a suspend are taken by the next resume, host ranges freed by a resume are taken by the
    next suspend, the same request is moved again while its last move is in flight: no wait in between."""
    geom = (4, 2, 64, 2, 16)                               # 256-byte rows, 4 KiB tiles, 2 KiB per token
    NB = 64
    t = Twin(geom, NB, 3 << 20, seed=9, chunk_bytes=16384, staging_slots=2)
    lens = [300, 257, 131, 16]                             # 19 + 17 + 9 + 1 = 46 of 64 blocks
    for rid, n in enumerate(lens):
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    for rnd in range(6):
        a, b = t.both("suspend_to_host", [0, 1])
        assert a == b
        a, b = t.both("resume_from_host", [1, 0])          # takes blocks the suspend just released
        assert a == b
        a, b = t.both("suspend_to_host", [2, 3, 0])        # request 0 again, its resume still in flight
        assert a == b
        a, b = t.both("resume_from_host", [0, 2, 3])
        assert a == b
    for rid in range(4):
        assert t.o.info(rid)[1]["blocks"].tolist() == t.g.info(rid)[1]["blocks"].tolist()
    t.assert_same_pool()
    t.close()


def test_transient_states_and_latency():
    geom = (4, 2, 64, 2, 16)
    t = Twin(geom, 64, 1 << 21, seed=4)
    t.both("admit", 1, 200)
    assert t.g.latency(1)[0] == kvr.ERR_BAD_STATE
    t.g.suspend_to_host([1])
    t.o.suspend_to_host([1])
    st = t.g.info(1)[1]["state"]
    assert st in (kvr.SUSPENDING, kvr.HOST)
    assert t.g.wait(1) == kvr.OK and t.g.info(1)[1]["state"] == kvr.HOST
    st, host_ms, dev_ms = t.g.latency(1)
    assert st == kvr.OK and host_ms > 0 and dev_ms > 0
    t.g.resume_from_host([1], kvr.SYNC)
    t.o.resume_from_host([1])
    assert t.g.info(1)[1]["state"] == kvr.ACTIVE
    assert t.g.wait(99) == kvr.ERR_UNKNOWN_REQUEST
    t.assert_same_pool()
    t.close()


def test_fp8_sized_elements():
    """dtype_bytes = 1 (fp8 KV): 1 KiB rows; the movers are byte-exact whatever the element type."""
    geom = (4, 8, 128, 1, 16)
    t = Twin(geom, 96, 1 << 22, seed=12, chunk_bytes=1 << 16)
    lens = [100, 257, 16, 1]
    for rid, n in enumerate(lens):
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    assert kvr.bytes_per_token(4, 8, 128, 1) == 8192
    ids = list(range(len(lens)))
    a, b = t.both("suspend_to_host", ids)
    assert a == b
    t.assert_same_images(ids)
    a, b = t.both("resume_from_host", ids)
    assert a == b
    t.assert_same_pool()
    t.close()


def test_strided_copy_route_rejects_an_oversized_pitch():
    # layer-major plane stride = num_blocks x tile; beyond the device's copy pitch limit the route is refused
    with pytest.raises(kvr.KvrError) as e:
        kvr.Pool(1, 8, 128, 2, 16, 1 << 17, 0, route=kvr.ROUTE_DMA2D, device_pool=256)
    assert e.value.status == kvr.ERR_GEOMETRY and "pitch" in str(e.value)


def test_wait_is_bounded():
    """kvr_wait with a zero budget on a move that is still in flight answers KVR_ERR_TIMEOUT at once and leaves
    the move alone; a later wait sees it finish."""
    geom = (32, 8, 128, 2, 16)
    n = 4096                                                 # 512 MiB image: ~9 ms on the link
    bpt = kvr.bytes_per_token(*geom[:4])
    dev = torch.zeros(512 * 16 * bpt, dtype=torch.uint8, device="cuda")
    with kvr.Pool(*geom, 512, n * bpt + 4096, device_pool=dev.data_ptr()) as g:
        assert g.admit(1, n)[0] == kvr.OK
        assert g.suspend_to_host([1])[0] == kvr.OK
        st = g.wait(1, 0)
        assert st in (kvr.ERR_TIMEOUT, kvr.OK)
        if st == kvr.ERR_TIMEOUT:
            assert "in flight" in kvr.last_error() and g.info(1)[1]["state"] == kvr.SUSPENDING
        assert g.wait(1, 10000) == kvr.OK and g.info(1)[1]["state"] == kvr.HOST
        assert g.stats()["ops_in_flight"] == 0


def test_caller_owned_pinned_arena_and_grid_cap():
    geom = (4, 2, 64, 2, 16)
    cap = 1 << 21
    arena = torch.empty(cap + 4096, dtype=torch.uint8).pin_memory()
    base = (arena.data_ptr() + 4095) // 4096 * 4096
    t = Twin(geom, 64, cap, seed=6, host_arena=base, max_ctas=3, chunk_bytes=65536)
    t.both("admit", 1, 500)
    t.both("admit", 2, 123)
    assert t.both("suspend_to_host", [1, 2])[1][0] == kvr.OK
    t.assert_same_images([1, 2])
    assert t.g.host_arena_ptr == base
    t.both("resume_from_host", [2, 1])
    t.assert_same_pool()
    t.close()


def test_tiny_config_full_size():
    """The benchmark's smallest configuration at full size: whole pool and every image compared."""
    w = CONFIGS["tiny"]
    seed = 20260830
    order = free_order(seed, w.num_blocks)
    lens = context_lengths(w.length_rule, w.n_requests, seed)
    t = Twin(w.geom, w.num_blocks, 1 << 28, seed=seed, order=order, flags=kvr.PROFILE)
    ids = list(range(w.n_requests))
    for rid, n in zip(ids, lens):
        assert t.both("admit", rid, int(n))[1][0] == kvr.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b == (kvr.OK, [kvr.OK] * 4)
    t.assert_same_images(ids)
    a, b = t.both("resume_from_host", ids)
    assert a == b
    t.assert_same_pool()
    s = t.g.stats()
    assert s["bytes_suspended"] == s["bytes_resumed"] == int(lens.sum()) * 32768
    assert s["gather_ms"] > 0 and s["scatter_ms"] > 0
    # the kernels' own stamps: a positive time, shorter than what the events around the launches saw
    assert 0 < s["gather_kernel_ms"] < s["gather_ms"] and 0 < s["scatter_kernel_ms"] < s["scatter_ms"]
    t.close()


@pytest.mark.parametrize("route", [kvr.ROUTE_MAPPED, kvr.ROUTE_STAGED, kvr.ROUTE_DMA2D], ids=["direct", "staged", "strided"])
def test_arena_in_device_memory(route):
    """The second tier may be device memory (a stand-in here for a peer GPU's HBM reached over NVLink): same
    bookkeeping, same image bytes, read back from the device arena."""
    geom = (4, 2, 64, 2, 16)
    cap = 1 << 21
    arena = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    t = Twin(geom, 96, cap, seed=15, host_arena=arena.data_ptr(), route=route, chunk_bytes=65536)
    lens = [500, 123, 16, 0, 77]
    ids = list(range(len(lens)))
    for rid, n in zip(ids, lens):
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b and t.g.wait() == kvr.OK
    dev_arena = arena.cpu().numpy()
    for rid in ids:
        d = t.o.info(rid)[1]
        off = t.g.info(rid)[1]["arena_offset"]
        assert off == d["arena_offset"]
        assert np.array_equal(dev_arena[off:off + d["image_bytes"]], d["image"])
    a, b = t.both("resume_from_host", ids[::-1])
    assert a == b
    t.assert_same_pool()
    t.close()


@pytest.mark.parametrize("route", [kvr.ROUTE_STAGED, kvr.ROUTE_MAPPED])
def test_arena_in_a_peer_gpus_memory(route):
    """The same with the arena on another GPU (the peer-HBM tier over NVLink): the library enables peer access, the
    copies follow the pointer and the direct route's kernels use plain loads, stores and single-CTA bulk copies.
    Needs two GPUs: skipped on a one-GPU machine."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    if not torch.cuda.can_device_access_peer(0, 1):
        pytest.skip("GPU 0 cannot address GPU 1")
    geom = (4, 2, 64, 2, 16)
    cap = 1 << 21
    arena = torch.zeros(cap, dtype=torch.uint8, device="cuda:1")
    torch.cuda.synchronize(1)
    t = Twin(geom, 96, cap, seed=15, host_arena=arena.data_ptr(), route=route, chunk_bytes=65536, staging_slots=3)
    lens = [500, 123, 16, 0, 77]
    ids = list(range(len(lens)))
    for rid, n in zip(ids, lens):
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b and t.g.wait() == kvr.OK
    peer = arena.cpu().numpy()
    for rid in ids:
        d = t.o.info(rid)[1]
        off = t.g.info(rid)[1]["arena_offset"]
        assert off == d["arena_offset"] and np.array_equal(peer[off:off + d["image_bytes"]], d["image"])
    a, b = t.both("resume_from_host", ids[::-1])
    assert a == b
    t.assert_same_pool()
    t.close()


@pytest.mark.parametrize("mode", MODES)
def test_guard_bands_stay_intact(mode):
    """Canary regions directly before and after the caller-owned pool and arena must survive a busy script:
    nothing the movers or the copies do may land outside the two buffers."""
    geom = SMALL
    NB, cap, guard = 48, 10 * 4096, 4096
    bpt = kvr.bytes_per_token(*geom[:4])
    pool_bytes = NB * geom[4] * bpt
    dev = torch.full((pool_bytes + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    host = torch.full((cap + 2 * guard + 4096,), 0x5A, dtype=torch.uint8).pin_memory()
    hbase = (host.data_ptr() + guard + 255) // 256 * 256
    hoff = hbase - host.data_ptr()
    order = np.random.default_rng(8).permutation(NB).astype(np.int32)
    g = kvr.Pool(*geom, NB, cap, initial_free_order=order, device_pool=dev.data_ptr() + guard, host_arena=hbase,
                 chunk_bytes=4096, staging_slots=2, **mode)
    o = orc.OrcPool(*geom, NB, cap, initial_free_order=order, with_data=False, layout=mode.get("layout", 0))
    ops = random_script(8, 250, max_tokens=70)
    la, lb = run_script(o, ops), run_script(g, ops)
    assert [x[1:3] for x in la] == [x[1:3] for x in lb]
    assert g.wait() == kvr.OK
    torch.cuda.synchronize()
    d = dev.cpu().numpy()
    assert (d[:guard] == 0x5A).all() and (d[guard + pool_bytes:] == 0x5A).all()
    h = host.numpy()
    assert (h[:hoff] == 0x5A).all() and (h[hoff + cap:] == 0x5A).all()
    assert g.stats()["bytes_suspended"] > 0
    g.close()


def test_library_owned_pool_and_arena():
    """device_pool = NULL and host_arena = NULL: the library allocates both.  Content goes in through
    kvr_import_from_device, so the host image of a request must be exactly the linear bytes that were imported
    (scatter then gather by the same table is the identity on valid tokens, as the oracle's own round trip shows)."""
    geom = (4, 8, 128, 2, 16)
    bpt = kvr.bytes_per_token(*geom[:4])
    with kvr.Pool(*geom, 300, 64 << 20, initial_free_order=np.random.default_rng(2).permutation(300)) as g:
        assert g.device_ptr and g.host_arena_ptr
        lens = [1000, 37, 512]
        ids = [1, 2, 3]
        for rid, n in zip(ids, lens):
            assert g.admit(rid, n)[0] == kvr.OK
        cap = sum(-(-n * bpt // 256) * 256 for n in lens)
        src = torch.randint(0, 256, (cap,), dtype=torch.uint8, device="cuda", generator=torch.Generator(device="cuda").manual_seed(4))
        torch.cuda.synchronize()
        st, offs = g.import_from_device(ids, src.data_ptr(), cap, kvr.SYNC)
        assert st == kvr.OK, kvr.last_error()
        host_src = src.cpu().numpy()
        assert g.suspend_to_host(ids, kvr.SYNC)[0] == kvr.OK
        for rid, n, off in zip(ids, lens, offs):
            assert np.array_equal(g.host_image(rid), host_src[int(off):int(off) + n * bpt])
        assert g.resume_from_host(ids[::-1], kvr.SYNC)[0] == kvr.OK
        out = torch.zeros(cap, dtype=torch.uint8, device="cuda")
        st, offs2 = g.export_to_device(ids, out.data_ptr(), cap, kvr.SYNC)
        assert st == kvr.OK and offs2.tolist() == offs.tolist()
        got = out.cpu().numpy()
        for n, off in zip(lens, offs):
            assert np.array_equal(got[int(off):int(off) + n * bpt], host_src[int(off):int(off) + n * bpt])


@pytest.mark.parametrize("geom", [(2, 8, 128, 2, 16), (8, 2, 128, 2, 16), (16, 1, 128, 1, 16)], ids=["tile32k", "tile8k", "tile2k"])
@pytest.mark.parametrize("mode", [MODES[1], MODES[3], MODES[6]])
def test_random_scripts_with_moves_that_stay_in_flight(mode, geom):
    """The same seeded scripts on images of tens of MiB, so that calls really do arrive while earlier moves are
    still on the link: bookkeeping as observed (including reported states) and all bytes must still equal the oracle's.
    Tiles of 32, 8 and 2 KiB: the movers claim one, four and sixteen units of work at a time."""
    t = Twin(geom, 2048, 300 << 20, seed=2, chunk_bytes=64 << 20, staging_slots=2, **mode)
    ops = random_script(2002, 160, max_tokens=6000, n_ids=12, batch=4)
    la, lb = run_script(t.o, ops), run_script(t.g, ops)
    for (op, sa, pa, snap_a), (_, sb, pb, snap_b) in zip(la, lb):
        assert (sa, pa) == (sb, pb) and snap_a == snap_b, op
    t.assert_same_images(range(12))
    t.assert_same_pool()
    t.close()


def test_retained_while_resuming_reports_retained():
    geom = (32, 8, 128, 2, 16)
    bpt = kvr.bytes_per_token(*geom[:4])
    dev = torch.zeros(1024 * 16 * bpt, dtype=torch.uint8, device="cuda")
    with kvr.Pool(*geom, 1024, (4096 * bpt) + 4096, device_pool=dev.data_ptr()) as g:
        assert g.admit(1, 4096)[0] == kvr.OK
        assert g.suspend_to_host([1], kvr.SYNC)[0] == kvr.OK
        assert g.resume_from_host([1])[0] == kvr.OK            # ~9 ms on the link
        assert g.info(1)[1]["state"] in (kvr.RESUMING, kvr.ACTIVE)
        assert g.retain_in_hbm([1])[0] == kvr.OK               # legal at once: the bookkeeping is settled
        assert g.info(1)[1]["state"] == kvr.RETAINED
        assert g.wait(1) == kvr.OK and g.info(1)[1]["state"] == kvr.RETAINED


def test_admit_waits_for_the_gather_that_still_reads_its_blocks():
    """A suspend is enqueued and, with no wait, a new request is admitted into exactly the blocks it released and the
    caller overwrites them at once.  kvr_request_admit must have let the gather finish first: the host image has to
    hold the old bytes."""
    geom = (32, 8, 128, 2, 16)
    bpt = kvr.bytes_per_token(*geom[:4])
    NB, n = 512, 4096                                       # 256 blocks = 512 MiB per request
    dev = torch.empty(NB * 16 * bpt, dtype=torch.uint8, device="cuda")
    dev.view(torch.bfloat16).normal_(generator=torch.Generator(device="cuda").manual_seed(3))
    tiles = dev.view(2 * 32, NB, 16 * 2048)
    with kvr.Pool(*geom, NB, n * bpt + 4096, device_pool=dev.data_ptr(), chunk_bytes=32 << 20) as g:
        a = g.admit(1, n)[1]
        assert g.admit(2, n)[0] == kvr.OK and g.stats()["blocks_free"] == 0
        idx = torch.from_numpy(a.astype(np.int64)).cuda()
        want = tiles.index_select(1, idx).reshape(64, n * 2048).cpu().numpy().reshape(-1)   # the image, by definition
        torch.cuda.synchronize()
        assert g.suspend_to_host([1])[0] == kvr.OK           # ~9 ms of link time, gather chunks spread over it
        st, c = g.admit(3, n)                                # takes the 256 blocks just released
        assert st == kvr.OK and sorted(c.tolist()) == sorted(a.tolist())
        tiles[:, idx] = 0xFF                                 # the caller's prefill, on its own stream
        torch.cuda.synchronize()
        assert g.wait() == kvr.OK
        assert np.array_equal(g.host_image(1), want)


def test_suspend_into_a_host_range_that_a_resume_is_still_reading():
    """The arena holds one image.  A resume releases the range at once (bookkeeping) while its copies are still
    reading it; the next suspend is placed on the same bytes with no wait in between and must not overwrite them early."""
    geom = (32, 8, 128, 2, 16)
    bpt = kvr.bytes_per_token(*geom[:4])
    NB, n = 768, 4096
    dev = torch.empty(NB * 16 * bpt, dtype=torch.uint8, device="cuda")
    dev.view(torch.bfloat16).normal_(generator=torch.Generator(device="cuda").manual_seed(5))
    tiles = dev.view(2 * 32, NB, 16 * 2048)

    def logical(blocks):
        idx = torch.from_numpy(np.asarray(blocks).astype(np.int64)).cuda()
        return tiles.index_select(1, idx).reshape(64, n * 2048).cpu().numpy().reshape(-1)
    for route in (kvr.ROUTE_STAGED, kvr.ROUTE_MAPPED, kvr.ROUTE_DMA2D):
        with kvr.Pool(*geom, NB, n * bpt, device_pool=dev.data_ptr(), route=route, chunk_bytes=32 << 20) as g:
            a, b = g.admit(1, n)[1], g.admit(2, n)[1]
            want_a, want_b = logical(a), logical(b)
            assert g.suspend_to_host([1], kvr.SYNC)[0] == kvr.OK and g.info(1)[1]["arena_offset"] == 0
            assert g.suspend_to_host([2])[0] == kvr.HOST_FULL                      # one image fills the tier
            assert g.resume_from_host([1])[0] == kvr.OK                            # reads [0, 512 MiB) for ~9 ms
            assert g.suspend_to_host([2])[0] == kvr.OK and g.info(2)[1]["arena_offset"] == 0
            assert g.wait() == kvr.OK
            assert np.array_equal(logical(g.info(1)[1]["blocks"]), want_a)         # request 1 came back whole
            assert np.array_equal(g.host_image(2), want_b)


def test_probe_link_measures_the_arena_and_refuses_when_it_holds_images():
    geom = (4, 8, 128, 2, 16)
    with kvr.Pool(*geom, 64, 64 << 20) as g:
        st, d2h, h2d = g.probe_link(32 << 20, 3)
        assert st == kvr.OK and 1.0 < d2h < 200.0 and 1.0 < h2d < 200.0      # a PCIe link, in GB/s
        g.admit(1, 100)
        assert g.suspend_to_host([1], kvr.SYNC)[0] == kvr.OK
        assert g.probe_link(32 << 20, 3)[0] == kvr.ERR_BAD_STATE
    with kvr.Pool(*geom, 64, 0) as g:
        assert g.probe_link()[0] == kvr.ERR_BAD_STATE                         # no arena at all


def test_two_threads_move_their_own_requests_concurrently():
    """Two caller threads suspend and resume disjoint requests on one pool at the same time.  Which blocks and host
    ranges each move gets depends on the interleaving, so the check is on content: every request comes back whole."""
    import threading
    geom = (8, 8, 128, 2, 16)                      # 32 KiB per token
    bpt = kvr.bytes_per_token(*geom[:4])
    NB, n = 1024, 1500                             # 94 blocks, 47 MiB per request
    dev = torch.empty(NB * 16 * bpt, dtype=torch.uint8, device="cuda")
    dev.view(torch.bfloat16).normal_(generator=torch.Generator(device="cuda").manual_seed(9))
    tiles = dev.view(2 * 8, NB, 16 * 2048)

    def logical(blocks):
        idx = torch.from_numpy(np.asarray(blocks).astype(np.int64)).cuda()
        full = tiles.index_select(1, idx).reshape(16, len(blocks) * 16, 2048)[:, :n]
        return full.cpu().numpy()
    with kvr.Pool(*geom, NB, 8 * n * bpt, device_pool=dev.data_ptr(), chunk_bytes=16 << 20,
                  initial_free_order=np.random.default_rng(9).permutation(NB)) as g:
        ids = list(range(8))
        want = {rid: logical(g.admit(rid, n)[1]) for rid in ids}
        torch.cuda.synchronize()
        errors = []

        def worker(mine):
            try:
                for _ in range(6):
                    assert g.suspend_to_host(mine)[0] == kvr.OK
                    assert g.resume_from_host(mine[::-1])[0] == kvr.OK
                for rid in mine:
                    assert g.wait(rid, 20000) == kvr.OK
            except Exception as e:
                errors.append(e)
        threads = [threading.Thread(target=worker, args=(ids[:4],)), threading.Thread(target=worker, args=(ids[4:],))]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
        assert not errors, errors
        assert g.wait() == kvr.OK
        for rid in ids:
            assert np.array_equal(logical(g.info(rid)[1]["blocks"]), want[rid]), rid
        check_invariants(g, ids)


@pytest.mark.parametrize("mode", MODES[:4])
def test_tiles_larger_than_one_bulk_piece(mode):
    """block_size 64 with 2 KiB rows gives 128 KiB tiles: the bulk mover cuts each into four 32 KiB pieces, and a
    ragged last block leaves some pieces short or empty."""
    geom = (2, 8, 128, 2, 64)
    t = Twin(geom, 64, 8 << 20, seed=17, chunk_bytes=1 << 20, **mode)
    lens = [100, 64, 1, 65, 17, 0, 127, 640]
    ids = list(range(len(lens)))
    for rid, n in zip(ids, lens):
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b
    t.assert_same_images(ids)
    a, b = t.both("resume_from_host", ids[::-1])
    assert a == b
    t.assert_same_pool()
    t.close()


@pytest.mark.parametrize("geom", [(3, 1, 24, 2, 5), (2, 3, 40, 4, 3), (1, 1, 8, 2, 1)], ids=["row48", "row480-f32", "row16-bs1"])
@pytest.mark.parametrize("mode", MODES[:3])
def test_odd_geometries(geom, mode):
    """Rows that are multiples of 16 bytes but of nothing larger, odd block sizes, 4-byte elements."""
    t = Twin(geom, 97, 1 << 20, seed=19, chunk_bytes=4096, **mode)
    rng = np.random.default_rng(19)
    lens = [int(x) for x in rng.integers(0, 9 * geom[4], size=9)]
    ids = list(range(len(lens)))
    for rid, n in zip(ids, lens):
        assert t.both("admit", rid, n)[1][0] == kvr.OK
    a, b = t.both("suspend_to_host", ids)
    assert a == b
    t.assert_same_images(ids)
    a, b = t.both("resume_from_host", ids[::-1])
    assert a == b
    t.assert_same_pool()
    t.close()


def test_an_arena_larger_than_host_memory_is_refused_politely():
    avail = int(open("/proc/meminfo").read().split("MemAvailable:")[1].split()[0]) * 1024
    with pytest.raises(kvr.KvrError) as e:
        kvr.Pool(4, 8, 128, 2, 16, 64, 4 * avail)
    assert e.value.status == kvr.ERR_NOMEM


def test_a_wait_that_runs_out_is_reported_and_the_pool_stays_usable():
    """The give-up path of the movers, made to happen safely: a thread polls a barrier nothing completes, gives up
    after its limit, writes the error word; kvr_wait reports it; after clearing, moves work as before."""
    geom = (4, 2, 64, 2, 16)
    t = Twin(geom, 64, 1 << 21, seed=23)
    assert t.g.selftest_bounded_wait() == kvr.OK and t.g.wait() == kvr.OK            # word cleared by the self-test
    assert t.g.selftest_bounded_wait(leave_error_set=True) == kvr.OK
    assert t.g.wait() == kvr.ERR_CUDA and "bounded wait" in kvr.last_error()
    assert t.g.clear_device_error() == kvr.OK and t.g.wait() == kvr.OK
    t.both("admit", 1, 300)
    a, b = t.both("suspend_to_host", [1])
    assert a == b
    t.assert_same_images([1])
    a, b = t.both("resume_from_host", [1])
    assert a == b
    t.assert_same_pool()
    t.close()


def test_low_latency_resume_completes_requests_one_by_one():
    """Same bytes and bookkeeping with KVR_LOW_LATENCY; every request is complete as soon as its own bytes are in:
    in order, the first long before the last, none later than under the default plan (where requests that share a
    chunk finish together)."""
    geom = (8, 8, 128, 2, 16)                      # 32 KiB per token
    t = Twin(geom, 512, 256 << 20, seed=29, chunk_bytes=256 << 20, staging_slots=2)
    ids = [0, 1, 2, 3]
    for rid in ids:
        assert t.both("admit", rid, 1500)[1][0] == kvr.OK        # 47 MiB each: all four fit one 256 MiB chunk
    lat = {}
    for flags in (0, kvr.LOW_LATENCY):
        assert t.o.suspend_to_host(ids) == t.g.suspend_to_host(ids, kvr.SYNC)
        assert t.o.resume_from_host(ids) == t.g.resume_from_host(ids, flags)
        assert t.g.wait() == kvr.OK
        lat[flags] = [t.g.latency(r)[2] for r in ids]
        t.assert_same_pool()
    for a, b in zip(lat[kvr.LOW_LATENCY], lat[0]):                   # never later than under the default plan
        assert a <= 1.2 * b + 0.3
    assert lat[kvr.LOW_LATENCY][0] < 0.5 * lat[kvr.LOW_LATENCY][3]   # one by one, in order
    assert sorted(lat[kvr.LOW_LATENCY]) == lat[kvr.LOW_LATENCY]
    t.close()
