"""The mixed tiering trace (retain / suspend / expire / resume events) on the GPU.

Small geometry: the CPU oracle carries the data too, so every host image and the final pool are compared byte for
byte.  Full geometry (Llama-3-8B-shaped KV, 256 requests, 48 GiB pool): the oracle carries the bookkeeping only and
is compared call by call; the data is checked by content -- every admitted request's blocks are stamped with a
pattern that encodes (request, plane, logical block, position), and the pattern must be intact, under the new
block table, whenever a request comes back from the host."""
import numpy as np
import pytest
import torch

import oracle as orc
from common import check_invariants
from gpu_common import Twin
from kvr_synth import CONFIGS, context_lengths, event_trace
from paper_2608_30830_b200 import kvr
from trace_driver import TraceRunner, host_ttl, mixture_mean

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


def thresholds(lengths, bpt, host_cap):
    c2 = host_cap / (float(np.mean(lengths)) * bpt)
    w_ref = mixture_mean()
    lam = 2 * c2 / w_ref                          # the paper's 2 x lambda_crit operating point
    return lam, host_ttl(lam, c2, w_ref)


class _RandomSync:
    """The library pool with a seeded mix of call styles: moves are synchronous or left in flight, resumes ask for
    low latency or not, and now and then the caller waits for everything.  Results must not depend on any of it."""

    def __init__(self, pool, seed):
        self._pool, self._rng = pool, np.random.default_rng(seed)

    def suspend_to_host(self, ids):
        return self._pool.suspend_to_host(ids, kvr.SYNC if self._rng.random() < 0.4 else 0)

    def resume_from_host(self, ids):
        flags = (kvr.SYNC if self._rng.random() < 0.4 else 0) | (kvr.LOW_LATENCY if self._rng.random() < 0.5 else 0)
        return self._pool.resume_from_host(ids, flags)

    def admit(self, rid, n):
        if self._rng.random() < 0.1:
            assert self._pool.wait() == kvr.OK
        return self._pool.admit(rid, n)

    def __getattr__(self, name):
        return getattr(self._pool, name)


@pytest.mark.parametrize("style", ["in-flight", "random-sync"])
@pytest.mark.parametrize("mode", [dict(route=kvr.ROUTE_STAGED, kernel=kvr.KERNEL_BULK),
                                  dict(route=kvr.ROUTE_MAPPED, kernel=kvr.KERNEL_WARP)], ids=["staged-bulk", "mapped-warp"])
def test_trace_small_geometry_with_data(mode, style):
    geom = (2, 2, 16, 2, 4)                        # 64-byte rows, 256 bytes per token
    n_req, NB, host_cap = 160, 130, 160 * 4096
    lengths = context_lengths(("lognormal", 64, 0.6, 4, 400), n_req, 21)
    lam, ttl = thresholds(lengths, 256, host_cap)
    events, _ = event_trace(n_req, 21, lam, 60.0, ttl)
    t = Twin(geom, NB, host_cap, seed=21, chunk_bytes=8192, staging_slots=2 if style == "in-flight" else 5, **mode)
    rng = np.random.default_rng(21)
    L, H, D, e, BS = geom
    o_view = t.o.data.reshape(2 * L, NB, BS * H * D * e)
    d_view = t.dev.view(2 * L, NB, BS * H * D * e)

    def fill(rid, blocks, n):                      # new content for every admission, same bytes on both sides
        if len(blocks) == 0:
            return
        fresh = rng.integers(0, 256, size=(2 * L, len(blocks), BS * H * D * e), dtype=np.uint8)
        o_view[:, blocks] = fresh
        d_view[:, torch.from_numpy(blocks.astype(np.int64)).cuda()] = torch.from_numpy(fresh).cuda()
        torch.cuda.synchronize()

    def after(name, args):
        if name == "suspend_to_host":
            t.assert_same_images(args[0])
    lib_pool = t.g if style == "in-flight" else _RandomSync(t.g, 5)
    counts = TraceRunner([t.o, lib_pool], lengths, fill=fill, after_call=after).run(events)
    for k in ("offloaded", "resumed_resident", "resumed_from_host", "recomputed", "ttl_expired", "demoted"):
        assert counts.get(k, 0) > 0, (k, counts)
    t.assert_same_pool()
    check_invariants(t.g, range(n_req))
    t.close()


def test_config4_trace_full_geometry():
    w = CONFIGS["trace"]
    seed = 20260830 + 3
    L, H, D, e, BS = w.geom
    bpt = kvr.bytes_per_token(L, H, D, e)
    lengths = context_lengths(w.length_rule, w.n_requests, seed)
    host_cap = 32 << 30
    lam, ttl = thresholds(lengths, bpt, host_cap)
    events, _ = event_trace(w.n_requests, seed, lam, 60.0, ttl)
    NB = w.num_blocks
    tile_words = BS * H * D * e // 8
    dev = torch.zeros(NB * BS * bpt // 8, dtype=torch.int64, device="cuda")
    view = dev.view(2 * L, NB, tile_words)
    order = np.random.default_rng(seed).permutation(NB).astype(np.int32)
    o = orc.OrcPool(*w.geom, NB, host_cap, initial_free_order=order, with_data=False)
    g = kvr.Pool(*w.geom, NB, host_cap, initial_free_order=order, device_pool=dev.data_ptr())
    plane_ix = torch.arange(2 * L, device="cuda", dtype=torch.int64).view(-1, 1, 1)
    word_ix = torch.arange(tile_words, device="cuda", dtype=torch.int64).view(1, 1, -1)
    epoch = {}

    def pattern(rid, nb):
        blk_ix = torch.arange(nb, device="cuda", dtype=torch.int64).view(1, -1, 1)
        return ((rid + 1000 * epoch[rid]) << 40) ^ (plane_ix << 32) ^ (blk_ix << 12) ^ word_ix

    def fill(rid, blocks, n):
        epoch[rid] = epoch.get(rid, 0) + 1          # a recomputed request gets new content
        if len(blocks):
            view[:, torch.from_numpy(blocks.astype(np.int64)).cuda()] = pattern(rid, len(blocks))
            torch.cuda.synchronize()                # the library's streams do not wait for torch's

    checked = [0]

    def verify(rid):
        assert g.wait(rid) == kvr.OK, kvr.last_error()
        d = g.info(rid)[1]
        n, blocks = d["n_tokens"], d["blocks"]
        if len(blocks) == 0:
            return
        got = view[:, torch.from_numpy(blocks.astype(np.int64)).cuda()]
        want = pattern(rid, len(blocks))
        full = n // BS                              # whole blocks: every word; last partial block: valid rows only
        assert torch.equal(got[:, :full], want[:, :full]), "request %d came back changed" % rid
        if full < len(blocks):
            valid_words = (n - full * BS) * H * D * e // 8
            assert torch.equal(got[:, full, :valid_words], want[:, full, :valid_words])
        checked[0] += 1

    steps = [0]

    def after(name, args):
        steps[0] += 1
        if steps[0] % 16 == 0:                      # bookkeeping is compared on every call; the O(N) sweeps every 16th
            check_invariants(g, range(w.n_requests))
            assert o.free_queue().tolist() == g.free_queue().tolist()
    counts = TraceRunner([o, g], lengths, fill=fill, verify=verify, after_call=after).run(events)
    assert g.wait() == kvr.OK, kvr.last_error()
    check_invariants(g, range(w.n_requests))
    so, sg = o.stats(), g.stats()
    for k in so:
        assert so[k] == sg[k], k
    assert counts["arrived"] == w.n_requests and counts.get("resumed_from_host", 0) > 50 and checked[0] > 100
    assert sg["bytes_suspended"] - sg["bytes_resumed"] - sg["bytes_expired_from_host"] == 0 and sg["host_used"] == 0
    print("config 4 trace:", counts, "GB suspended %.1f resumed %.1f" % (sg["bytes_suspended"] / 1e9, sg["bytes_resumed"] / 1e9))
    g.close()
    o.close()


def test_live_controller_with_data():
    """The clock-driven controller (grace period in HBM, offload, one-shot timers, eviction of the longest
    suspended copy) on the GPU pool, next to the oracle's controller on the CPU pool: same decisions, same cost,
    and the same bytes in every surviving host image and in the pool at the end."""
    from kvr_synth import paper_wait_family, poisson_arrivals
    from oracle.controller import LIVE, TTL, OrcController
    from test_controller_cpu import PRICES, run_trace
    geom = (2, 2, 16, 2, 4)                        # 256 bytes per token
    n, NB, host_cap = 200, 700, 40 * 4096
    rng = np.random.default_rng(33)
    lengths = rng.integers(1, 120, size=n)
    mean_img = float(np.mean(lengths)) * 256
    w_ref = 1800.0
    lam = 2.5 * (host_cap / mean_img) / w_ref
    arrive, wait = poisson_arrivals(n, lam, 33), paper_wait_family("mixture", n, 33)
    t = Twin(geom, NB, host_cap, seed=33, chunk_bytes=8192, staging_slots=2)
    L, H, D, e, BS = geom
    o_view = t.o.data.reshape(2 * L, NB, BS * H * D * e)
    d_view = t.dev.view(2 * L, NB, BS * H * D * e)
    fills = {}

    def on_admit(i, blocks):                       # the same fresh bytes on both sides (seeded per admission)
        k = fills.get(i, 0)
        fills[i] = k + 1
        fresh = np.random.default_rng([33, i, k]).integers(0, 256, size=(2 * L, len(blocks), BS * H * D * e), dtype=np.uint8)
        if pool_is_gpu[0]:
            d_view[:, torch.from_numpy(blocks.astype(np.int64)).cuda()] = torch.from_numpy(fresh).cuda()
            torch.cuda.synchronize()
        else:
            o_view[:, blocks] = fresh
    pool_is_gpu = [False]
    co = OrcController(t.o, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=20.0, branch=TTL, admission=LIVE)
    lo = run_trace(co, t.o, arrive, wait, lengths, on_admit=on_admit)
    pool_is_gpu[0] = True
    fills.clear()
    cg = kvr.Controller(t.g, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=20.0, branch=TTL, admission=kvr.ADMIT_LIVE)
    lg = run_trace(cg, t.g, arrive, wait, lengths, on_admit=on_admit)      # release() waits for a resume in flight
    assert lo == lg
    so, sg = co.stats(), cg.stats()
    for k in so:
        assert sg[k] == pytest.approx(so[k], rel=1e-12), k
    assert so["resumed_host"] > 20 and so["evicted_lru"] > 0 and so["ttl_expired"] > 0 and so["resumed_hbm"] > 0
    t.assert_same_pool()
    cg.close()
    t.close()


class _SharingPool:
    """A pool whose plain admissions share the first `ns` blocks of a long-lived donor request: the paper's workload
    shape (one system prefix, private suffixes) driven through code that only knows `admit`."""

    def __init__(self, pool, donor, ns, bs):
        self._pool, self._donor, self._ns, self._bs = pool, donor, ns, bs

    def admit(self, rid, n_private):
        return self._pool.admit_sharing(rid, self._ns * self._bs + n_private, self._donor, self._ns)

    def __getattr__(self, name):
        return getattr(self._pool, name)


def test_live_controller_over_a_shared_prefix_with_data():
    """The live controller when every context shares one system prefix: only private suffixes travel, the prefix
    stays resident as long as any context (active, pinned or on the host) refers to it, and decisions, costs, images
    and final pool bytes equal the oracle's."""
    from kvr_synth import paper_wait_family, poisson_arrivals
    from oracle.controller import LIVE, TTL, OrcController
    from test_controller_cpu import PRICES, run_trace
    geom = (2, 2, 16, 2, 4)                        # 256 bytes per token
    L, H, D, e, BS = geom
    n, NB, host_cap, ns = 160, 700, 32 * 4096, 9   # a 36-token prefix
    rng = np.random.default_rng(41)
    lengths = rng.integers(1, 100, size=n)         # private suffix lengths
    mean_img = float(np.mean(lengths)) * 256
    w_ref = 1800.0
    lam = 2.5 * (host_cap / mean_img) / w_ref
    arrive, wait = poisson_arrivals(n, lam, 41), paper_wait_family("mixture", n, 41)
    t = Twin(geom, NB, host_cap, seed=41, chunk_bytes=8192, staging_slots=3)
    o_view = t.o.data.reshape(2 * L, NB, BS * H * D * e)
    d_view = t.dev.view(2 * L, NB, BS * H * D * e)
    PREFIX = 10_000
    a, b = t.both("admit", PREFIX, ns * BS)
    assert a[0] == b[0] == orc.OK and a[1].tolist() == b[1].tolist()
    prefix_blocks = a[1]
    fills = {}
    pool_is_gpu = [False]

    def on_admit(i, blocks):                       # fresh bytes for the private blocks only, the same on both sides
        assert blocks[:ns].tolist() == prefix_blocks.tolist()
        mine = blocks[ns:]
        k = fills.get(i, 0)
        fills[i] = k + 1
        fresh = np.random.default_rng([41, i, k]).integers(0, 256, size=(2 * L, len(mine), BS * H * D * e), dtype=np.uint8)
        if pool_is_gpu[0]:
            d_view[:, torch.from_numpy(mine.astype(np.int64)).cuda()] = torch.from_numpy(fresh).cuda()
            torch.cuda.synchronize()
        else:
            o_view[:, mine] = fresh
    so_pool, sg_pool = _SharingPool(t.o, PREFIX, ns, BS), _SharingPool(t.g, PREFIX, ns, BS)
    co = OrcController(t.o, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=20.0, branch=TTL, admission=LIVE)
    lo = run_trace(co, so_pool, arrive, wait, lengths, on_admit=on_admit)
    pool_is_gpu[0] = True
    fills.clear()
    cg = kvr.Controller(t.g, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=20.0, branch=TTL, admission=kvr.ADMIT_LIVE)
    lg = run_trace(cg, sg_pool, arrive, wait, lengths, on_admit=on_admit)
    assert lo == lg
    so, sg = co.stats(), cg.stats()
    for k in so:
        assert sg[k] == pytest.approx(so[k], rel=1e-12), k
    assert so["resumed_host"] > 15 and so["ttl_expired"] + so["evicted_lru"] > 0
    ps, pg = t.o.stats(), t.g.stats()
    assert ps["bytes_suspended"] == pg["bytes_suspended"] == pg["gather_bytes"] > 0      # suffix bytes only
    assert t.g.refcount(int(prefix_blocks[0])) == t.o.refcount(int(prefix_blocks[0])) == 1     # only the owner is left
    t.assert_same_pool()
    check_invariants(t.g, list(range(n)) + [PREFIX])
    cg.close()
    t.close()
