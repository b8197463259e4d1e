"""The benchmark configurations at full size on the GPU, in the launch configuration bench.py times
(staged route, default mover and chunk sizes).

A host mirror of a 64-128 GiB pool does not exist, so parity is shown four ways:
  * bookkeeping (statuses, block tables, arena offsets, free queue) against a data-less oracle pool, call by call;
  * EVERY image byte: the image, by definition, is image[plane][t] = pool[plane][table[t / BS]][t % BS]; that
    expression is evaluated on the device with torch indexing (pinned once against the oracle's gather on a small
    pool, below) and compared with the whole image the library wrote, request by request, after the suspend under
    the old tables and after the resume under the new ones; and every pool row outside the resumed requests' valid
    slots is shown unchanged through per-row checksums taken before and after;
  * sampled token rows: the oracle names, one by one, the pool byte offset and the image byte offset of a sampled
    (request, layer, plane, token); the bytes found there on the device / in the pinned arena must be equal;
  * one whole request: its blocks are read back into a small relabelled host pool, the oracle gathers that pool
    element by element, and the result must equal the image the GPU wrote, byte for byte.
"""
import gc

import numpy as np
import pytest
import torch

import oracle as orc
from common import check_invariants
from kvr_synth import CONFIGS, context_lengths, event_trace, free_order, occupancy_fillers
from paper_2608_30830_b200 import kvr

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

SEED = 20260830


def host_avail():
    return int(open("/proc/meminfo").read().split("MemAvailable:")[1].split()[0]) * 1024


def cleanup():
    gc.collect()
    torch.cuda.empty_cache()


class Rig:
    """A full-size library pool over torch device memory filled with bf16 N(0,1), next to a data-less oracle."""

    def __init__(self, geom, NB, host_cap, seed, **kw):
        self.geom, self.NB = geom, NB
        L, H, D, e, BS = geom
        self.row = H * D * e
        self.bpt = kvr.bytes_per_token(L, H, D, e)
        self.dev = torch.empty(NB * BS * self.bpt, dtype=torch.uint8, device="cuda")
        gen = torch.Generator(device="cuda").manual_seed(seed)
        v = self.dev.view(torch.bfloat16)
        for i in range(0, v.numel(), 1 << 28):
            v[i:i + (1 << 28)].normal_(generator=gen)
        torch.cuda.synchronize()
        order = free_order(seed, NB)
        self.o = orc.OrcPool(*geom, NB, host_cap, initial_free_order=order, with_data=False)
        self.g = kvr.Pool(*geom, NB, host_cap, initial_free_order=order, device_pool=self.dev.data_ptr(), **kw)
        self.rows = self.dev.view(-1, self.row)            # the pool as rows of one token of one plane
        self.rng = np.random.default_rng(seed)

    def both(self, name, *args):
        a = getattr(self.o, name)(*args)
        b = getattr(self.g, name)(*args)
        if name == "admit":
            assert a[0] == b[0] and (a[1] is None or a[1].tolist() == b[1].tolist()), (name, args)
        else:
            assert a == b, (name, args, a, b)
        return b

    def sample(self, ids, k):
        """k sampled (request, layer, plane, token) with the oracle's pool and image offsets of their rows."""
        L, H, D, e, BS = self.geom
        out = []
        live = [r for r in ids if self.o.info(r)[1]["n_tokens"] > 0]
        for _ in range(k):
            rid = int(self.rng.choice(live))
            d = self.o.info(rid)[1]
            n = d["n_tokens"]
            l, kv = int(self.rng.integers(L)), int(self.rng.integers(2))
            # bias towards block edges and the ragged tail
            t = int(self.rng.choice([0, n - 1, max(0, n - 1 - (n - 1) % BS), int(self.rng.integers(n)), int(self.rng.integers(n))]))
            blk = int(d["blocks"][t // BS])
            po = orc.pool_offset(L, H, D, e, BS, self.NB, l, kv, blk, t % BS)
            io = orc.image_offset(L, H, D, e, n, l, kv, t)
            assert po % self.row == 0 and io % self.row == 0
            out.append((rid, l, kv, t, po, io))
        return out

    def read_pool_rows(self, samples):
        idx = torch.tensor([s[4] // self.row for s in samples], device="cuda")
        return self.rows.index_select(0, idx).cpu().numpy()

    def read_image_rows(self, samples):
        out = np.empty((len(samples), self.row), dtype=np.uint8)
        for i, (rid, _, _, _, _, io) in enumerate(samples):
            out[i] = self.g.host_image(rid)[io:io + self.row]
        return out

    def resample_pool_offsets(self, samples):
        """Same logical rows after a resume: offsets under the request's new table."""
        L, H, D, e, BS = self.geom
        out = []
        for rid, l, kv, t, _, io in samples:
            blk = int(self.o.info(rid)[1]["blocks"][t // BS])
            out.append((rid, l, kv, t, orc.pool_offset(L, H, D, e, BS, self.NB, l, kv, blk, t % BS), io))
        return out

    def whole_request_image(self, rid):
        """Oracle image of one request, computed from its blocks read back into a relabelled mini pool."""
        L, H, D, e, BS = self.geom
        d = self.o.info(rid)[1]
        blocks = torch.tensor(d["blocks"].astype(np.int64), device="cuda")
        tile = BS * self.row
        mini = self.dev.view(2 * L, self.NB, tile).index_select(1, blocks).cpu().numpy().reshape(-1)
        return orc.gather(mini, L, H, D, e, BS, d["nb"], np.arange(d["nb"]), d["n_tokens"])

    def row_sums(self):
        """One wrapping int64 sum per pool row (one token slot of one plane of one block): shape (2L, NB, BS)."""
        L, H, D, e, BS = self.geom
        return self.dev.view(torch.int64).view(2 * L * self.NB * BS, self.row // 8).sum(dim=1).view(2 * L, self.NB, BS)

    def image_by_definition(self, table, n, p0, p1):
        """Planes [p0, p1) of the image of a request with this table and n tokens, from the pool as it is now."""
        return image_by_definition(self.dev, self.geom, self.NB, table, n, p0, p1)

    def assert_whole_images(self, ids, tables, images, slab_bytes=1 << 30, tokens=None):
        """Every byte of every image (numpy views of the pinned arena) against the definition under `tables`
        (`tokens`: how many tokens each table covers, when that is not the whole request)."""
        L, H, D, e, BS = self.geom
        for rid in ids:
            n = int(tokens[rid]) if tokens is not None else int(self.o.info(rid)[1]["n_tokens"])
            if n == 0:
                continue
            img = torch.from_numpy(images[rid]).view(2 * L, n, self.row)
            step = max(1, slab_bytes // (n * self.row))
            for p0 in range(0, 2 * L, step):
                p1 = min(2 * L, p0 + step)
                want = self.image_by_definition(tables[rid], n, p0, p1)
                got = img[p0:p1].cuda()
                assert torch.equal(got, want), "image of request %d differs in planes %d..%d" % (rid, p0, p1)
                del want, got

    def close(self):
        self.g.close()
        self.o.close()
        del self.rows, self.dev
        cleanup()


def image_by_definition(dev_pool, geom, NB, table, n, p0=0, p1=None):
    """image[plane][t][:] = pool[plane][table[t // BS]][t % BS][:] for planes [p0, p1), as a (planes, n, row) uint8
    tensor on the device: the definition of the host image, written with torch indexing (layer-major pool)."""
    L, H, D, e, BS = geom
    row = H * D * e
    p1 = 2 * L if p1 is None else p1
    blocks = torch.as_tensor(np.asarray(table, dtype=np.int64), device=dev_pool.device)
    tiles = dev_pool.view(2 * L, NB, BS * row)[p0:p1].index_select(1, blocks)          # (planes, nb, tile)
    return tiles.reshape(p1 - p0, len(table) * BS, row)[:, :n]


def untouched_rows(rig, ids, others, k=256):
    """Oracle-addressed rows a resume of `ids` must leave alone (same tuple shape as Rig.sample: offset at [4])."""
    L, H, D, e, BS = rig.geom
    out = []
    for rid in ids:                                   # tail slots of a partial last block
        d = rig.o.info(rid)[1]
        n = d["n_tokens"]
        if n % BS:
            l, kv = int(rig.rng.integers(L)), int(rig.rng.integers(2))
            for slot in {n % BS, BS - 1}:
                out.append((rid, l, kv, -1, orc.pool_offset(L, H, D, e, BS, rig.NB, l, kv, int(d["blocks"][-1]), slot), 0))
    pool_blocks = list(rig.o.free_queue()[:64])       # blocks still free after the resume
    for rid in others[:8]:                            # blocks of other live requests
        pool_blocks += list(rig.o.info(rid)[1]["blocks"][:8])
    for _ in range(k):
        if not pool_blocks:
            break
        blk = int(rig.rng.choice(pool_blocks))
        l, kv, slot = int(rig.rng.integers(L)), int(rig.rng.integers(2)), int(rig.rng.integers(BS))
        out.append((-1, l, kv, -1, orc.pool_offset(L, H, D, e, BS, rig.NB, l, kv, blk, slot), 0))
    return out


def touched_mask(rig, ids):
    """(NB, BS) bool: the token slots a resume of `ids` writes (valid slots of their current blocks)."""
    BS = rig.geom[4]
    mask = torch.zeros(rig.NB, BS, dtype=torch.bool)
    for rid in ids:
        d = rig.o.info(rid)[1]
        n, blocks = int(d["n_tokens"]), d["blocks"].astype(np.int64)
        if n == 0:
            continue
        mask[torch.from_numpy(blocks[:n // BS])] = True
        if n % BS:
            mask[int(blocks[-1]), :n % BS] = True
    return mask.cuda()


def suspend_resume_checked(rig, ids, whole=None, k=1536, others=()):
    samples = rig.sample(ids, k)
    before = rig.read_pool_rows(samples)
    want_whole = rig.whole_request_image(whole) if whole is not None else None
    sums0 = rig.row_sums()
    old_tables = {rid: rig.o.info(rid)[1]["blocks"].copy() for rid in ids}
    st, per = rig.both("suspend_to_host", ids)
    assert st == kvr.OK
    assert rig.g.wait() == kvr.OK, kvr.last_error()
    assert np.array_equal(rig.read_image_rows(samples), before)           # image rows = the oracle-addressed pool rows
    assert np.array_equal(rig.read_pool_rows(samples), before)            # the suspend left the pool alone
    assert torch.equal(rig.row_sums(), sums0)                             # ... every row of it
    images = {rid: rig.g.host_image(rid) for rid in ids}                  # views of the arena; they outlive the resume
    rig.assert_whole_images(ids, old_tables, images)                      # every image byte, by definition
    if whole is not None:
        assert np.array_equal(rig.g.host_image(whole), want_whole)
    for rid in ids:
        assert rig.o.info(rid)[1]["arena_offset"] == rig.g.info(rid)[1]["arena_offset"]
    # the oracle resumes first: its new tables name the rows that must NOT change -- the slots behind the last valid
    # token of a partial last block, and rows of blocks that stay free or belong to other requests
    ro = rig.o.resume_from_host(ids)
    untouched = untouched_rows(rig, ids, others)
    keep = rig.read_pool_rows(untouched) if untouched else None
    rg = rig.g.resume_from_host(ids)
    assert ro == rg and rg[0] == kvr.OK
    assert rig.g.wait() == kvr.OK, kvr.last_error()
    if untouched:
        assert np.array_equal(rig.read_pool_rows(untouched), keep)
    for rid in ids:
        assert rig.o.info(rid)[1]["blocks"].tolist() == rig.g.info(rid)[1]["blocks"].tolist()
    after = rig.resample_pool_offsets(samples)
    assert np.array_equal(rig.read_pool_rows(after), before)              # same logical rows under the new tables
    new_tables = {rid: rig.o.info(rid)[1]["blocks"].copy() for rid in ids}
    rig.assert_whole_images(ids, new_tables, images)                      # every byte landed where the new tables say
    same = rig.row_sums() == sums0                                        # and nothing else in the pool changed
    assert bool((same | touched_mask(rig, ids).unsqueeze(0)).all()), "a row outside the resumed requests changed"
    del same, sums0
    if whole is not None:
        assert np.array_equal(rig.whole_request_image(whole), want_whole)
    assert rig.o.free_queue().tolist() == rig.g.free_queue().tolist()


def test_definition_on_the_device_equals_the_oracle_gather():
    """Pins image_by_definition (the torch expression the full-size checks rely on) to the oracle, element by
    element, on a pool small enough to mirror on the host: ragged length, shuffled table, several planes."""
    geom = (3, 2, 64, 2, 4)
    L, H, D, e, BS = geom
    NB = 96
    rng = np.random.default_rng(5)
    host_pool = rng.integers(0, 256, size=NB * BS * 2 * L * H * D * e, dtype=np.uint8)
    dev_pool = torch.from_numpy(host_pool).cuda()
    for n in (1, 4, 37, 40, 163):
        nb = -(-n // BS)
        table = rng.permutation(NB)[:nb].astype(np.int32)
        want = orc.gather(host_pool, L, H, D, e, BS, NB, table, n)
        got = image_by_definition(dev_pool, geom, NB, table, n).cpu().numpy().reshape(-1)
        assert np.array_equal(got, want), n
        part = image_by_definition(dev_pool, geom, NB, table, n, 2, 5).cpu().numpy().reshape(-1)
        assert np.array_equal(part, want.reshape(2 * L, -1)[2:5].reshape(-1))


def test_config2_llama3_8b_shaped_full_size():
    w = CONFIGS["llama3_8b"]
    seed = SEED + 1
    lens = context_lengths(w.length_rule, w.n_requests, seed)
    used = int(sum(-(-int(n) // w.block_size) for n in lens))
    fillers = occupancy_fillers(w.num_blocks, w.block_size, used, w.occupancy, seed)
    bpt = kvr.bytes_per_token(*w.geom[:4])
    host_cap = int(lens.sum()) * bpt + (64 << 20)
    if host_avail() < host_cap + (16 << 30):
        pytest.skip("host memory too small for the 37 GB arena")
    rig = Rig(w.geom, w.num_blocks, host_cap, seed, flags=kvr.PROFILE)
    ids = list(range(len(lens)))
    order = [(i, int(n)) for i, n in zip(ids, lens)] + [(1000 + i, int(n)) for i, n in enumerate(fillers)]
    np.random.default_rng(seed).shuffle(order)
    for rid, n in order:
        assert rig.both("admit", rid, n)[0] == kvr.OK
    assert abs(1 - rig.g.stats()["blocks_free"] / w.num_blocks - 0.70) < 0.001
    suspend_resume_checked(rig, ids, whole=int(np.argmin(lens)), others=[1000 + i for i in range(len(fillers))])
    s = rig.g.stats()
    assert s["bytes_suspended"] == s["bytes_resumed"] == s["gather_bytes"] == s["scatter_bytes"] == int(lens.sum()) * bpt
    check_invariants(rig.g, ids + [1000 + i for i in range(len(fillers))])
    rig.close()


def test_config3_gqa64_resume_burst():
    w = CONFIGS["gqa64"]
    seed = SEED + 2
    bpt = kvr.bytes_per_token(*w.geom[:4])
    n_req = w.n_requests
    free_dev, _ = torch.cuda.mem_get_info()
    NB = w.num_blocks
    while NB * w.block_size * bpt + (8 << 30) > free_dev:                   # scale rule: smaller pool, same geometry
        NB -= 4096
    while n_req > 1 and (n_req * 16384 * bpt + (32 << 30) > host_avail() or n_req * 1024 * 2 > NB):
        n_req -= 1
    print("gqa64: requests_requested=%d requests_run=%d num_blocks=%d" % (w.n_requests, n_req, NB))
    host_cap = n_req * 16384 * bpt + (64 << 20)
    rig = Rig(w.geom, NB, host_cap, seed)
    ids = list(range(n_req))
    # live filler requests between the batch's admissions, so the free list is interleaved with live blocks
    fid = 1000
    for rid in ids:
        assert rig.both("admit", rid, 16384)[0] == kvr.OK
        if rig.o.stats()["blocks_free"] > (n_req - rid) * 1024 + 600:
            assert rig.both("admit", fid, 4096)[0] == kvr.OK
            fid += 1
    suspend_resume_checked(rig, ids, whole=None, k=1024, others=list(range(1000, fid)))
    rig.close()


def test_config5_long_context_overlapped_suspend_and_resume():
    """block_size 8, 128k-token requests with fully shuffled ids; a suspend of one half runs while the other half
    resumes, on the library's separate stream pairs, with no wait between the two calls."""
    w = CONFIGS["longctx"]
    seed = SEED + 4
    bpt = kvr.bytes_per_token(*w.geom[:4])
    n_tok = 131072
    n_req = w.n_requests
    free_dev, _ = torch.cuda.mem_get_info()
    while n_req > 2 and (n_req * n_tok * bpt + (24 << 30) > free_dev or n_req * n_tok * bpt + (40 << 30) > host_avail()):
        n_req -= 2
    print("longctx: requests_requested=%d requests_run=%d" % (w.n_requests, n_req))
    NB = n_req * (n_tok // w.block_size)
    host_cap = n_req * n_tok * bpt + (64 << 20)
    rig = Rig(w.geom, NB, host_cap, seed)
    ids = list(range(n_req))
    for rid in ids:
        assert rig.both("admit", rid, n_tok)[0] == kvr.OK
    half = n_req // 2
    out_first, stay = ids[:half], ids[half:]
    s_out = rig.sample(out_first, 512)
    rows_out = rig.read_pool_rows(s_out)
    sums0 = rig.row_sums()
    tables = {rid: rig.o.info(rid)[1]["blocks"].copy() for rid in ids}
    assert rig.both("suspend_to_host", out_first)[0] == kvr.OK             # phase A (untimed): one half on the host
    assert rig.g.wait() == kvr.OK
    assert np.array_equal(rig.read_image_rows(s_out), rows_out)
    assert torch.equal(rig.row_sums(), sums0)
    images = {rid: rig.g.host_image(rid) for rid in out_first}
    rig.assert_whole_images(out_first, tables, images)                     # every byte of the first half's images
    s_stay = rig.sample(stay, 512)
    rows_stay = rig.read_pool_rows(s_stay)
    # phase B: both directions at once
    assert rig.both("suspend_to_host", stay)[0] == kvr.OK
    assert rig.both("resume_from_host", out_first)[0] == kvr.OK
    assert rig.g.wait() == kvr.OK, kvr.last_error()
    assert np.array_equal(rig.read_image_rows(s_stay), rows_stay)
    assert np.array_equal(rig.read_pool_rows(rig.resample_pool_offsets(s_out)), rows_out)
    for rid in out_first:
        assert rig.o.info(rid)[1]["blocks"].tolist() == rig.g.info(rid)[1]["blocks"].tolist()
    # the overlapped pair, completely: the second half's images under the tables they had (their blocks were freed,
    # and the overlapped resume took blocks from the head of the queue, i.e. other ones: see the assert), and the
    # first half under its new tables; every other row unchanged
    new_out = {rid: rig.o.info(rid)[1]["blocks"].copy() for rid in out_first}
    taken = set(int(b) for rid in out_first for b in new_out[rid])
    images.update({rid: rig.g.host_image(rid) for rid in stay})
    if not taken & set(int(b) for rid in stay for b in tables[rid]):
        rig.assert_whole_images(stay, tables, images)
    rig.assert_whole_images(out_first, new_out, images)
    same = rig.row_sums() == sums0
    assert bool((same | touched_mask(rig, out_first).unsqueeze(0)).all())
    del same
    assert rig.both("resume_from_host", stay)[0] == kvr.OK
    assert rig.g.wait() == kvr.OK
    assert np.array_equal(rig.read_pool_rows(rig.resample_pool_offsets(s_stay)), rows_stay)
    new_stay = {rid: rig.o.info(rid)[1]["blocks"].copy() for rid in stay}
    rig.assert_whole_images(stay, new_stay, images)
    same = rig.row_sums() == sums0
    assert bool((same | touched_mask(rig, ids).unsqueeze(0)).all())
    del same, sums0
    check_invariants(rig.g, ids)
    rig.close()


def test_paper_shaped_contexts_sharing_one_prefix_full_size():
    """One TP4 rank of the paper's model (80 layers, 2 KV heads: 8 KiB tiles), 32 gate contexts of 8,400 tokens over
    one shared 5,392-token prefix (337 whole blocks), pool at 50 % occupancy.  Only the 3,008-token suffixes move:
    every image byte against the definition over the private part of the table, the prefix blocks untouched and
    still referenced while the requests are on the host, every other pool row unchanged by the round trip."""
    w = CONFIGS["paper_shape"]
    seed = SEED + 6
    L, H, D, e, BS = w.geom
    bpt = kvr.bytes_per_token(*w.geom[:4])
    n_ctx, shared_blocks = 8400, w.extra["shared_tokens"] // BS
    n_priv = n_ctx - shared_blocks * BS
    ids = list(range(w.n_requests))
    host_cap = len(ids) * (n_priv * bpt + 4096) + (64 << 20)
    rig = Rig(w.geom, w.num_blocks, host_cap, seed)
    PREFIX = 900
    assert rig.both("admit", PREFIX, shared_blocks * BS)[0] == kvr.OK
    used = shared_blocks + len(ids) * (-(-n_ctx // BS) - shared_blocks)
    fillers = occupancy_fillers(w.num_blocks, BS, used, w.occupancy, seed)
    order = [(i, n_ctx) for i in ids] + [(1000 + i, int(n)) for i, n in enumerate(fillers)]
    np.random.default_rng(seed).shuffle(order)
    for rid, n in order:
        if rid < 900:
            a = rig.o.admit_sharing(rid, n, PREFIX, shared_blocks)
            b = rig.g.admit_sharing(rid, n, PREFIX, shared_blocks)
            assert a[0] == b[0] == kvr.OK and a[1].tolist() == b[1].tolist()
        else:
            assert rig.both("admit", rid, n)[0] == kvr.OK
    assert rig.both("release", PREFIX) == kvr.OK
    prefix = rig.g.sharing(0)[1]
    assert len(prefix) == shared_blocks and rig.g.refcount(int(prefix[0])) == len(ids)
    sums0 = rig.row_sums()
    private = {rid: rig.o.info(rid)[1]["blocks"][shared_blocks:].copy() for rid in ids}
    st, per = rig.both("suspend_to_host", ids)
    assert st == kvr.OK
    assert rig.g.wait() == kvr.OK, kvr.last_error()
    s = rig.g.stats()
    assert s["bytes_suspended"] == s["gather_bytes"] == len(ids) * n_priv * bpt          # 246 MB per context, not 688 MB
    assert s["blocks_pinned"] == shared_blocks and rig.g.refcount(int(prefix[0])) == len(ids)
    assert torch.equal(rig.row_sums(), sums0)
    images = {rid: rig.g.host_image(rid) for rid in ids}
    tokens = {rid: n_priv for rid in ids}
    rig.assert_whole_images(ids, private, images, tokens=tokens)
    ro = rig.o.resume_from_host(ids[::-1])
    rg = rig.g.resume_from_host(ids[::-1])
    assert ro == rg and rg[0] == kvr.OK
    assert rig.g.wait() == kvr.OK, kvr.last_error()
    new_private = {}
    for rid in ids:
        t = rig.o.info(rid)[1]["blocks"]
        assert t.tolist() == rig.g.info(rid)[1]["blocks"].tolist() and t[:shared_blocks].tolist() == prefix.tolist()
        new_private[rid] = t[shared_blocks:].copy()
    rig.assert_whole_images(ids, new_private, images, tokens=tokens)
    # nothing but the valid slots of the new private blocks changed: the shared prefix in particular did not
    mask = torch.zeros(rig.NB, BS, dtype=torch.bool)
    for rid in ids:
        mask[torch.from_numpy(new_private[rid][:n_priv // BS].astype(np.int64))] = True
        if n_priv % BS:
            mask[int(new_private[rid][-1]), :n_priv % BS] = True
    same = rig.row_sums() == sums0
    assert bool((same | mask.cuda().unsqueeze(0)).all())
    assert rig.o.free_queue().tolist() == rig.g.free_queue().tolist()
    check_invariants(rig.g, ids + [1000 + i for i in range(len(fillers))])
    rig.close()
