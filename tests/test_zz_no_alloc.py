"""kvr_gather_noalloc, the entry point for callers that cannot allocate device memory (an engine that has
given all of HBM to its own block allocator, or a path that must not take the device-wide synchronisation
an allocation implies).  It must write exactly what kvr_export_to_device writes for the same request, and both
must equal the image the CPU oracle gathers, element by element, from a host copy of the same pool bytes.

Two calls in a row share the library's fixed scratch array, so the second call (a shorter request with a
different table) also proves that nothing left over from the first one is read.  This file is named to be
collected last; it passes alone in a fresh process and after the rest of the suite."""
import numpy as np
import pytest
import torch

import oracle as orc
from paper_2608_30830_b200 import kvr

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]

GEOM = (4, 8, 128, 2, 16)        # 2 KiB rows, 32 KiB tiles, 16 KiB per token
NB = 512


def test_matches_export_to_device_on_two_calls_in_a_row():
    bpt = kvr.bytes_per_token(*GEOM[:4])
    dev_pool = torch.empty(NB * GEOM[4] * bpt, dtype=torch.uint8, device="cuda")
    dev_pool.view(torch.bfloat16).normal_(generator=torch.Generator(device="cuda").manual_seed(7))
    torch.cuda.synchronize()
    order = np.random.default_rng(7).permutation(NB).astype(np.int32)
    with kvr.Pool(*GEOM, NB, 0, initial_free_order=order, device_pool=dev_pool.data_ptr()) as pool:
        lens = {1: 3001, 2: 517}                  # ragged tails; the second request is shorter
        tables = {rid: pool.admit(rid, n)[1] for rid, n in lens.items()}
        stream = torch.cuda.Stream()
        for rid in (1, 2):                        # two calls in a row on one stream, no wait in between
            n = lens[rid]
            want = torch.zeros(n * bpt, dtype=torch.uint8, device="cuda")
            st, offs = pool.export_to_device([rid], want.data_ptr(), want.numel(), kvr.SYNC)
            assert st == kvr.OK and offs.tolist() == [0], kvr.last_error()
            lens[rid] = (n, want)
        got = {rid: torch.full((lens[rid][0] * bpt,), 0xA5, dtype=torch.uint8, device="cuda") for rid in (1, 2)}
        torch.cuda.synchronize()
        for rid in (1, 2):
            st = kvr.gather_noalloc(dev_pool.data_ptr(), GEOM, NB, tables[rid], lens[rid][0], got[rid].data_ptr(),
                                    stream.cuda_stream)
            assert st == kvr.OK, kvr.last_error()
        stream.synchronize()
        host_pool = dev_pool.cpu().numpy()
        for rid in (1, 2):
            assert torch.equal(got[rid], lens[rid][1]), "request %d differs from kvr_export_to_device" % rid
            want = orc.gather(host_pool, *GEOM, NB, tables[rid], lens[rid][0])
            assert np.array_equal(got[rid].cpu().numpy(), want), "request %d differs from the oracle's image" % rid
        assert got[1].any() and got[2].any()


def test_largest_table_the_scratch_holds_and_a_page_locked_table():
    """nb == KVR_NOALLOC_MAX_BLOCKS: the table fills the fixed array to its last entry.  The table is handed over
    in page-locked memory and overwritten right after the call returns: the call must have taken its own copy."""
    geom = (1, 1, 16, 1, 1)                       # one token per block, 16-byte rows, 32 bytes per token
    nb = kvr.NOALLOC_MAX_BLOCKS
    NBp = nb + 7
    rng = np.random.default_rng(11)
    host_pool = rng.integers(0, 256, size=NBp * 32, dtype=np.uint8)
    dev_pool = torch.from_numpy(host_pool).cuda()
    table = rng.permutation(NBp)[:nb].astype(np.int32)
    pinned = torch.from_numpy(table.copy()).pin_memory()
    got = torch.full((nb * 32,), 0xA5, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    st = kvr.gather_noalloc(dev_pool.data_ptr(), geom, NBp, pinned.numpy(), nb, got.data_ptr(), stream.cuda_stream)
    pinned.fill_(0)                               # the caller reuses its table at once
    assert st == kvr.OK, kvr.last_error()
    stream.synchronize()
    want = orc.gather(host_pool, *geom, NBp, table, nb)
    out = got.cpu().numpy()
    assert np.array_equal(out, want)
    # the last table entry is honoured: token nb-1 of the K plane and of the V plane
    last = int(table[-1])
    assert np.array_equal(out[(nb - 1) * 16:nb * 16], host_pool[last * 16:(last + 1) * 16])
    assert np.array_equal(out[(2 * nb - 1) * 16:], host_pool[(NBp + last) * 16:(NBp + last + 1) * 16])


def test_rejects_what_does_not_fit_or_is_malformed():
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    geom = (1, 1, 16, 1, 1)                       # one token per block, 32 bytes per token
    too_many = kvr.NOALLOC_MAX_BLOCKS + 1
    table = np.zeros(too_many, dtype=np.int32)
    st = kvr.gather_noalloc(buf.data_ptr(), geom, 4, table, too_many, buf.data_ptr())
    assert st == kvr.ERR_INVALID_ARG and "KVR_NOALLOC_MAX_BLOCKS" in kvr.last_error()
    assert kvr.gather_noalloc(buf.data_ptr(), geom, 4, [0, 4], 2, buf.data_ptr()) == kvr.ERR_INVALID_ARG   # id out of range
    assert kvr.gather_noalloc(buf.data_ptr(), geom, 4, [0, 1], 3, buf.data_ptr()) == kvr.ERR_INVALID_ARG   # nb != ceil(n/BS)
    assert kvr.gather_noalloc(buf.data_ptr(), (1, 1, 3, 1, 1), 4, [0], 1, buf.data_ptr()) == kvr.ERR_GEOMETRY
    # a tile beyond 1 GiB (block_size x row bytes) is refused before any size is narrowed to int
    assert kvr.gather_noalloc(buf.data_ptr(), (1, 64, 16384, 4, 1024), 4, [0], 1, buf.data_ptr()) == kvr.ERR_GEOMETRY
    assert "1 GiB" in kvr.last_error()
    assert kvr.gather_noalloc(buf.data_ptr(), geom, 4, [], 0, buf.data_ptr()) == kvr.OK                    # empty request
