"""Pins for the CPU oracle: values the paper prints, closed forms, numpy
restatements of special cases, and brute force on tiny pools.  CPU only."""
import itertools

import numpy as np
import pytest

import oracle as orc
from kvr_synth import fill_bytes


# ---- bytes per token and the paper's worked sizes (Appendix B) ---------------

def test_bytes_per_token_paper_example(golden):
    L, H, D, e = (int(x) for x in golden["bpt_factors"])
    assert orc.bytes_per_token(L, H, D, e) == int(golden["bpt_llama31_70b"][0]) == 327680


@pytest.mark.parametrize("L,kib", [(8, 32), (32, 128), (64, 256)])
def test_bytes_per_token_benchmark_geometries(L, kib):
    assert orc.bytes_per_token(L, 8, 128, 2) == kib * 1024


def test_bytes_per_token_rejects_nonpositive():
    for bad in [(0, 8, 128, 2), (8, 0, 128, 2), (8, 8, -1, 2), (8, 8, 128, 0)]:
        assert orc.bytes_per_token(*bad) == 0


def test_paper_context_sizes(golden):
    bpt = orc.bytes_per_token(80, 8, 128, 2)
    suffix = int(golden["suffix_tokens"][0]) * bpt
    ctx = int(golden["context_tokens"][0]) * bpt
    assert suffix == 983_040_000 and ctx == 2_752_512_000
    assert round(suffix / 1e9, 2) == golden["suffix_gb_printed"][0]
    assert round(ctx / 1e9, 2) == golden["context_gb_printed"][0]
    # the printed copy bandwidths are payload / time with that payload
    assert abs(ctx / golden["d2h_seconds"][0] / 1e9 - golden["d2h_gbs_printed"][0]) < 0.06
    assert abs(ctx / golden["h2d_seconds"][0] / 1e9 - golden["h2d_gbs_printed"][0]) < 0.1
    # an oracle image has exactly that many bytes
    p = orc.OrcPool(80, 8, 128, 2, 16, 1024, 1 << 40, with_data=False)
    assert p.admit(1, 8400)[0] == orc.OK and p.suspend_to_host([1])[0] == orc.OK
    assert p.info(1)[1]["image_bytes"] == ctx
    assert p.stats()["host_used"] == -(-ctx // 4096) * 4096


# ---- index arithmetic against numpy's own row-major rule -------------------------

def test_offsets_match_numpy_strides():
    rng = np.random.default_rng(0)
    for _ in range(200):
        L, H, D, e, BS, NB = (int(rng.integers(1, 5)) for _ in range(6))
        n = int(rng.integers(1, 40))
        l, kv = int(rng.integers(L)), int(rng.integers(2))
        blk, slot, h, d, b = (int(rng.integers(x)) for x in (NB, BS, H, D, e))
        t = int(rng.integers(n))
        assert orc.pool_offset(L, H, D, e, BS, NB, l, kv, blk, slot, h, d, b) == \
            np.ravel_multi_index((l, kv, blk, slot, h, d, b), (L, 2, NB, BS, H, D, e))
        assert orc.image_offset(L, H, D, e, n, l, kv, t, h, d, b) == \
            np.ravel_multi_index((l, kv, t, h, d, b), (L, 2, n, H, D, e))


def test_offsets_are_64_bit():
    # last byte of a 144 GiB pool and of a 16 GiB image
    L, H, D, e, BS, NB = 32, 8, 128, 2, 8, 147456
    assert orc.pool_offset(L, H, D, e, BS, NB, L - 1, 1, NB - 1, BS - 1, H - 1, D - 1, e - 1) == \
        L * 2 * NB * BS * H * D * e - 1
    n = 131072
    assert orc.image_offset(L, H, D, e, n, L - 1, 1, n - 1, H - 1, D - 1, e - 1) == n * 131072 - 1


# ---- gather / scatter: brute force with a dictionary, numpy fancy indexing ---------

def dict_gather(pool, L, H, D, e, BS, NB, bt, n):
    """Third formulation: name every pool byte by (layer, plane, block, slot, head, dim, byte)
    in a dictionary, then list the image in its own nested order."""
    names = {}
    it = iter(pool.tolist())
    for key in itertools.product(range(L), range(2), range(NB), range(BS), range(H), range(D), range(e)):
        names[key] = next(it)
    out = []
    for l, kv, t, h, d, b in itertools.product(range(L), range(2), range(n), range(H), range(D), range(e)):
        out.append(names[(l, kv, bt[t // BS], t % BS, h, d, b)])
    return np.asarray(out, dtype=np.uint8)


def test_gather_brute_force_every_table():
    rng = np.random.default_rng(1)
    cases = 0
    for NB, BS in [(3, 1), (4, 2), (3, 3), (6, 1), (5, 2)]:
        for L, H, D, e in [(1, 1, 1, 1), (2, 1, 2, 1), (1, 2, 1, 2), (2, 2, 2, 1)]:
            pool = rng.integers(0, 256, size=L * 2 * NB * BS * H * D * e, dtype=np.uint8)
            for nb in range(0, min(NB, 4) + 1):
                for bt in itertools.permutations(range(NB), nb):
                    lo = (nb - 1) * BS + 1 if nb else 0
                    for n in range(lo, nb * BS + 1):
                        got = orc.gather(pool, L, H, D, e, BS, NB, bt, n)
                        want = dict_gather(pool, L, H, D, e, BS, NB, bt, n)
                        assert np.array_equal(got, want), (NB, BS, L, H, D, e, bt, n)
                        cases += 1
    assert cases > 4000


def numpy_gather(pool, L, H, D, e, BS, NB, bt, n):
    row = H * D * e
    v = pool.reshape(L, 2, NB, BS, row)
    return v[:, :, np.asarray(bt, dtype=np.int64)].reshape(L, 2, -1, row)[:, :, :n].reshape(-1)


@pytest.mark.parametrize("n", [0, 1, 15, 16, 17, 160, 163])
def test_gather_equals_numpy_fancy_indexing(n):
    L, H, D, e, BS, NB = 3, 2, 8, 2, 16, 40
    pool = fill_bytes(7, n, L * 2 * NB * BS * H * D * e)
    rng = np.random.default_rng(n)
    nb = -(-n // BS)
    for bt in (np.arange(nb), rng.permutation(NB)[:nb]):
        got = orc.gather(pool, L, H, D, e, BS, NB, bt, n)
        assert np.array_equal(got, numpy_gather(pool, L, H, D, e, BS, NB, bt, n))


def test_identity_table_is_a_plain_slice():
    # with bt = 0..nb-1 and n a multiple of BS each plane's image is the first n token rows of the plane
    L, H, D, e, BS, NB = 2, 2, 4, 2, 4, 8
    pool = fill_bytes(3, 0, L * 2 * NB * BS * H * D * e)
    n = 5 * BS
    img = orc.gather(pool, L, H, D, e, BS, NB, np.arange(5), n).reshape(L, 2, n * H * D * e)
    planes = pool.reshape(L, 2, NB * BS * H * D * e)
    assert np.array_equal(img, planes[:, :, : n * H * D * e])


def test_scatter_is_inverse_and_touches_only_valid_slots():
    L, H, D, e, BS, NB = 2, 2, 4, 2, 4, 12
    row = H * D * e
    rng = np.random.default_rng(5)
    for n in [1, 3, 4, 5, 11, 12, 19]:
        nb = -(-n // BS)
        pool = fill_bytes(11, n, L * 2 * NB * BS * row).copy()
        src = rng.permutation(NB)[:nb]
        img = orc.gather(pool, L, H, D, e, BS, NB, src, n)
        before = pool.copy()
        dst = rng.permutation(NB)[:nb]
        orc.scatter(pool, img, L, H, D, e, BS, NB, dst, n)
        # logical content under the new table equals the image
        assert np.array_equal(orc.gather(pool, L, H, D, e, BS, NB, dst, n), img)
        # every byte outside the valid slots of the destination blocks is unchanged
        mask = np.zeros((L, 2, NB, BS, row), dtype=bool)
        for t in range(n):
            mask[:, :, dst[t // BS], t % BS, :] = True
        changed = (pool != before).reshape(mask.shape)
        assert not (changed & ~mask).any()
        # and the valid slots hold exactly the image rows
        v = pool.reshape(L, 2, NB, BS, row)
        im = img.reshape(L, 2, n, row)
        for t in range(n):
            assert np.array_equal(v[:, :, dst[t // BS], t % BS], im[:, :, t])


def test_transposed_or_swapped_planes_would_fail():
    # K and V planes, and layers, carry different bytes: the image keeps plane 0 before plane 1
    L, H, D, e, BS, NB = 2, 1, 2, 1, 2, 3
    pool = np.zeros((L, 2, NB, BS, H * D * e), dtype=np.uint8)
    for l in range(L):
        for kv in range(2):
            pool[l, kv] = 10 * l + kv + 1
    img = orc.gather(pool.reshape(-1), L, H, D, e, BS, NB, [2, 0], 3).reshape(L, 2, 3 * H * D * e)
    assert (img[0, 0] == 1).all() and (img[0, 1] == 2).all() and (img[1, 0] == 11).all() and (img[1, 1] == 12).all()


# ---- block-major pool layout [NB][L][2][BS][H][D][e]: same pins ------------------------

def test_block_major_offsets_match_numpy_strides():
    rng = np.random.default_rng(3)
    for _ in range(200):
        L, H, D, e, BS, NB = (int(rng.integers(1, 5)) for _ in range(6))
        l, kv = int(rng.integers(L)), int(rng.integers(2))
        blk, slot, h, d, b = (int(rng.integers(x)) for x in (NB, BS, H, D, e))
        assert orc.pool_offset(L, H, D, e, BS, NB, l, kv, blk, slot, h, d, b, layout=orc.BLOCK_MAJOR) == \
            np.ravel_multi_index((blk, l, kv, slot, h, d, b), (NB, L, 2, BS, H, D, e))


def dict_gather_block_major(pool, L, H, D, e, BS, NB, bt, n):
    names = {}
    it = iter(pool.tolist())
    for key in itertools.product(range(NB), range(L), range(2), range(BS), range(H), range(D), range(e)):
        names[key] = next(it)
    out = [names[(bt[t // BS], l, kv, t % BS, h, d, b)]
           for l, kv, t, h, d, b in itertools.product(range(L), range(2), range(n), range(H), range(D), range(e))]
    return np.asarray(out, dtype=np.uint8)


def test_block_major_gather_brute_force_and_numpy():
    rng = np.random.default_rng(4)
    cases = 0
    for NB, BS in [(3, 1), (4, 2), (3, 3)]:
        for L, H, D, e in [(1, 1, 1, 1), (2, 1, 2, 1), (2, 2, 1, 2)]:
            pool = rng.integers(0, 256, size=NB * L * 2 * BS * H * D * e, dtype=np.uint8)
            for nb in range(0, NB + 1):
                for bt in itertools.permutations(range(NB), nb):
                    for n in range((nb - 1) * BS + 1 if nb else 0, nb * BS + 1):
                        got = orc.gather(pool, L, H, D, e, BS, NB, bt, n, layout=orc.BLOCK_MAJOR)
                        assert np.array_equal(got, dict_gather_block_major(pool, L, H, D, e, BS, NB, bt, n))
                        if nb:
                            v = pool.reshape(NB, L, 2, BS, H * D * e)[np.asarray(bt)]          # [nb][L][2][BS][row]
                            want = v.transpose(1, 2, 0, 3, 4).reshape(L, 2, nb * BS, -1)[:, :, :n].reshape(-1)
                            assert np.array_equal(got, want)
                        cases += 1
    assert cases > 500


def test_block_major_scatter_round_trip_and_pool_object():
    L, H, D, e, BS, NB = 2, 2, 4, 2, 4, 10
    rng = np.random.default_rng(6)
    p = orc.OrcPool(L, H, D, e, BS, NB, 1 << 20, initial_free_order=rng.permutation(NB), layout=orc.BLOCK_MAJOR)
    p.data[:] = fill_bytes(6, 0, p.data.size)
    p.admit(1, 13)
    tbl = p.info(1)[1]["blocks"]
    want = orc.gather(p.data, L, H, D, e, BS, NB, tbl, 13, layout=orc.BLOCK_MAJOR).copy()
    before = p.data.copy()
    p.suspend_to_host([1])
    assert np.array_equal(p.info(1)[1]["image"], want) and np.array_equal(p.data, before)
    p.data.reshape(NB, -1)[p.free_queue()] ^= 0xFF
    mid = p.data.copy()
    p.resume_from_host([1])
    new = p.info(1)[1]["blocks"]
    assert np.array_equal(orc.gather(p.data, L, H, D, e, BS, NB, new, 13, layout=orc.BLOCK_MAJOR), want)
    # only the valid slots of the destination blocks changed
    mask = np.zeros((NB, L, 2, BS, H * D * e), dtype=bool)
    for t in range(13):
        mask[new[t // BS], :, :, t % BS] = True
    assert not ((p.data != mid).reshape(mask.shape) & ~mask).any()
