"""The staged route's planner (host logic) without a GPU: kvr_test_plan returns the launches, link copies and
kernel segments planned for one move through a staging ring; a byte-level simulation of what the kernels and the
copies would do with that plan must reproduce every image exactly, stay inside the ring and inside each launch's
slots, never cross the ring's end inside a segment or a copy, and follow the sizing rules."""
import numpy as np
import pytest

from paper_2608_30830_b200 import kvr

GEOMS = [(2, 2, 16, 2, 4), (1, 1, 16, 1, 2), (3, 2, 16, 2, 8)]     # tiles of 256, 32 and 512 bytes


def tile_off(n, nb, BS, row, q):
    """Byte offset of tile q (plane-major, then block) inside an image of n tokens."""
    plane, b = divmod(q, nb)
    return (plane * n + b * BS) * row


def simulate(geom, lens, slot, slots, launch, ring_next, resume, flags=0, ss=0, rs=0):
    L, H, D, e, BS = geom
    row, bpt, planes = H * D * e, 2 * L * H * D * e, 2 * L
    tile = BS * row
    chunks, copies, segs, nxt = kvr.test_plan(geom, lens, slot, slots, launch, ring_next, resume, flags, ss, rs)
    S = slot * slots
    # where each image lives in the arena, and which item a table offset names
    lin_off, bt_off, lin, bt = [], {}, 0, 0
    for i, n in enumerate(lens):
        nb = -(-n // BS)
        lin_off.append(lin)
        if nb:
            bt_off[bt] = i
        lin += -(-n * bpt // 4096) * 4096
        bt += -(-nb * 4 // 16) * 16
    arena_bytes = max(lin, 1)
    want = np.zeros(arena_bytes, dtype=np.int64)                   # label of every image byte: item and offset
    for i, n in enumerate(lens):
        want[lin_off[i]:lin_off[i] + n * bpt] = (i + 1) * 10**9 + np.arange(n * bpt)
    got = np.zeros(arena_bytes, dtype=np.int64)
    first = ring_next
    ci = 0
    for k, (cf, cn, payload, ncop, sb, ns) in enumerate(chunks):
        assert cf == first and 1 <= cn <= launch, (k, cf, first, cn)
        ring = np.zeros(S, dtype=np.int64)                         # what this launch's kernel puts into the ring
        written = np.zeros(S, dtype=bool)
        seen = 0
        for off, img0, tb, tc, nb in segs[sb:sb + ns]:
            i = bt_off[off]
            n = lens[i]
            assert nb == -(-n // BS) and tc >= 1 and tb + tc <= planes * nb
            a = tile_off(n, nb, BS, row, tb)
            b = n * bpt if tb + tc == planes * nb else tile_off(n, nb, BS, row, tb + tc)
            lo, hi = img0 + a, img0 + b
            assert 0 <= lo < hi <= S, "a segment leaves the ring or wraps"
            v = (lo - cf * slot) % S                                # position inside the launch
            assert v + (hi - lo) <= cn * slot, "a segment leaves its launch's slots"
            assert not written[lo:hi].any(), "two segments of one launch overlap in the ring"
            written[lo:hi] = True
            # the kernel moves whole tiles (valid tokens only): tile q of the image lands at img0 + tile_off(q)
            ring[lo:hi] = (i + 1) * 10**9 + np.arange(a, b)
            seen += hi - lo
        assert seen == payload
        moved = 0
        for ck, cl, cr, cv, cb in copies[ci:ci + ncop]:
            assert ck == k and cb > 0
            assert cr == (cf * slot + cv) % S and cr + cb <= S, "a copy's ring offset disagrees with its position or wraps"
            assert cv + cb <= cn * slot
            assert written[cr:cr + cb].all(), "a copy reads ring bytes no segment wrote"
            assert (got[cl:cl + cb] == 0).all(), "an arena byte is copied twice"
            got[cl:cl + cb] = ring[cr:cr + cb]
            moved += cb
        ci += ncop
        assert moved == payload <= launch * slot
        first = (first + cn) % slots
    assert ci == len(copies) and nxt == first
    assert np.array_equal(got, want), "the plan does not reproduce the images"
    return chunks, copies


@pytest.mark.parametrize("seed", range(40))
def test_random_plans_reproduce_every_image(seed):
    rng = np.random.default_rng(seed)
    geom = GEOMS[seed % len(GEOMS)]
    L, H, D, e, BS = geom
    tile = BS * H * D * e
    slot = int(rng.choice([4096, 8192, 12288, 16384]))
    slots = int(rng.integers(2, 10))
    launch = int(rng.integers(1, slots))
    lens = [int(x) for x in rng.integers(0, 300, size=int(rng.integers(1, 10)))]
    for resume in (False, True):
        for flags in (0, kvr.LOW_LATENCY):
            simulate(geom, lens, slot, slots, launch, int(rng.integers(slots)), resume, flags,
                     ss=int(rng.choice([0, 4096, 65536])), rs=int(rng.choice([0, 4096, 65536])))


def test_sizing_rules_by_hand():
    geom = (2, 2, 16, 2, 4)                       # 256 bytes per token
    slot, slots, launch = 8192, 8, 7
    # a 100 KiB move, thresholds at 4 KiB: suspend = [slot][7 slots][rest], resume = [7 slots][rest - slot][slot]
    lens = [400]                                  # 102,400 bytes
    ch, _ = simulate(geom, lens, slot, slots, launch, 0, False, ss=4096, rs=4096)
    assert ch[0][2] <= slot and ch[0][1] == 1 and ch[1][2] > 6 * slot and ch[:, 2].sum() == 102400
    ch, _ = simulate(geom, lens, slot, slots, launch, 0, True, ss=4096, rs=4096)
    assert ch[0][2] > 6 * slot and ch[-1][2] <= slot + 256 and len(ch) == 3
    # below the threshold: one launch each way (it fits 7 slots? no: 102,400 > 57,344, so two launches, no small one)
    ch, _ = simulate(geom, lens, slot, slots, launch, 0, False, ss=1 << 20, rs=1 << 20)
    assert len(ch) == 2 and ch[0][2] > 6 * slot
    ch, _ = simulate(geom, [150], slot, slots, launch, 5, True, ss=1 << 20, rs=1 << 20)      # 38,400 bytes: one launch
    assert len(ch) == 1 and ch[0][0] == 5 and ch[0][1] == 5
    # low-latency resume: every request ends a launch
    lens = [60, 10, 90, 33]
    ch, cp = simulate(geom, lens, slot, slots, launch, 2, True, kvr.LOW_LATENCY, ss=1 << 20, rs=1 << 20)
    ends = np.cumsum(ch[:, 2])
    for total in np.cumsum([n * 256 for n in lens]):
        assert total in ends
    # a launch that wraps: it starts at slot 6 of 8 and covers 7 slots, so some segment starts again at offset 0
    ch, cp = simulate(geom, [220], slot, slots, launch, 6, False, ss=1 << 20)
    assert ch[0][0] == 6 and ch[0][1] >= 3 and (cp[:, 2] == 0).any()


def test_rejects_bad_arguments():
    with pytest.raises(kvr.KvrError):
        kvr.test_plan((2, 2, 16, 2, 4), [10], 8192, 4, 4)           # a launch may cover at most all slots but one
    with pytest.raises(kvr.KvrError):
        kvr.test_plan((2, 2, 16, 2, 4), [10], 100, 4, 3)            # slot size not a multiple of 4096
    with pytest.raises(kvr.KvrError):
        kvr.test_plan((2, 2, 16, 2, 4), [-1], 8192, 4, 3)
