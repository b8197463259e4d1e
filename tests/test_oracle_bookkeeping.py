"""Pins for the oracle's bookkeeping: hand-worked allocator and arena sequences,
the state table of the three retention states, the paper's occupancy
arithmetic, conservation invariants and round trips under relabelling."""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle as orc
from kvr_synth import fill_bytes, free_order

GEOM = (2, 2, 4, 2, 4)           # L, H, D, e, BS -> 64 bytes per token
BPT = 2 * 2 * 2 * 4 * 2


def mk(NB=16, cap=1 << 20, order=None, data=True, geom=GEOM):
    return orc.OrcPool(*geom, NB, cap, initial_free_order=order, with_data=data)


def check_invariants(p, ids):
    """Conservation, disjointness, host accounting: properties that hold after every call."""
    s = p.stats()
    seen = list(p.free_queue())
    held = 0
    host = 0
    for rid in ids:
        stt, d = p.info(rid)
        if stt != orc.OK:
            continue
        if d["state"] in (orc.ACTIVE, orc.RETAINED):
            seen += list(d["blocks"])
            held += d["nb"]
        if d["state"] == orc.HOST:
            host += -(-d["image_bytes"] // 4096) * 4096
    assert s["blocks_free"] + held == p.NB == s["blocks_total"]
    assert s["blocks_active"] + s["blocks_pinned"] == held
    assert sorted(seen) == list(range(p.NB))
    assert s["host_used"] == host <= s["host_capacity"]
    assert s["bytes_suspended"] - s["bytes_resumed"] - s["bytes_expired_from_host"] >= 0


# ---- free queue: FIFO, worked by hand ----------------------------------------

def test_free_queue_fifo_by_hand():
    p = mk(NB=8)
    assert p.admit(1, 9)[1].tolist() == [0, 1, 2]          # ceil(9/4) = 3 blocks from the head
    assert p.admit(2, 4)[1].tolist() == [3]
    assert p.free_queue().tolist() == [4, 5, 6, 7]
    assert p.suspend_to_host([1]) == (orc.OK, [orc.OK])    # 0,1,2 go to the tail in logical order
    assert p.free_queue().tolist() == [4, 5, 6, 7, 0, 1, 2]
    assert p.resume_from_host([1]) == (orc.OK, [orc.OK])   # takes the three oldest free ids
    assert p.info(1)[1]["blocks"].tolist() == [4, 5, 6]
    assert p.free_queue().tolist() == [7, 0, 1, 2]
    assert p.release(2) == orc.OK
    assert p.free_queue().tolist() == [7, 0, 1, 2, 3]


def test_initial_free_order_is_respected_and_validated():
    order = free_order(3, 16)
    p = mk(NB=16, order=order)
    assert p.admit(1, 20)[1].tolist() == order[:5].tolist()
    with pytest.raises(ValueError):
        mk(NB=4, order=[0, 1, 1, 3])
    with pytest.raises(ValueError):
        mk(NB=4, order=[0, 1, 2, 4])


def test_resume_into_named_blocks():
    p = mk(NB=8)
    p.admit(1, 8)
    p.suspend_to_host([1])                                  # free: 2..7, 0, 1
    assert p.resume_from_host_into(1, [7, 7]) == orc.ERR_INVALID_ARG
    assert p.resume_from_host_into(1, [7]) == orc.ERR_INVALID_ARG
    p.admit(2, 4)                                           # takes block 2
    assert p.resume_from_host_into(1, [2, 3]) == orc.ERR_INVALID_ARG   # 2 is live
    assert p.resume_from_host_into(1, [6, 0]) == orc.OK
    assert p.info(1)[1]["blocks"].tolist() == [6, 0]
    assert p.free_queue().tolist() == [3, 4, 5, 7, 1]       # the others keep their order


def test_admit_into_named_blocks():
    p = mk(NB=8)
    assert p.admit_into(1, 9, [5, 2]) == orc.ERR_INVALID_ARG            # 9 tokens need 3 blocks
    assert p.admit_into(1, 9, [5, 2, 2]) == orc.ERR_INVALID_ARG
    assert p.admit_into(1, 9, [5, 2, 8]) == orc.ERR_INVALID_ARG
    assert p.admit_into(1, 9, [5, 2, 7]) == orc.OK
    assert p.info(1)[1]["blocks"].tolist() == [5, 2, 7] and p.free_queue().tolist() == [0, 1, 3, 4, 6]
    assert p.admit_into(2, 4, [5]) == orc.ERR_INVALID_ARG               # 5 is live now
    assert p.admit_into(1, 4, [0]) == orc.ERR_BAD_STATE
    assert p.admit_into(3, 0, []) == orc.OK and p.info(3)[1]["nb"] == 0
    p.expire([1])
    assert p.free_queue().tolist() == [0, 1, 3, 4, 6, 5, 2, 7] and p.admit_into(1, 4, [7]) == orc.OK
    check_invariants(p, [1, 2, 3])


# ---- host arena: first fit, 4 KiB granules, worked by hand --------------------------

def test_arena_first_fit_by_hand():
    # 64 B/token: 100 tokens -> 6400 B -> 8192 B range; 64 tokens -> 4096 B; 10 tokens -> 640 B -> 4096 B
    p = mk(NB=128, cap=5 * 4096, data=False)
    for rid, n in [(1, 100), (2, 64), (3, 10), (4, 64)]:
        assert p.admit(rid, n)[0] == orc.OK
    assert p.suspend_to_host([1, 2, 3])[1] == [orc.OK] * 3
    assert [p.info(r)[1]["arena_offset"] for r in (1, 2, 3)] == [0, 8192, 12288]
    s = p.stats()
    assert s["host_used"] == 16384 and s["host_largest_hole"] == 4096
    # full: a 2-granule image does not fit in the one free granule; nobody is displaced
    p.admit(5, 100)
    assert p.suspend_to_host([5]) == (orc.HOST_FULL, [orc.HOST_FULL])
    assert p.info(5)[1]["state"] == orc.ACTIVE and p.stats()["host_full_rejects"] == 1
    # expiry frees capacity for a later arrival (Appendix D): drop request 1, then 5 fits at offset 0
    assert p.expire([1])[0] == orc.OK
    assert p.suspend_to_host([5])[0] == orc.OK and p.info(5)[1]["arena_offset"] == 0
    # lowest hole first: free 2 (hole at 8192), the next one-granule image lands there, not at the end
    assert p.resume_from_host([2])[0] == orc.OK
    assert p.suspend_to_host([4])[0] == orc.OK and p.info(4)[1]["arena_offset"] == 8192
    check_invariants(p, range(1, 6))


def test_zero_token_request_holds_nothing():
    p = mk(NB=4, cap=4096)
    assert p.admit(1, 0) [0] == orc.OK and p.info(1)[1]["nb"] == 0
    assert p.suspend_to_host([1])[0] == orc.OK
    assert p.stats()["host_used"] == 0 and p.info(1)[1]["image_bytes"] == 0
    assert p.resume_from_host([1])[0] == orc.OK and p.info(1)[1]["state"] == orc.ACTIVE


# ---- the three retention states and their transitions (Section 3.1, Appendix D) ---

def fresh(state):
    p = mk(NB=8, cap=1 << 16)
    p.admit(1, 6)
    if state == orc.RETAINED:
        p.retain_in_hbm([1])
    if state == orc.HOST:
        p.suspend_to_host([1])
    if state == orc.EXPIRED:
        p.expire([1])
    assert p.info(1)[1]["state"] == state
    return p


TABLE = {
    # (state, call): (status, new state)
    (orc.ACTIVE, "retain"): (orc.OK, orc.RETAINED),
    (orc.ACTIVE, "suspend"): (orc.OK, orc.HOST),
    (orc.ACTIVE, "expire"): (orc.OK, orc.EXPIRED),
    (orc.ACTIVE, "resume"): (orc.ERR_BAD_STATE, orc.ACTIVE),
    (orc.RETAINED, "retain"): (orc.ERR_BAD_STATE, orc.RETAINED),
    (orc.RETAINED, "suspend"): (orc.OK, orc.HOST),
    (orc.RETAINED, "expire"): (orc.OK, orc.EXPIRED),
    (orc.RETAINED, "resume"): (orc.RESIDENT, orc.ACTIVE),      # beta_1 = 0: nothing moves
    (orc.HOST, "retain"): (orc.ERR_BAD_STATE, orc.HOST),
    (orc.HOST, "suspend"): (orc.ERR_BAD_STATE, orc.HOST),
    (orc.HOST, "expire"): (orc.OK, orc.EXPIRED),
    (orc.HOST, "resume"): (orc.OK, orc.ACTIVE),
    (orc.EXPIRED, "retain"): (orc.ERR_BAD_STATE, orc.EXPIRED),
    (orc.EXPIRED, "suspend"): (orc.ERR_BAD_STATE, orc.EXPIRED),
    (orc.EXPIRED, "expire"): (orc.ERR_BAD_STATE, orc.EXPIRED),  # one-shot
    (orc.EXPIRED, "resume"): (orc.RECOMPUTE, orc.EXPIRED),
}


@pytest.mark.parametrize("state,call", sorted(TABLE))
def test_transition_table(state, call):
    p = fresh(state)
    fn = dict(retain=p.retain_in_hbm, suspend=p.suspend_to_host, expire=p.expire, resume=p.resume_from_host)[call]
    want_status, want_state = TABLE[(state, call)]
    assert fn([1]) == (want_status, [want_status])
    assert p.info(1)[1]["state"] == want_state
    check_invariants(p, [1])


def test_resident_resume_keeps_the_block_table():
    p = mk(NB=8)
    blocks = p.admit(1, 10)[1].tolist()
    p.retain_in_hbm([1])
    assert p.stats()["blocks_pinned"] == 3
    assert p.resume_from_host([1])[0] == orc.RESIDENT
    assert p.info(1)[1]["blocks"].tolist() == blocks and p.stats()["blocks_pinned"] == 0


def test_unknown_request_and_batch_folding():
    p = mk(NB=8)
    p.admit(1, 4)
    p.admit(2, 4)
    p.retain_in_hbm([2])
    assert p.suspend_to_host([9]) == (orc.ERR_UNKNOWN_REQUEST, [orc.ERR_UNKNOWN_REQUEST])
    # errors dominate positive outcomes; among non-errors the largest code is returned
    assert p.resume_from_host([2, 1, 9]) == (orc.ERR_BAD_STATE, [orc.RESIDENT, orc.ERR_BAD_STATE, orc.ERR_UNKNOWN_REQUEST])
    # a request named twice is handled in order
    assert p.suspend_to_host([1, 1]) == (orc.ERR_BAD_STATE, [orc.OK, orc.ERR_BAD_STATE])
    assert p.admit(1, 4)[0] == orc.ERR_BAD_STATE
    assert p.admit(3, -1)[0] == orc.ERR_INVALID_ARG


def test_expired_request_can_be_readmitted_or_released():
    p = mk(NB=8)
    p.admit(1, 8)
    p.expire([1])
    assert p.stats()["recompute_marked"] == 1 and p.stats()["blocks_free"] == 8
    assert p.resume_from_host([1])[0] == orc.RECOMPUTE
    assert p.admit(1, 12)[0] == orc.OK and p.info(1)[1]["nb"] == 3   # recompute done by the caller
    assert p.release(1) == orc.OK and p.info(1)[0] == orc.ERR_UNKNOWN_REQUEST
    assert p.stats()["blocks_free"] == 8


def test_hbm_full_leaves_everything_unchanged():
    p = mk(NB=4)
    p.admit(1, 16)
    p.suspend_to_host([1])
    p.admit(2, 5)                                           # 2 of 4 blocks
    before = (p.free_queue().tolist(), p.stats()["host_used"])
    assert p.resume_from_host([1])[0] == orc.HBM_FULL
    assert (p.free_queue().tolist(), p.stats()["host_used"]) == before
    assert p.info(1)[1]["state"] == orc.HOST and p.stats()["hbm_full_rejects"] == 1
    assert p.admit(3, 9)[0] == orc.HBM_FULL


# ---- the paper's occupancy arithmetic (Appendix A) ------------------------------

def test_paper_pool_occupancy(golden):
    pool_tokens = int(golden["pool_tokens"][0])
    ctx = int(golden["context_tokens"][0])
    NB = pool_tokens // 16
    assert NB == 42548
    p = orc.OrcPool(80, 8, 128, 2, 16, NB, 0, with_data=False)
    occ = {}
    n = 0
    while True:
        st_, _ = p.admit(1000 + n, ctx)
        if st_ != orc.OK:
            assert st_ == orc.HBM_FULL
            break
        n += 1
        s = p.stats()
        occ[n] = 100.0 * (s["blocks_total"] - s["blocks_free"]) / s["blocks_total"]
        assert s["blocks_active"] == 525 * n
    assert n == int(golden["fill_contexts"][0])             # "around N ~ 81 ... fills the pool"
    for N, pct in zip(golden["sweep_contexts"], golden["sweep_occupancy_pct"]):
        assert abs(occ[int(N)] - pct) < 0.6                 # "approximately 31/62/80/89 %"


# ---- data: suspend leaves the pool alone, resume restores content under any relabelling ---

def logical(p, rid):
    d = p.info(rid)[1]
    L, H, D, e, BS = p.geom
    return orc.gather(p.data, L, H, D, e, BS, p.NB, d["blocks"], d["n_tokens"])


def test_suspend_does_not_touch_the_pool_and_image_is_logical_content():
    p = mk(NB=16, order=free_order(1, 16))
    p.data[:] = fill_bytes(1, 0, p.data.size)
    p.admit(1, 13)
    want = logical(p, 1).copy()
    before = p.data.copy()
    p.suspend_to_host([1])
    assert np.array_equal(p.data, before)
    assert np.array_equal(p.info(1)[1]["image"], want) and want.size == 13 * BPT


@settings(max_examples=60, deadline=None, derandomize=True)
@given(st.integers(0, 2**31), st.lists(st.integers(0, 36), min_size=1, max_size=5))
def test_round_trip_under_any_relabelling(seed, lengths):
    NB = 48
    rng = np.random.default_rng(seed)
    p = mk(NB=NB, order=rng.permutation(NB))
    p.data[:] = fill_bytes(seed, 1, p.data.size)
    ids = list(range(1, len(lengths) + 1))
    for rid, n in zip(ids, lengths):
        assert p.admit(rid, n)[0] == orc.OK
    want = {rid: logical(p, rid).copy() for rid in ids}
    assert p.suspend_to_host(ids)[0] == orc.OK
    check_invariants(p, ids)
    # overwrite every free block so stale bytes cannot fake a pass
    v = p.data.reshape(GEOM[0], 2, NB, -1)
    v[:, :, p.free_queue()] ^= 0xFF
    for rid in ids:
        nb = p.info(rid)[1]["nb"]
        if rng.random() < 0.5:
            assert p.resume_from_host([rid])[0] == orc.OK
        else:
            dst = rng.permutation(p.free_queue())[:nb]
            assert p.resume_from_host_into(rid, dst) == orc.OK
            assert p.info(rid)[1]["blocks"].tolist() == dst.tolist()
        check_invariants(p, ids)
    for rid in ids:
        assert np.array_equal(logical(p, rid), want[rid])
    s = p.stats()
    assert s["bytes_suspended"] == s["bytes_resumed"] == sum(lengths) * BPT and s["host_used"] == 0
