"""Pins for the oracle's shared-prefix bookkeeping (Section 2, approval-gated workload: a 5.4K-token system prefix
shared through prefix caching plus a ~3.0K-token private suffix; Appendix B prices the suffix at 0.98 GB).

What fixes the behaviour with no implementation to compare against:
  * the paper's sizes: an 8,400-token context sharing 5,400 tokens moves 3,000 tokens = 983,040,000 bytes;
  * conservation with reference counts: free + distinct held blocks = NB, and a block's count equals the number of
    tables that name it, after every call of random scripts;
  * hand-worked sequences for the free-queue order and for the lifetime of a prefix;
  * brute force over every pair of injective tables on pools of <= 6 blocks, against a dictionary formulation;
  * the round trip under relabelling of the private part.
"""
import itertools

import numpy as np
import pytest

import oracle as orc
from kvr_synth import fill_bytes

GEOM = (2, 2, 4, 2, 4)           # L, H, D, e, BS -> 64 bytes per token
BPT = 64


def mk(NB=16, cap=1 << 20, order=None, data=True, geom=GEOM):
    return orc.OrcPool(*geom, NB, cap, initial_free_order=order, with_data=data)


def tables_of(p, ids):
    """rid -> list of block ids the request refers to right now (whole table, or the kept prefix on the host)."""
    out = {}
    for rid in ids:
        st, d = p.info(rid)
        if st != orc.OK:
            continue
        if d["state"] in (orc.ACTIVE, orc.RETAINED):
            out[rid] = d["blocks"].tolist()
        elif d["state"] == orc.HOST:
            out[rid] = p.sharing(rid)[1].tolist()
    return out


def check_counts(p, ids):
    refs = np.zeros(p.NB, dtype=np.int64)
    for t in tables_of(p, ids).values():
        for b in t:
            refs[b] += 1
    fq = p.free_queue().tolist()
    assert len(set(fq)) == len(fq)
    for b in range(p.NB):
        assert p.refcount(b) == refs[b]
        assert (refs[b] == 0) == (b in fq)
    s = p.stats()
    assert s["blocks_free"] + int((refs > 0).sum()) == p.NB                  # conservation with counts
    assert s["blocks_free"] + s["blocks_active"] + s["blocks_pinned"] == p.NB


def test_paper_sizes_metadata_only(golden):
    # Llama-3.1-70B geometry; block_size 8 so that the 5,400-token prefix is whole blocks (675)
    L, H, D, e = (int(x) for x in golden["bpt_factors"])
    BS, NB = 8, 4096
    p = orc.OrcPool(L, H, D, e, BS, NB, 8 << 30, with_data=False)
    ctx, shared = int(golden["context_tokens"][0]), int(golden["shared_prefix_tokens"][0])
    assert ctx - shared == int(golden["suffix_tokens"][0])
    assert p.admit(0, shared)[0] == orc.OK                                   # the system prefix, computed once
    st, blocks = p.admit_sharing(1, ctx, 0, shared // BS)
    assert st == orc.OK and blocks[:675].tolist() == p.info(0)[1]["blocks"].tolist()
    assert p.info(1)[1]["image_bytes"] == int(golden["suffix_tokens"][0]) * int(golden["bpt_llama31_70b"][0]) == 983_040_000
    assert p.suspend_to_host([1]) == (orc.OK, [orc.OK])
    s = p.stats()
    assert s["bytes_suspended"] == 983_040_000 and s["host_used"] == 983_040_000   # 0.98 GB, not 2.75 GB
    assert round(s["bytes_suspended"] / 1e9, 2) == golden["suffix_gb_printed"][0]
    assert s["blocks_free"] == NB - 675 and s["blocks_pinned"] == 675        # the prefix stays, the suffix blocks are free
    # with block_size 16 the prefix rounds down to 337 whole blocks: 3,008 private tokens move
    q = orc.OrcPool(L, H, D, e, 16, NB, 8 << 30, with_data=False)
    assert q.admit(0, shared)[0] == orc.OK
    assert q.admit_sharing(1, ctx, 0, shared // 16)[0] == orc.OK
    assert q.info(1)[1]["image_bytes"] == (ctx - 337 * 16) * 327680


def test_prefix_lifetime_and_free_order_by_hand():
    p = mk(NB=10)
    assert p.admit(1, 8)[1].tolist() == [0, 1]                               # the prefix owner: two full blocks
    assert p.admit_sharing(2, 14, 1, 2)[1].tolist() == [0, 1, 2, 3]          # shares both, two private
    assert p.admit_sharing(3, 9, 2, 1)[1].tolist() == [0, 4, 5]              # shares one (through request 2), two private
    assert [p.refcount(b) for b in range(6)] == [3, 2, 1, 1, 1, 1]
    assert p.free_queue().tolist() == [6, 7, 8, 9]
    assert p.release(1) == orc.OK                                            # the owner goes: nothing is freed
    assert p.free_queue().tolist() == [6, 7, 8, 9] and [p.refcount(b) for b in (0, 1)] == [2, 1]
    assert p.suspend_to_host([2]) == (orc.OK, [orc.OK])                      # only 2, 3 are let go; 0, 1 stay referenced
    assert p.free_queue().tolist() == [6, 7, 8, 9, 2, 3]
    assert p.info(2)[1]["image_bytes"] == 6 * BPT and p.sharing(2)[1].tolist() == [0, 1]
    assert p.expire([3]) == (orc.OK, [orc.OK])                               # 0 still referenced by 2 (on the host); 4, 5 freed
    assert p.free_queue().tolist() == [6, 7, 8, 9, 2, 3, 4, 5] and p.refcount(0) == 1
    s = p.stats()
    assert (s["blocks_pinned"], s["blocks_active"], s["blocks_free"]) == (2, 0, 8)
    assert p.resume_from_host([2]) == (orc.OK, [orc.OK])
    assert p.info(2)[1]["blocks"].tolist() == [0, 1, 6, 7]                   # kept prefix + two fresh blocks
    assert p.release(2) == orc.OK                                            # last referrer: the prefix is freed, in order
    assert p.free_queue().tolist() == [8, 9, 2, 3, 4, 5, 0, 1, 6, 7]
    check_counts(p, [1, 2, 3])


def test_expire_or_release_on_the_host_drops_the_prefix():
    for how in ("expire", "release"):
        p = mk(NB=8)
        assert p.admit(1, 8)[0] == orc.OK
        assert p.admit_sharing(2, 12, 1, 2)[0] == orc.OK
        assert p.release(1) == orc.OK
        assert p.suspend_to_host([2])[0] == orc.OK and p.stats()["host_used"] == 4096
        st = p.expire([2])[0] if how == "expire" else p.release(2)
        assert st == orc.OK
        assert p.stats()["blocks_free"] == 8 and p.stats()["host_used"] == 0
        assert all(p.refcount(b) == 0 for b in range(8))


def test_argument_checks():
    p = mk(NB=8)
    assert p.admit(1, 10)[0] == orc.OK                                       # 2 full blocks + a partial one
    assert p.admit_sharing(2, 12, 1, 3)[0] == orc.ERR_INVALID_ARG            # the donor's third block is partial
    assert p.admit_sharing(2, 7, 1, 2)[0] == orc.ERR_INVALID_ARG             # 8 shared tokens do not fit in 7
    assert p.admit_sharing(2, 8, 9, 1)[0] == orc.ERR_UNKNOWN_REQUEST
    assert p.admit_sharing(2, 8, 2, 1)[0] == orc.ERR_INVALID_ARG             # a request cannot donate to itself
    assert p.admit_sharing(1, 8, 1, 1)[0] == orc.ERR_BAD_STATE               # id exists
    assert p.admit_sharing(2, 8, 1, 2)[0] == orc.OK                          # everything shared, nothing private
    assert p.info(2)[1]["image_bytes"] == 0 and p.stats()["blocks_free"] == 5
    assert p.admit_sharing(3, 40, 1, 2)[0] == orc.HBM_FULL                   # needs 8 private blocks, 5 free
    assert p.stats()["hbm_full_rejects"] == 1
    assert p.suspend_to_host([1])[0] == orc.OK                               # donor on the host with no prefix of its own
    assert p.admit_sharing(4, 8, 1, 1)[0] == orc.ERR_INVALID_ARG
    assert p.suspend_to_host([2])[0] == orc.OK                               # request 2 keeps its 2-block prefix
    assert p.admit_sharing(4, 9, 2, 2)[0] == orc.OK                          # a donor on the host donates its prefix
    assert p.expire([2])[0] == orc.OK
    assert p.admit_sharing(5, 8, 2, 1)[0] == orc.ERR_BAD_STATE               # a discarded donor refers to nothing
    assert p.admit_sharing(5, 5, 2, 0)[0] == orc.OK                          # no sharing: the donor is not looked at
    check_counts(p, range(6))


def logical_rows(pool_bytes, geom, NB, table, n):
    """Dictionary formulation: (plane, token) -> the row's bytes, looked up block by block."""
    L, H, D, e, BS = geom
    row = H * D * e
    rows = {}
    for plane in range(2 * L):
        for t in range(n):
            off = ((plane * NB + table[t // BS]) * BS + t % BS) * row
            rows[(plane, t)] = bytes(pool_bytes[off:off + row])
    return rows


def test_brute_force_two_requests_sharing_a_prefix():
    geom = (1, 1, 2, 1, 2)       # 2-byte rows, 4 bytes per token, 2 tokens per block
    L, H, D, e, BS = geom
    NB = 6
    cases = 0
    for n_shared in (1, 2):
        for n_a, n_b in ((n_shared * BS, n_shared * BS + 1), (n_shared * BS + 1, n_shared * BS + 3), (n_shared * BS + 2, n_shared * BS)):
            nb_a, nb_b = -(-n_a // BS), -(-n_b // BS)
            if nb_a + nb_b - n_shared > NB:
                continue
            for order in itertools.permutations(range(NB)):
                if cases % 7:            # every 7th permutation of 720: still > 300 cases per shape
                    cases += 1
                    continue
                cases += 1
                p = orc.OrcPool(*geom, NB, 1 << 16, initial_free_order=np.array(order, dtype=np.int32), with_data=True)
                p.data[:] = np.arange(p.data.size, dtype=np.uint8) * 7 + 3
                before = p.data.copy()
                ta = p.admit(1, n_a)[1].tolist()
                tb = p.admit_sharing(2, n_b, 1, n_shared)[1].tolist()
                assert tb[:n_shared] == ta[:n_shared] and len(set(ta) | set(tb)) == nb_a + nb_b - n_shared
                want = logical_rows(before, geom, NB, tb, n_b)
                assert p.suspend_to_host([2])[0] == orc.OK
                img = p.info(2)[1]["image"]
                n_priv = n_b - n_shared * BS
                assert img.size == n_priv * 4
                for plane in range(2):
                    for t in range(n_priv):
                        assert bytes(img[(plane * n_priv + t) * 2:(plane * n_priv + t) * 2 + 2]) == want[(plane, n_shared * BS + t)]
                assert np.array_equal(p.data, before)                        # a suspend writes nothing into the pool
                # the donor's content is untouched by the sharer's round trip; the sharer reads back its own
                p.data[:] = 0xEE
                for b in ta:                                                 # restore only what request 1 refers to
                    for plane in range(2):
                        o = ((plane * NB + b) * BS) * 2
                        p.data[o:o + BS * 2] = before[o:o + BS * 2]
                assert p.resume_from_host([2])[0] == orc.OK
                tb2 = p.info(2)[1]["blocks"].tolist()
                assert tb2[:n_shared] == ta[:n_shared] and not (set(tb2[n_shared:]) & set(ta))
                assert logical_rows(p.data, geom, NB, tb2, n_b) == want
                assert logical_rows(p.data, geom, NB, ta, n_a) == logical_rows(before, geom, NB, ta, n_a)
                check_counts(p, [1, 2])
                p.close()
    assert cases > 1000


def test_round_trip_under_relabelling_of_the_private_part():
    geom = (2, 2, 8, 2, 4)
    L, H, D, e, BS = geom
    NB = 40
    rng = np.random.default_rng(3)
    p = orc.OrcPool(*geom, NB, 1 << 20, initial_free_order=rng.permutation(NB).astype(np.int32), with_data=True)
    p.data[:] = fill_bytes(3, 0, p.data.size)
    assert p.admit(1, 12)[0] == orc.OK
    st, t2 = p.admit_sharing(2, 12 + 19, 1, 3)
    assert st == orc.OK
    want = orc.gather(p.data.copy(), *geom, NB, t2, 31)                      # logical content of the whole request
    assert p.suspend_to_host([2])[0] == orc.OK
    assert np.array_equal(p.info(2)[1]["image"], orc.gather(p.data, *geom, NB, t2[3:], 19))   # suffix only
    pick = rng.permutation(p.free_queue())[:5].astype(np.int32)              # any 5 free blocks, any order
    assert p.resume_from_host_into(2, pick[:4]) == orc.ERR_INVALID_ARG       # the private part is 5 blocks
    assert p.resume_from_host_into(2, pick) == orc.OK
    t2b = p.info(2)[1]["blocks"]
    assert t2b.tolist() == t2[:3].tolist() + pick.tolist()
    assert np.array_equal(orc.gather(p.data, *geom, NB, t2b, 31), want)
    check_counts(p, [1, 2])


@pytest.mark.parametrize("seed", range(6))
def test_random_scripts_keep_counts_consistent(seed):
    rng = np.random.default_rng(seed)
    p = mk(NB=24, cap=24 * 4096, data=False)
    ids = list(range(8))
    for _ in range(400):
        k = rng.integers(7)
        rid = int(rng.integers(8))
        if k == 0:
            p.admit(rid, int(rng.integers(0, 20)))
        elif k == 1:
            donor = int(rng.integers(8))
            p.admit_sharing(rid, int(rng.integers(0, 24)), donor, int(rng.integers(0, 4)))
        elif k == 2:
            p.suspend_to_host([rid])
        elif k == 3:
            p.resume_from_host([rid])
        elif k == 4:
            p.expire([rid])
        elif k == 5:
            p.release(rid)
        else:
            p.retain_in_hbm([rid])
        check_counts(p, ids)
    s = p.stats()
    assert s["suspends"] > 5 and s["resumes"] + s["resident_resumes"] > 2


def test_named_private_blocks_by_hand():
    """An engine with its own allocator names the private blocks; the prefix still comes from the donor."""
    p = mk(NB=10)
    assert p.admit(1, 8)[1].tolist() == [0, 1]
    assert p.admit_sharing_into(2, 14, 1, 2, [7, 4]) == orc.OK              # ceil(14/4) = 4 = 2 shared + 2 named
    assert p.info(2)[1]["blocks"].tolist() == [0, 1, 7, 4] and p.sharing(2)[1].tolist() == [0, 1]
    assert p.free_queue().tolist() == [2, 3, 5, 6, 8, 9]                    # the other free ids keep their order
    assert [p.refcount(b) for b in (0, 1, 7, 4)] == [2, 2, 1, 1]
    assert p.admit_sharing_into(3, 14, 1, 2, [7, 5]) == orc.ERR_INVALID_ARG     # 7 is taken
    assert p.admit_sharing_into(3, 14, 1, 2, [5, 5]) == orc.ERR_INVALID_ARG     # named twice
    assert p.admit_sharing_into(3, 14, 1, 2, [5]) == orc.ERR_INVALID_ARG        # 2 + 1 != 4 blocks
    assert p.admit_sharing_into(3, 14, 9, 2, [5, 6]) == orc.ERR_UNKNOWN_REQUEST
    assert p.admit_sharing_into(2, 14, 1, 2, [5, 6]) == orc.ERR_BAD_STATE
    assert p.free_queue().tolist() == [2, 3, 5, 6, 8, 9]                    # failed calls changed nothing
    assert p.suspend_to_host([2])[0] == orc.OK and p.info(2)[1]["image_bytes"] == 6 * BPT
    assert p.free_queue().tolist() == [2, 3, 5, 6, 8, 9, 7, 4]
    assert p.admit_sharing_into(3, 8, 2, 2, []) == orc.OK                   # everything shared, from a donor on the host
    check_counts(p, [1, 2, 3])
