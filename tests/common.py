"""Shared test helpers: a call-script generator and a runner that works on the oracle pool and on the
library pool alike (both expose the same method names), plus observation helpers."""
import numpy as np

import oracle as orc

COMMON_STATS = ["blocks_total", "blocks_free", "blocks_active", "blocks_pinned", "host_capacity", "host_used",
                "host_largest_hole", "n_active", "n_retained", "n_host", "n_expired", "suspends", "resumes",
                "resident_resumes", "expires", "recompute_marked", "host_full_rejects", "hbm_full_rejects",
                "bytes_suspended", "bytes_resumed", "bytes_expired_from_host"]


def random_script(seed, n_ops, max_tokens, n_ids=12, batch=4, sharing=False):
    """A seeded list of calls over a small id space; illegal calls are included on purpose.  With sharing=True
    some admissions name a donor and a number of shared prefix blocks (often illegal ones, on purpose)."""
    rng = np.random.default_rng(seed)
    ops = []
    kinds = ["admit", "admit", "admit_into", "retain", "suspend", "suspend", "expire", "resume", "resume",
             "resume_into", "release"]
    if sharing:
        kinds += ["admit_sharing", "admit_sharing", "admit_sharing", "admit_sharing_into"]
    for _ in range(n_ops):
        kind = rng.choice(kinds)
        if kind in ("admit_sharing", "admit_sharing_into"):
            ops.append((kind, int(rng.integers(n_ids)), int(rng.integers(0, max_tokens + 1)),
                        int(rng.integers(n_ids)), int(rng.integers(0, 5)), int(rng.integers(2**31))))
        elif kind == "admit":
            ops.append(("admit", int(rng.integers(n_ids)), int(rng.integers(0, max_tokens + 1))))
        elif kind == "admit_into":
            ops.append(("admit_into", int(rng.integers(n_ids)), int(rng.integers(0, max_tokens + 1)), int(rng.integers(2**31))))
        elif kind in ("release", "resume_into"):
            ops.append((kind, int(rng.integers(n_ids)), int(rng.integers(2**31))))
        else:
            k = int(rng.integers(1, batch + 1))
            ops.append((kind, [int(x) for x in rng.integers(n_ids, size=k)]))
    return ops


def snapshot(pool, ids):
    """Everything observable about the bookkeeping, in a comparable form."""
    reqs = {}
    for rid in ids:
        st, d = pool.info(rid)
        if st != orc.OK:
            reqs[rid] = st
            continue
        state = d["state"]
        # transient states settle to these
        state = {2: 3, 4: 0}.get(state, state)
        reqs[rid] = (state, d["n_tokens"], d["nb"], d["image_bytes"], d["arena_offset"],
                     None if d["blocks"] is None else d["blocks"].tolist(), pool.sharing(rid)[1].tolist())
    s = pool.stats()
    fq = pool.free_queue().tolist()
    counts = [pool.refcount(b) for b in range(s["blocks_total"])] if s["blocks_total"] <= 4096 else None
    return reqs, fq, {k: int(s[k]) for k in COMMON_STATS}, counts


def run_script(pool, ops, n_ids=12, after_each=None):
    """Run the calls; returns a log of (call, status, per-request statuses, snapshot)."""
    log = []
    for op in ops:
        kind = op[0]
        per = None
        if kind == "admit":
            st, blocks = pool.admit(op[1], op[2])
            per = None if blocks is None else blocks.tolist()
        elif kind == "admit_sharing":
            st, blocks = pool.admit_sharing(op[1], op[2], op[3], op[4])
            per = None if blocks is None else blocks.tolist()
        elif kind == "admit_sharing_into":
            n_private = max(-(-op[2] // pool.geom[4]) - op[4], 0)
            fq = pool.free_queue()
            pick = np.random.default_rng(op[5]).permutation(fq)[:n_private]
            if len(pick) < n_private:                # not enough free blocks: name an invalid list
                pick = np.concatenate([pick, np.zeros(n_private - len(pick), dtype=np.int32) - 1])
            st = pool.admit_sharing_into(op[1], op[2], op[3], op[4], pick.astype(np.int32))
        elif kind == "admit_into":
            bs = pool.geom[4]
            nb = -(-op[2] // bs)
            fq = pool.free_queue()
            pick = np.random.default_rng(op[3]).permutation(fq)[:nb]
            if len(pick) < nb:                       # not enough free blocks: name an invalid list
                pick = np.concatenate([pick, np.zeros(nb - len(pick), dtype=np.int32) - 1])
            st = pool.admit_into(op[1], op[2], pick.astype(np.int32))
        elif kind == "release":
            st = pool.release(op[1])
        elif kind == "resume_into":
            s0, d = pool.info(op[1])
            fq = pool.free_queue()
            nb = d["nb"] - len(pool.sharing(op[1])[1]) if s0 == orc.OK else 1     # the private part is what moves
            pick = np.random.default_rng(op[2]).permutation(fq)[:nb]
            if len(pick) < nb:                       # not enough free blocks: name an invalid list
                pick = np.concatenate([pick, np.zeros(nb - len(pick), dtype=np.int32) - 1])
            st = pool.resume_from_host_into(op[1], pick.astype(np.int32))
        else:
            fn = dict(retain=pool.retain_in_hbm, suspend=pool.suspend_to_host, expire=pool.expire,
                      resume=pool.resume_from_host)[kind]
            st, per = fn(op[1])
        log.append((op, st, per, snapshot(pool, range(n_ids))))
        if after_each:
            after_each(op, st)
    return log


def check_invariants(pool, ids):
    """Pool conservation, reference counts and host accounting (properties, valid for either implementation)."""
    s = pool.stats()
    fq = list(pool.free_queue())
    refs = np.zeros(s["blocks_total"], dtype=np.int64)
    host = 0
    for rid in ids:
        st, d = pool.info(rid)
        if st != orc.OK:
            continue
        state = {2: 3, 4: 0}.get(d["state"], d["state"])
        if state in (orc.ACTIVE, orc.RETAINED):
            np.add.at(refs, d["blocks"], 1)
        if state == orc.HOST:
            np.add.at(refs, pool.sharing(rid)[1], 1)                # the prefix a request on the host still refers to
            host += -(-d["image_bytes"] // 4096) * 4096
    held = int((refs > 0).sum())
    assert s["blocks_free"] + held == s["blocks_total"]             # free + distinct held = NB
    assert s["blocks_active"] + s["blocks_pinned"] == held
    assert sorted(fq) == np.flatnonzero(refs == 0).tolist()
    if s["blocks_total"] <= 4096:
        assert [pool.refcount(b) for b in range(s["blocks_total"])] == refs.tolist()
    assert s["host_used"] == host <= s["host_capacity"]
    assert s["bytes_suspended"] - s["bytes_resumed"] - s["bytes_expired_from_host"] >= 0
