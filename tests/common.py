"""Shared test helpers: a call-script generator and a runner that works on the oracle pool and on the
library pool alike (both expose the same method names), plus observation helpers."""
import numpy as np

import oracle as orc

COMMON_STATS = ["blocks_total", "blocks_free", "blocks_active", "blocks_pinned", "host_capacity", "host_used",
                "host_largest_hole", "n_active", "n_retained", "n_host", "n_expired", "suspends", "resumes",
                "resident_resumes", "expires", "recompute_marked", "host_full_rejects", "hbm_full_rejects",
                "bytes_suspended", "bytes_resumed", "bytes_expired_from_host"]


def random_script(seed, n_ops, max_tokens, n_ids=12, batch=4):
    """A seeded list of calls over a small id space; illegal calls are included on purpose."""
    rng = np.random.default_rng(seed)
    ops = []
    for _ in range(n_ops):
        kind = rng.choice(["admit", "admit", "admit_into", "retain", "suspend", "suspend", "expire", "resume", "resume",
                           "resume_into", "release"])
        if kind == "admit":
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
                     None if d["blocks"] is None else d["blocks"].tolist())
    s = pool.stats()
    return reqs, pool.free_queue().tolist(), {k: int(s[k]) for k in COMMON_STATS}


def run_script(pool, ops, n_ids=12, after_each=None):
    """Run the calls; returns a log of (call, status, per-request statuses, snapshot)."""
    log = []
    for op in ops:
        kind = op[0]
        per = None
        if kind == "admit":
            st, blocks = pool.admit(op[1], op[2])
            per = None if blocks is None else blocks.tolist()
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
            nb = d["nb"] if s0 == orc.OK else 1
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
    """Pool conservation, disjointness and host accounting (properties, valid for either implementation)."""
    s = pool.stats()
    seen = list(pool.free_queue())
    held = host = 0
    for rid in ids:
        st, d = pool.info(rid)
        if st != orc.OK:
            continue
        state = {2: 3, 4: 0}.get(d["state"], d["state"])
        if state in (orc.ACTIVE, orc.RETAINED):
            seen += list(d["blocks"])
            held += d["nb"]
        if state == orc.HOST:
            host += -(-d["image_bytes"] // 4096) * 4096
    assert s["blocks_free"] + held == s["blocks_total"]
    assert s["blocks_active"] + s["blocks_pinned"] == held
    assert sorted(seen) == list(range(s["blocks_total"]))
    assert s["host_used"] == host <= s["host_capacity"]
    assert s["bytes_suspended"] - s["bytes_resumed"] - s["bytes_expired_from_host"] >= 0
