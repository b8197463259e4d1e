"""The live controller: the oracle is pinned to the replay of the policy oracle (equal-sized contexts, replay
admission) and to hand-worked eviction orders; the library's controller (on a metadata-only pool) must then take the
same decisions, leave the same bookkeeping and charge the same cost as the oracle's on seeded traces."""
import math

import numpy as np
import pytest

import oracle as orc
from common import snapshot
from kvr_synth import paper_wait_family, poisson_arrivals
from oracle import policy
from oracle.controller import LIVE, REPLAY, RETAIN, TTL, OrcController
from paper_2608_30830_b200 import kvr

GEOM = (2, 2, 4, 2, 4)            # 64 bytes per token
PRICES = (0.0176, 0.02, 1.91)


def run_trace(ctl, pool, arrive, wait, lengths, on_event=None, on_admit=None):
    """Suspend at arrive[i], resume at arrive[i] + wait[i]; admits before the suspension, releases after the resume.
    A resume that must recompute re-admits (the prefill).  Returns the list of (event, request, status)."""
    ev = sorted([(float(a), 0, i) for i, a in enumerate(arrive)] + [(float(a + w), 1, i) for i, (a, w) in enumerate(zip(arrive, wait))])
    log = []
    for t, kind, i in ev:
        if kind == 0:
            st, blocks = pool.admit(i, int(lengths[i]))
            assert st == orc.OK, st
            if on_admit:
                on_admit(i, blocks)
            s = ctl.suspend(i, t)
        else:
            s = ctl.resume(i, t)
            if s == orc.RECOMPUTE:
                assert pool.admit(i, int(lengths[i]))[0] == orc.OK
            assert pool.release(i) == orc.OK
        log.append((kind, i, s))
        if on_event:
            on_event(t, kind, i, s)
    return log


@pytest.mark.parametrize("family,mult,branch", [("lognormal", 2, RETAIN), ("exponential", 3, RETAIN),
                                                 ("mixture", 3, TTL), ("mixture", 0.5, TTL), ("lognormal", 2, TTL)])
def test_oracle_controller_reproduces_the_replay(family, mult, branch):
    # equal-sized contexts: the byte-capacity tier is exactly C2 slots, so the controller must charge what the
    # slot replay charges (offload at suspension, replay admission, HBM never full)
    c2, w_ref, n = 40, 1800.0, 1200
    lam = mult * c2 / w_ref
    arrive, wait = poisson_arrivals(n, lam, 3), paper_wait_family(family, n, 3)
    tokens = 60                                                     # 3840 B -> one 4096-byte granule
    pool = orc.OrcPool(*GEOM, 16 * n, c2 * 4096, with_data=False)
    ctl = OrcController(pool, PRICES, lam, w_ref, c2=c2, branch=branch, admission=REPLAY)
    run_trace(ctl, pool, arrive, wait, [tokens] * n)
    ttl = policy.t2(lam, c2, w_ref, PRICES[1], PRICES[2]) if branch == TTL else math.inf
    want_cost, want_frac = policy.replay(arrive, wait, c2, ttl, PRICES[1], PRICES[2])
    s = ctl.stats()
    assert s["gpu_cost"] / n == pytest.approx(want_cost, rel=1e-9)
    assert s["resumed_host"] / n == pytest.approx(want_frac) and s["tracked"] == 0
    assert s["resumed_host"] + s["recomputed"] == n and s["resumed_hbm"] == 0


def test_live_admission_evicts_the_longest_suspended_by_hand():
    pool = orc.OrcPool(*GEOM, 64, 2 * 4096, with_data=False)       # two one-granule slots
    ctl = OrcController(pool, PRICES, 0.0, 1800.0, c2=2, branch=RETAIN, admission=LIVE)
    for rid in (1, 2, 3):
        pool.admit(rid, 60)
    assert ctl.suspend(1, 10.0) == orc.OK and ctl.suspend(2, 20.0) == orc.OK
    assert ctl.suspend(3, 30.0) == orc.OK                           # tier full: request 1 (oldest) is discarded
    assert pool.info(1)[1]["state"] == orc.EXPIRED and pool.info(2)[1]["state"] == orc.HOST
    assert ctl.resume(1, 40.0) == orc.RECOMPUTE and ctl.resume(2, 41.0) == orc.OK and ctl.resume(3, 42.0) == orc.OK
    s = ctl.stats()
    assert s["evicted_lru"] == 1 and s["gpu_cost"] == pytest.approx(1.91 + 0.02 + 0.02)


def test_live_admission_discards_an_expired_timer_before_any_lru_victim_by_hand():
    """Appendix D, live rule: "blocks whose timer has expired" are evicted before least-recently-used suspended
    blocks.  Worked by hand with exact numbers: prices (0.5, 1, 3), C2 = 3, W_ref = 96, lambda = 5/32 give
    alpha_2 = 1/8 and t_2 = 16 s; grace 10 s.  X and W go to the host under host-retain (no timers); after the
    branch is frozen to cpu_ttl, Y is offloaded at 24 (timer due at 40) and Z's offload falls due at 40 as well.
    The tier is full at that instant: Y's timer has run out, so Y goes -- not X, which has been suspended longest."""
    prices, c2, w_ref, lam = (0.5, 1.0, 3.0), 3, 96.0, 5.0 / 32.0
    cal_arrive = [0, 1, 2, 30, 31, 32, 40, 41, 42]
    cal_wait = [1000.0] * 3 + [1.0] * 6              # host-retain: 3 b2 + 6 b3 = 21; cpu_ttl: 3 b3 + 6 b2 = 15 -> cpu_ttl
    po = orc.OrcPool(*GEOM, 64, 3 * 4096, with_data=False)
    pg = kvr.Pool(*GEOM, 64, 3 * 4096, flags=kvr.METADATA_ONLY)
    co = OrcController(po, prices, lam, w_ref, c2=c2, hbm_grace_s=10.0, branch=RETAIN, admission=LIVE)
    cg = kvr.Controller(pg, prices, lam, w_ref, c2=c2, hbm_grace_s=10.0, branch=kvr.BRANCH_RETAIN, admission=kvr.ADMIT_LIVE)
    X, W, Y, Z = 9, 7, 8, 1
    for pool, ctl in ((po, co), (pg, cg)):
        assert ctl.stats()["t2"] == 16.0
        for rid in (X, W, Y, Z):
            assert pool.admit(rid, 60)[0] == orc.OK
        assert ctl.suspend(X, 0.0) == orc.RESIDENT and ctl.suspend(W, 1.0) == orc.RESIDENT
        assert ctl.advance(12.0) == (orc.OK, 2, 0)                      # both on the host, no timers
        assert ctl.calibrate(cal_arrive, cal_wait) == TTL
        assert ctl.suspend(Y, 14.0) == orc.RESIDENT
        assert ctl.advance(25.0) == (orc.OK, 1, 0)                      # Y on the host since 24, timer due at 40
        assert ctl.suspend(Z, 30.0) == orc.RESIDENT                     # offload due at 40 too
        st, n_off, n_exp = ctl.advance(41.0)
        assert (st, n_off) == (orc.OK, 1)
        states = {rid: pool.info(rid)[1]["state"] for rid in (X, W, Y, Z)}
        assert states == {X: orc.HOST, W: orc.HOST, Y: orc.EXPIRED, Z: orc.HOST}
        s = ctl.stats()
        assert s["ttl_expired"] == 1 and s["evicted_lru"] == 0 and s["not_admitted"] == 0
        assert ctl.resume(Y, 42.0) == orc.RECOMPUTE and ctl.resume(X, 43.0) == orc.OK
        # HBM time: X 10 s, W 10 s, Y 10 s, Z 10 s at alpha_1 = 0.5; one recompute, one host resume
        assert ctl.stats()["gpu_cost"] == pytest.approx(0.5 * 40 + 3.0 + 1.0)
    assert snapshot(po, [X, W, Y, Z]) == snapshot(pg, [X, W, Y, Z])


def test_grace_period_timer_and_hbm_cost_by_hand():
    pool = orc.OrcPool(*GEOM, 64, 8 * 4096, with_data=False)
    lam = 2 * 4 / 100.0                                             # c2 = 4, w_ref = 100 -> t2 = (1.91-0.02)/1.91*100
    ctl = OrcController(pool, PRICES, lam, 100.0, c2=4, hbm_grace_s=5.0, branch=TTL, admission=REPLAY)
    t2 = (1.91 - 0.02) / 1.91 * 100.0
    assert ctl.t2 == pytest.approx(t2)
    for rid in (1, 2, 3):
        pool.admit(rid, 60)
    assert ctl.suspend(1, 0.0) == orc.RESIDENT and ctl.suspend(2, 1.0) == orc.RESIDENT and ctl.suspend(3, 2.0) == orc.RESIDENT
    assert ctl.resume(1, 3.0) == orc.RESIDENT                       # back within the grace period: 3 s of HBM
    assert ctl.advance(6.5) == (orc.OK, 1, 0)                       # request 2 offloaded at t = 6 (5 s of HBM)
    assert pool.info(2)[1]["state"] == orc.HOST and pool.info(3)[1]["state"] == orc.RETAINED
    assert ctl.resume(3, 50.0) == orc.OK                            # offloaded at 7 on the way, timer not yet due
    assert ctl.resume(2, 6.0 + t2 + 1.0) == orc.RECOMPUTE           # its timer fired at 6 + t2
    s = ctl.stats()
    assert s["ttl_expired"] == 1 and s["offloaded"] == 2
    assert s["gpu_cost"] == pytest.approx(0.0176 * (3 + 5 + 5) + 0.02 + 1.91)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("admission,branch,grace", [(REPLAY, TTL, 0.0), (LIVE, TTL, 30.0), (LIVE, RETAIN, 0.0), (REPLAY, RETAIN, 45.0)])
def test_library_controller_matches_the_oracle(seed, admission, branch, grace):
    n, NB, host_cap = 300, 4000, 24 * 4096
    rng = np.random.default_rng(seed)
    lengths = rng.integers(1, 200, size=n)                          # 1..4 granules per image
    mean_img = float(np.mean(lengths)) * 64
    w_ref = 1800.0
    lam = 2.5 * (host_cap / mean_img) / w_ref
    arrive = poisson_arrivals(n, lam, seed)
    wait = paper_wait_family("mixture", n, seed)
    order = rng.permutation(NB).astype(np.int32)
    po = orc.OrcPool(*GEOM, NB, host_cap, initial_free_order=order, with_data=False)
    pg = kvr.Pool(*GEOM, NB, host_cap, initial_free_order=order, flags=kvr.METADATA_ONLY)
    co = OrcController(po, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=grace, branch=branch, admission=admission)
    cg = kvr.Controller(pg, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=grace, branch=branch, admission=admission)
    lo = run_trace(co, po, arrive, wait, lengths)
    lg = run_trace(cg, pg, arrive, wait, lengths)
    assert lo == lg
    so, sg = co.stats(), cg.stats()
    for k in so:
        assert sg[k] == pytest.approx(so[k], rel=1e-12), k
    assert snapshot(po, range(n)) == snapshot(pg, range(n))
    assert so["offloaded"] > 50 and so["recomputed"] > 10
    if admission == LIVE:
        assert so["evicted_lru"] > 0 and so["not_admitted"] == 0
    else:
        assert so["not_admitted"] > 0
    if branch == TTL:
        assert so["ttl_expired"] > 0


def test_calibration_freezes_the_cheaper_branch():
    c2, w_ref = 40, 1800.0
    lam = 3 * c2 / w_ref
    for family, want in (("lognormal", RETAIN), ("mixture", TTL)):
        arrive, wait = poisson_arrivals(4000, lam, 9), paper_wait_family(family, 4000, 9)
        po = orc.OrcPool(*GEOM, 64, c2 * 4096, with_data=False)
        pg = kvr.Pool(*GEOM, 64, c2 * 4096, flags=kvr.METADATA_ONLY)
        co = OrcController(po, PRICES, lam, w_ref, c2=c2)
        cg = kvr.Controller(pg, PRICES, lam, w_ref, c2=c2)
        assert co.calibrate(arrive, wait) == cg.calibrate(arrive, wait) == want
        assert cg.stats()["branch"] == want


def test_controller_rejects_bad_configs_and_time_travel():
    pg = kvr.Pool(*GEOM, 64, 1 << 16, flags=kvr.METADATA_ONLY)
    with pytest.raises(kvr.KvrError):
        kvr.Controller(pg, (0.0, 0.02, 1.91), 0.1, 1800.0, c2=4)
    with pytest.raises(kvr.KvrError):
        kvr.Controller(pg, PRICES, 0.1, 1800.0)                        # neither c2 nor a mean image size
    c = kvr.Controller(pg, PRICES, 0.1, 1800.0, c2=4)
    pg.admit(1, 10)
    assert c.suspend(1, 100.0) == kvr.OK
    assert c.advance(50.0)[0] == kvr.ERR_INVALID_ARG                   # the clock never runs backwards
    assert c.suspend(1, 101.0) == kvr.ERR_BAD_STATE and c.resume(7, 102.0) == kvr.ERR_UNKNOWN_REQUEST


class SharingPool:
    """A pool whose plain admissions share the first `ns` blocks of a long-lived donor request: the paper's workload
    shape (one system prefix, private suffixes) driven through code that only knows `admit`."""

    def __init__(self, pool, donor, ns, bs):
        self._pool, self._donor, self._ns, self._bs = pool, donor, ns, bs

    def admit(self, rid, n_private):
        return self._pool.admit_sharing(rid, self._ns * self._bs + n_private, self._donor, self._ns)

    def __getattr__(self, name):
        return getattr(self._pool, name)


def test_library_controller_matches_the_oracle_over_a_shared_prefix():
    """Every context shares one system prefix (Section 2): the tier holds private suffixes only, the prefix stays
    resident while any context refers to it, and the library's controller decides exactly as the oracle's."""
    n, NB, host_cap, ns, PREFIX = 160, 700, 32 * 4096, 9, 10_000
    rng = np.random.default_rng(41)
    lengths = rng.integers(1, 100, size=n)
    mean_img = float(np.mean(lengths)) * 64
    w_ref = 1800.0
    lam = 2.5 * (host_cap / mean_img) / w_ref
    arrive, wait = poisson_arrivals(n, lam, 41), paper_wait_family("mixture", n, 41)
    order = rng.permutation(NB).astype(np.int32)
    po = orc.OrcPool(*GEOM, NB, host_cap, initial_free_order=order, with_data=False)
    pg = kvr.Pool(*GEOM, NB, host_cap, initial_free_order=order, flags=kvr.METADATA_ONLY)
    for pool in (po, pg):
        assert pool.admit(PREFIX, ns * 4)[0] == orc.OK
    co = OrcController(po, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=20.0, branch=TTL, admission=LIVE)
    cg = kvr.Controller(pg, PRICES, lam, w_ref, mean_image_bytes=mean_img, hbm_grace_s=20.0, branch=TTL, admission=LIVE)
    lo = run_trace(co, SharingPool(po, PREFIX, ns, 4), arrive, wait, lengths)
    lg = run_trace(cg, SharingPool(pg, PREFIX, ns, 4), arrive, wait, lengths)
    assert lo == lg
    so, sg = co.stats(), cg.stats()
    for k in so:
        assert sg[k] == pytest.approx(so[k], rel=1e-12), k
    ids = list(range(n)) + [PREFIX]
    assert snapshot(po, ids) == snapshot(pg, ids)
    assert so["resumed_host"] > 10 and so["offloaded"] > 50
    assert po.stats()["bytes_suspended"] == pg.stats()["bytes_suspended"] < so["offloaded"] * 100 * 64     # suffixes only
    assert pg.refcount(int(pg.info(PREFIX)[1]["blocks"][0])) == 1            # every sharer has let go again
