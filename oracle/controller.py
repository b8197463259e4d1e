"""CPU oracle of the live retention controller.  TEST INFRASTRUCTURE ONLY.

The rules, in the paper's words restated (Section 3.4; Appendix D, live-controller paragraph):
  * a suspended context is pinned in HBM and, after a grace period (0 = at once: t_1 is about one second), moved
    to host DRAM;
  * under the cpu_ttl(lambda) branch it then carries a one-shot timer t_2(lambda); when it fires before the
    resume, the host copy is discarded and the context is never re-scored;
  * a full host tier rejects the newcomer (replay rule: residents are never displaced) or, under the live rule,
    makes room by priority: first a copy whose timer has already run out, then the copy that has been suspended
    longest (the class in between, transient blocks of active requests, cannot occur in a tier of suspended contexts);
  * a resume costs 0 from HBM plus alpha_1 per second it was pinned there, beta_2 from the host copy, beta_3
    otherwise (Eq. 1).
Everything is linear scans over a dictionary: no heaps, no sets, no shared code with the library.
"""
import math

from . import orc
from . import policy

IN_HBM, ON_HOST, GONE = 1, 2, 3
RETAIN, TTL = 0, 1
REPLAY, LIVE = 0, 1


class OrcController:
    def __init__(self, pool, prices, lam, w_ref, c2=0.0, mean_image_bytes=0.0, hbm_grace_s=0.0, branch=RETAIN,
                 admission=REPLAY):
        self.pool = pool
        self.alpha1, self.beta2, self.beta3 = prices
        self.lam, self.w_ref, self.grace, self.branch, self.admission = lam, w_ref, hbm_grace_s, branch, admission
        self.c2 = c2 if c2 > 0 else pool.stats()["host_capacity"] / mean_image_bytes
        self.t2 = policy.t2(lam, self.c2, w_ref, self.beta2, self.beta3)
        self.now = -math.inf
        self.ctx = {}                       # id -> [where, suspended_at, deadline]
        self.st = dict(suspended=0, offloaded=0, not_admitted=0, ttl_expired=0, evicted_lru=0, resumed_host=0,
                       resumed_hbm=0, recomputed=0, gpu_cost=0.0)

    def calibrate(self, arrive, wait):
        slots = max(int(math.floor(self.c2)), 1)
        choice = policy.select_branch(arrive, wait, self.lam, slots, self.w_ref, self.beta2, self.beta3)[0]
        self.branch = TTL if choice == "ttl" else RETAIN
        return self.branch

    def _offload(self, rid):
        c = self.ctx[rid]
        c[2] = math.inf
        while True:
            st, _ = self.pool.suspend_to_host([rid])
            if st == orc.OK:
                break
            assert st == orc.HOST_FULL, st
            # live rule (Appendix D): evict by priority.  First, copies whose timer has already run out at this
            # instant (due at the same time as this offload, not fired yet); the paper's second class -- transient
            # blocks of active requests -- does not exist in a host tier that holds suspended contexts only; then
            # the copy that has been suspended longest.
            expired = [(v[2], k) for k, v in self.ctx.items() if v[0] == ON_HOST and v[2] <= self.now]
            if self.admission == LIVE and expired:
                _, victim = min(expired)
                assert self.pool.expire([victim])[0] == orc.OK
                self.ctx[victim][0], self.ctx[victim][2] = GONE, math.inf
                self.st["ttl_expired"] += 1
                continue
            on_host = [(v[1], k) for k, v in self.ctx.items() if v[0] == ON_HOST]
            if self.admission == LIVE and on_host:
                _, victim = min(on_host)                      # suspended longest
                assert self.pool.expire([victim])[0] == orc.OK
                self.ctx[victim][0], self.ctx[victim][2] = GONE, math.inf
                self.st["evicted_lru"] += 1
                continue
            assert self.pool.expire([rid])[0] == orc.OK
            self.st["gpu_cost"] += self.alpha1 * (self.now - c[1])
            c[0] = GONE
            self.st["not_admitted"] += 1
            return orc.HOST_FULL
        self.st["gpu_cost"] += self.alpha1 * (self.now - c[1])
        c[0] = ON_HOST
        self.st["offloaded"] += 1
        if self.branch == TTL:
            c[2] = self.now + self.t2
        return orc.OK

    def advance(self, t):
        assert t >= self.now
        n_off = n_exp = 0
        while True:
            due = [(v[2], k) for k, v in self.ctx.items() if v[2] <= t]
            if not due:
                break
            deadline, rid = min(due)                          # earliest deadline first, ties by id
            self.now = max(self.now, deadline)
            c = self.ctx[rid]
            if c[0] == IN_HBM:
                if self._offload(rid) == orc.OK:
                    n_off += 1
            else:
                assert self.pool.expire([rid])[0] == orc.OK
                c[0], c[2] = GONE, math.inf
                self.st["ttl_expired"] += 1
                n_exp += 1
        self.now = t
        return orc.OK, n_off, n_exp

    def suspend(self, rid, now):
        self.advance(now)
        if rid in self.ctx and self.ctx[rid][0] != GONE:
            return orc.ERR_BAD_STATE
        st, _ = self.pool.retain_in_hbm([rid])
        if st != orc.OK:
            return st
        self.ctx[rid] = [IN_HBM, now, math.inf]
        self.st["suspended"] += 1
        if self.grace > 0:
            self.ctx[rid][2] = now + self.grace
            return orc.RESIDENT
        return self._offload(rid)

    def resume(self, rid, now):
        self.advance(now)
        if rid not in self.ctx:
            return orc.ERR_UNKNOWN_REQUEST
        c = self.ctx[rid]
        st, _ = self.pool.resume_from_host([rid])
        if st == orc.HBM_FULL or st < 0:
            return st
        if st == orc.RESIDENT:
            self.st["gpu_cost"] += self.alpha1 * (now - c[1])
            self.st["resumed_hbm"] += 1
        elif st == orc.OK:
            self.st["gpu_cost"] += self.beta2
            self.st["resumed_host"] += 1
        else:
            self.st["gpu_cost"] += self.beta3
            self.st["recomputed"] += 1
        del self.ctx[rid]
        return st

    def stats(self):
        d = dict(self.st)
        d.update(tracked=len(self.ctx), t2=self.t2, branch=self.branch)
        return d
