"""Driver for the mixed tiering trace (the benchmark's fourth configuration).

The thresholds come from the paper's price vector: t_1 = beta_2 / alpha_1 and t* = beta_3 / alpha_1 (Eq. 2),
lambda_crit = C_2 / W_ref, alpha_2(lambda) = max(0, lambda - lambda_crit) * beta_3 / C_2 and
t_2(lambda) = (beta_3 - beta_2) / alpha_2(lambda), infinite at or below lambda_crit (Eq. 3).  The driver is test
code: it turns those thresholds and the seeded event list into library calls, applies every call to each pool it is
given, and demands identical outcomes."""
import math

ALPHA1, BETA2, BETA3 = 0.0176, 0.02, 1.91


def hbm_break_evens(alpha1=ALPHA1, beta2=BETA2, beta3=BETA3):
    return beta2 / alpha1, beta3 / alpha1                       # Eq. 2: t_1, t*


def host_ttl(lam, c2, w_ref, beta2=BETA2, beta3=BETA3):
    lam_crit = c2 / w_ref
    alpha2 = max(0.0, lam - lam_crit) * beta3 / c2              # Eq. 3
    return math.inf if lam <= lam_crit else (beta3 - beta2) / alpha2


def mixture_mean(exp_mean=1800.0, logn_median=120.0, sigma=1.0):
    """Mean of the 50/50 wait mixture: exponential mean, lognormal mean = median * exp(sigma^2 / 2)."""
    return 0.5 * exp_mean + 0.5 * logn_median * math.exp(sigma * sigma / 2)


class TraceRunner:
    """Applies the event list to every pool in `pools` (same call on each) and compares outcomes.

    fill(rid, blocks, n_tokens) is called after every admission; verify(rid, blocks, n_tokens) before a resumed or
    resident request is released.  OK/RESIDENT/RECOMPUTE/HOST_FULL/HBM_FULL are handled the way the paper's replay
    does: not admitted -> recompute at resume; HBM full -> the oldest retained request is demoted to host."""

    OK, RESIDENT, RECOMPUTE, HOST_FULL, HBM_FULL = 0, 1, 2, 3, 4

    def __init__(self, pools, lengths, fill=None, verify=None, after_call=None):
        self.pools, self.lengths = pools, lengths
        self.fill, self.verify, self.after_call = fill, verify, after_call
        self.retained = []            # arrival order of requests currently RETAINED
        self.alive = set()
        self.counts = {}

    def call(self, name, *args):
        outs = [getattr(p, name)(*args) for p in self.pools]
        first = outs[0]
        for o in outs[1:]:
            if name == "admit":
                assert o[0] == first[0] and (o[1] is None or o[1].tolist() == first[1].tolist()), (name, args)
            else:
                assert o == first, (name, args, o, first)
        if self.after_call:
            self.after_call(name, args)
        return first

    def bump(self, key):
        self.counts[key] = self.counts.get(key, 0) + 1

    def make_room(self):
        """HBM full: demote the oldest retained request to host (expire it if the host is full too)."""
        if not self.retained:
            return False
        victim = self.retained.pop(0)
        st, _ = self.call("suspend_to_host", [victim])
        if st == self.HOST_FULL:
            self.call("expire", [victim])
            self.bump("demote_expired")
        else:
            assert st == self.OK
            self.bump("demoted")
        return True

    def admit(self, rid):
        n = int(self.lengths[rid])
        while True:
            st, blocks = self.call("admit", rid, n)
            if st == self.OK:
                if self.fill:
                    self.fill(rid, blocks, n)
                return True
            assert st == self.HBM_FULL
            if not self.make_room():
                return False

    def run(self, events):
        for _, _, kind, rid in events:
            if kind == "arrive":
                if not self.admit(rid):
                    self.bump("dropped")
                    continue
                self.alive.add(rid)
                assert self.call("retain_in_hbm", [rid])[0] == self.OK          # suspension: stay in HBM first
                self.retained.append(rid)
                self.bump("arrived")
            elif rid not in self.alive:
                continue
            elif kind == "offload":
                if rid in self.retained:                                        # still waiting in HBM: move to host
                    self.retained.remove(rid)
                    st, _ = self.call("suspend_to_host", [rid])
                    if st == self.HOST_FULL:                                    # not admitted: recompute at resume
                        assert self.call("expire", [rid])[0] == self.OK
                        self.bump("not_admitted")
                    else:
                        assert st == self.OK
                        self.bump("offloaded")
            elif kind == "expire":
                st, _ = self.call("expire", [rid])                              # one-shot timer
                self.bump("ttl_expired" if st == self.OK else "ttl_noop")
            elif kind == "resume":
                while True:
                    st, _ = self.call("resume_from_host", [rid])
                    if st != self.HBM_FULL:
                        break
                    assert self.make_room(), "HBM full with nothing to demote"
                if st == self.RESIDENT:
                    self.retained.remove(rid)
                    self.bump("resumed_resident")
                elif st == self.OK:
                    self.bump("resumed_from_host")
                else:
                    assert st == self.RECOMPUTE
                    self.bump("recomputed")
                    if not self.admit(rid):                                     # re-prefill by the caller
                        self.call("release", rid)
                        self.alive.discard(rid)
                        continue
                if self.verify:
                    self.verify(rid)
                assert self.call("release", rid) == self.OK
                self.alive.discard(rid)
        return self.counts
