"""CPU checks of the trace thresholds against the paper's printed values, and of the trace driver on the oracle and
the library's bookkeeping (metadata-only pool)."""
import math

import numpy as np

import oracle as orc
from common import check_invariants
from kvr_synth import context_lengths, event_trace
from paper_2608_30830_b200 import kvr
from trace_driver import TraceRunner, hbm_break_evens, host_ttl, mixture_mean


def test_thresholds_match_printed_values(golden):
    a1, b2, b3 = golden["price_vector_h100"]
    t1, tstar = hbm_break_evens(a1, b2, b3)
    assert abs(t1 - golden["t1_tstar_h100_printed"][0]) < 0.01 and round(tstar) == golden["t1_tstar_h100_printed"][1]
    t1a, tsa = hbm_break_evens(0.0232, 0.02, 2.61)
    assert abs(t1a - golden["t1_tstar_a100_printed"][0]) < 0.01 and abs(tsa - golden["t1_tstar_a100_printed"][1]) < 1
    c2, w = golden["c2_wref"]
    lam_crit = c2 / w
    assert abs(lam_crit - 0.236) < 0.001
    assert host_ttl(0.5 * lam_crit, c2, w) == math.inf and host_ttl(lam_crit, c2, w) == math.inf
    # at twice the critical load the timer is (beta3 - beta2) / beta3 of the reference wait; at 3x, half of that
    assert abs(host_ttl(2 * lam_crit, c2, w) - (b3 - b2) / b3 * w) < 1e-6
    assert abs(host_ttl(3 * lam_crit, c2, w) - 0.5 * (b3 - b2) / b3 * w) < 1e-6
    assert abs(mixture_mean() - 998.9) < 0.05


def test_trace_on_oracle_and_library_bookkeeping():
    geom = (2, 2, 4, 2, 4)
    n_req, NB = 200, 130
    lengths = context_lengths(("lognormal", 64, 0.6, 4, 512), n_req, 11)
    bpt = orc.bytes_per_token(*geom[:4])
    host_cap = 40 * 4096
    mean_img = float(np.mean(lengths)) * bpt
    c2 = host_cap / mean_img
    w_ref = mixture_mean()
    lam = 2 * c2 / w_ref
    ttl = host_ttl(lam, c2, w_ref)
    events, waits = event_trace(n_req, 11, lam, 60.0, ttl)
    order = np.random.default_rng(11).permutation(NB).astype(np.int32)
    o = orc.OrcPool(*geom, NB, host_cap, initial_free_order=order, with_data=False)
    g = kvr.Pool(*geom, NB, host_cap, initial_free_order=order, flags=kvr.METADATA_ONLY)
    ids = range(n_req)

    def after(name, args):
        check_invariants(g, ids)
        assert o.free_queue().tolist() == g.free_queue().tolist()
    counts = TraceRunner([o, g], lengths, after_call=after).run(events)
    assert counts["arrived"] >= 150
    for k in ("offloaded", "resumed_resident", "resumed_from_host", "recomputed", "ttl_expired", "demoted", "not_admitted"):
        assert counts.get(k, 0) > 0, (k, counts)
    so, sg = o.stats(), g.stats()
    for k in so:
        assert so[k] == sg[k], k
    assert sg["n_active"] == sg["n_retained"] == sg["n_host"] == 0 and sg["host_used"] == 0
