"""CPU oracle of the retention policy's arithmetic and of its measured-cost replay.  TEST INFRASTRUCTURE ONLY.

Plain fp64 Python, one statement per formula, in the paper's notation:
  Eq. 1  C_j(l) = alpha_j * l + beta_j                          (cost of l seconds in state j)
  Eq. 2  t_1 = beta_2 / alpha_1,  t* = beta_3 / alpha_1          (HBM break-evens)
  Eq. 3  lambda_crit = C_2 / W_ref
         alpha_2(lambda) = max(0, lambda - lambda_crit) * beta_3 / C_2
         t_2(lambda) = inf if lambda <= lambda_crit else (beta_3 - beta_2) / alpha_2(lambda)
Replay (Appendix D): every context is offloaded at suspension; it is admitted iff one of the C_2 host slots is
free at that moment, residents are never displaced; an admitted context leaves its slot at its resume or when its
one-shot timer fires, whichever comes first; a resume that finds its host copy pays beta_2, any other pays beta_3.
Controller (Section 3.4): replay the calibration waits under host-retain and under cpu_ttl(lambda) and keep the
cheaper branch.

Pins (tests): the cross-platform table's t_1 / t*, the load-sweep table's exact entries (0.020 at half the critical
load) and its fixed-timer columns against the closed form beta_2 P(W <= T) + beta_3 P(W > T).
"""
import math


def cost_line(alpha, beta, seconds):
    return alpha * seconds + beta


def break_evens(alpha1, beta2, beta3):
    return beta2 / alpha1, beta3 / alpha1


def lambda_crit(c2, w_ref):
    return c2 / w_ref


def alpha2(lam, c2, w_ref, beta3):
    return max(0.0, lam - lambda_crit(c2, w_ref)) * beta3 / c2


def t2(lam, c2, w_ref, beta2, beta3):
    if lam <= lambda_crit(c2, w_ref):
        return math.inf
    return (beta3 - beta2) / alpha2(lam, c2, w_ref, beta3)


def replay(arrivals, waits, c2, ttl, beta2, beta3):
    """Mean GPU opportunity cost per request and the fraction resumed from a host copy (Appendix D, replay rules).
    arrivals must be non-decreasing.  ttl may be math.inf (host-retain).

    The host tier is a plain list with one entry per occupied slot: the time at which that resident leaves.
    Readings of the two ties the paper does not spell out: a resident whose departure falls exactly on an
    arrival has left (its slot is free for that arrival), and a wait exactly equal to the timer resumes in time
    (the copy is still there: beta_2)."""
    occupied = []                   # departure times of the residents, in order of admission
    total = 0.0
    from_host = 0
    for a, w in zip(arrivals, waits):
        a, w = float(a), float(w)
        # residents leave at their resume or when their one-shot timer fires; nobody is ever displaced
        occupied = [leave for leave in occupied if leave > a]
        admitted = len(occupied) < c2               # admission iff a host slot is free at the arrival
        if admitted:
            occupied.append(a + min(w, ttl))        # the slot is held until min(wait, timer)
        if admitted and w <= ttl:
            total += beta2                          # the resume finds its host copy
            from_host += 1
        else:
            total += beta3                          # timer fired first, or never admitted: recompute
    n = len(arrivals)
    return total / n, from_host / n


def select_branch(arrivals, waits, lam, c2, w_ref, beta2, beta3):
    """('retain' | 'ttl', cost_retain, cost_ttl, t2) from a calibration sample; ties go to host-retain."""
    ttl = t2(lam, c2, w_ref, beta2, beta3)
    c_retain, _ = replay(arrivals, waits, c2, math.inf, beta2, beta3)
    c_ttl, _ = replay(arrivals, waits, c2, ttl, beta2, beta3)
    return ("ttl" if c_ttl < c_retain else "retain"), c_retain, c_ttl, ttl
