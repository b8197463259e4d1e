"""Input generators (numpy PCG64 streams keyed by (seed, stream id))."""
from dataclasses import dataclass, field

import numpy as np

DEFAULT_SEED = 20260830


@dataclass
class Workload:
    """Shape of one benchmark configuration (sizes only; no data)."""
    name: str
    layers: int
    kv_heads: int
    head_dim: int
    dtype_bytes: int
    block_size: int
    num_blocks: int
    n_requests: int
    length_rule: tuple            # ("uniform", lo, hi) | ("lognormal", median, sigma, lo, hi) | ("fixed", n)
    occupancy: float = 0.0        # fraction of the pool held by live requests before the timed part
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def geom(self):
        return (self.layers, self.kv_heads, self.head_dim, self.dtype_bytes, self.block_size)


# The five configurations of the benchmark definition, at full size.
CONFIGS = {
    "tiny": Workload("tiny", 8, 8, 128, 2, 16, 4096, 4, ("uniform", 256, 2048),
                     notes="4 requests, block ids permuted, suspend all then resume all"),
    "llama3_8b": Workload("llama3_8b", 32, 8, 128, 2, 16, 32768, 32,
                          ("lognormal", 8192, 0.6, 1024, 32768), occupancy=0.70,
                          notes="32 requests, fragmented pool at 70% occupancy"),
    "gqa64": Workload("gqa64", 64, 8, 128, 2, 16, 32768, 16, ("fixed", 16384), occupancy=0.75,
                      notes="resume burst, free list interleaved with live blocks"),
    "trace": Workload("trace", 32, 8, 128, 2, 16, 24576, 256,
                      ("lognormal", 4096, 0.6, 256, 32768),
                      notes="mixed tiering trace: retain / suspend / expire / resume events"),
    "longctx": Workload("longctx", 32, 8, 128, 2, 8, 147456, 8, ("fixed", 131072),
                        notes="8 x 128k tokens, block_size 8, ids fully shuffled"),
    # not one of the five benchmark configurations: the paper's own model as one tensor-parallel rank sees it
    # (Llama-3.1-70B, 80 layers, 8 KV heads / TP4 = 2 per GPU): 512-byte rows, 8 KiB tiles, 80 KiB per token per GPU
    "paper_70b_tp4": Workload("paper_70b_tp4", 80, 2, 128, 2, 16, 32768, 32,
                              ("lognormal", 8192, 0.6, 1024, 32768), occupancy=0.70,
                              notes="per-GPU KV shard of the paper's serving setup; small tiles"),
    # not one of the five either: the paper's workload shape on that rank -- a median gate context of 8.4K tokens of
    # which a 5.4K-token system prefix is shared by every request and ~3.0K tokens are private (Section 2)
    "paper_shape": Workload("paper_shape", 80, 2, 128, 2, 16, 32768, 32, ("fixed", 8400), occupancy=0.50,
                            notes="32 gate contexts of 8,400 tokens sharing one 5,400-token prefix",
                            extra={"shared_tokens": 5400}),
}


def _rng(seed, stream):
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def free_order(seed, num_blocks):
    """A seeded permutation of the block ids: the pool's initial free-queue order."""
    return _rng(seed, 1).permutation(num_blocks).astype(np.int32)


def context_lengths(rule, n, seed):
    """Token counts of n requests under a length rule."""
    r = _rng(seed, 2)
    kind = rule[0]
    if kind == "uniform":
        return r.integers(rule[1], rule[2] + 1, size=n).astype(np.int64)
    if kind == "lognormal":
        _, median, sigma, lo, hi = rule
        x = np.exp(np.log(median) + sigma * r.standard_normal(n))
        return np.clip(np.rint(x), lo, hi).astype(np.int64)
    if kind == "fixed":
        return np.full(n, rule[1], dtype=np.int64)
    raise ValueError(kind)


def bf16_normal_bits(seed, stream, count):
    """count draws of N(0,1) rounded to bfloat16 (round to nearest even), as uint16 bit patterns."""
    x = _rng(seed, 1000 + stream).standard_normal(count, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def fill_bytes(seed, stream, nbytes, dtype_bytes=2):
    """nbytes of KV content: bf16 N(0,1) values when dtype_bytes == 2, uniform bytes otherwise."""
    if dtype_bytes == 2 and nbytes % 2 == 0:
        return bf16_normal_bits(seed, stream, nbytes // 2).view(np.uint8)
    return _rng(seed, 1000 + stream).integers(0, 256, size=nbytes, dtype=np.uint8)


def occupancy_fillers(num_blocks, block_size, used_blocks, occupancy, seed, mean_tokens=4096):
    """Token counts of extra live requests that bring the pool to the given occupancy."""
    target = int(round(occupancy * num_blocks))
    need = target - used_blocks
    r = _rng(seed, 3)
    out = []
    while need > 0:
        n_tok = int(np.clip(np.rint(np.exp(np.log(mean_tokens) + 0.6 * r.standard_normal())), 64, 32768))
        nb = min(-(-n_tok // block_size), need)
        out.append(nb * block_size)
        need -= nb
    return np.asarray(out, dtype=np.int64)


def wait_mixture(n, seed, exp_mean_s=1800.0, logn_median_s=120.0, logn_sigma=1.0):
    """Approval waits: 50/50 mixture of exponential waits and short lognormal waits (seconds)."""
    r = _rng(seed, 4)
    pick = r.random(n) < 0.5
    w_exp = r.exponential(exp_mean_s, size=n)
    w_log = np.exp(np.log(logn_median_s) + logn_sigma * r.standard_normal(n))
    return np.where(pick, w_exp, w_log)


def event_trace(n_requests, seed, arrival_rate, t_offload, t_expire):
    """Time-ordered events of the mixed tiering trace.

    Each request arrives (Poisson arrivals at `arrival_rate`), is retained in
    HBM at its suspension, is offloaded to host `t_offload` seconds later if it
    is still waiting, is expired `t_expire` seconds after the offload if it is
    still waiting (None = never), and resumes after its wait.  The thresholds
    are inputs: the caller derives them from the paper's price vector.
    Returns a list of (time, order, kind, request) with kind in
    {"arrive", "offload", "expire", "resume"}; ties break by insertion order.
    """
    r = _rng(seed, 5)
    gaps = r.exponential(1.0 / arrival_rate, size=n_requests)
    arrive = np.cumsum(gaps)
    waits = wait_mixture(n_requests, seed)
    ev = []
    for i in range(n_requests):
        t0, w = float(arrive[i]), float(waits[i])
        ev.append((t0, len(ev), "arrive", i))
        if w > t_offload:
            ev.append((t0 + t_offload, len(ev), "offload", i))
            if t_expire is not None and w > t_offload + t_expire:
                ev.append((t0 + t_offload + t_expire, len(ev), "expire", i))
        ev.append((t0 + w, len(ev), "resume", i))
    ev.sort()
    return ev, waits


def paper_wait_family(name, n, seed, mean_s=1800.0):
    """Waits of the paper's three replay families, each with mean `mean_s`: 'lognormal' (sigma 1),
    'exponential', 'mixture' (half exponential with mean 60 s, half lognormal with sigma 0.7 and mean 3,540 s)."""
    r = _rng(seed, 6)
    if name == "lognormal":
        sigma = 1.0
        return np.exp(np.log(mean_s) - sigma * sigma / 2 + sigma * r.standard_normal(n))
    if name == "exponential":
        return r.exponential(mean_s, size=n)
    if name == "mixture":
        scale = mean_s / 1800.0
        pick = r.random(n) < 0.5
        short = r.exponential(60.0 * scale, size=n)
        sigma = 0.7
        long_ = np.exp(np.log(3540.0 * scale) - sigma * sigma / 2 + sigma * r.standard_normal(n))
        return np.where(pick, short, long_)
    raise ValueError(name)


def poisson_arrivals(n, rate, seed):
    """Arrival times of n requests of a Poisson process of the given rate."""
    return np.cumsum(_rng(seed, 7).exponential(1.0 / rate, size=n))
