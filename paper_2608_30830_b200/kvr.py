"""ctypes binding of libkvr.so: same names as the C ABI (include/kvr.h), argument marshalling only."""
import ctypes as C
import os

import numpy as np

from . import build as _build

OK, RESIDENT, RECOMPUTE, HOST_FULL, HBM_FULL = 0, 1, 2, 3, 4
ERR_INVALID_ARG, ERR_UNKNOWN_REQUEST, ERR_BAD_STATE, ERR_GEOMETRY = -1, -2, -3, -4
ERR_CUDA, ERR_TIMEOUT, ERR_NOMEM = -5, -6, -7
ACTIVE, RETAINED, SUSPENDING, HOST, RESUMING, EXPIRED = 0, 1, 2, 3, 4, 5
SYNC = 1
LOW_LATENCY = 2
METADATA_ONLY, PROFILE = 1, 2
ROUTE_AUTO, ROUTE_STAGED, ROUTE_MAPPED, ROUTE_DMA2D = 0, 1, 2, 3
FAIL_CUDA, FAIL_ALLOC = 0, 1
LAYER_MAJOR, BLOCK_MAJOR = 0, 1
KERNEL_WARP, KERNEL_BULK = 1, 2
ALL = 2**64 - 1


class KvrError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__("kvr status %d: %s" % (status, msg))
        self.status = status


class Geometry(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("layers", "kv_heads", "head_dim", "dtype_bytes", "block_size")]


class Config(C.Structure):
    _fields_ = [("g", Geometry), ("num_blocks", C.c_int32), ("device", C.c_int32),
                ("host_capacity_bytes", C.c_uint64), ("chunk_bytes", C.c_uint64),
                ("staging_slots", C.c_int32), ("route", C.c_int32), ("kernel", C.c_int32),
                ("max_ctas", C.c_int32), ("flags", C.c_uint32), ("layout", C.c_int32),
                ("device_pool", C.c_void_p), ("host_arena", C.c_void_p),
                ("initial_free_order", C.POINTER(C.c_int32)),
                ("device_staging", C.c_void_p), ("streams", C.c_void_p * 4),
                ("suspend_single_bytes", C.c_uint64), ("resume_single_bytes", C.c_uint64), ("copy_piece_bytes", C.c_uint64),
                ("max_moves_in_flight", C.c_int32), ("bulk_warps", C.c_int32), ("bulk_stages", C.c_int32),
                ("bulk_piece_bytes", C.c_int32)]


class Prices(C.Structure):
    _fields_ = [("alpha1", C.c_double), ("beta2", C.c_double), ("beta3", C.c_double)]


class ControllerConfig(C.Structure):
    _fields_ = [("prices", Prices), ("lambda_", C.c_double), ("c2", C.c_double), ("mean_image_bytes", C.c_double),
                ("w_ref", C.c_double), ("hbm_grace_s", C.c_double), ("branch", C.c_int32), ("admission", C.c_int32)]


class ControllerStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("suspended", "offloaded", "not_admitted", "ttl_expired", "evicted_lru",
                                         "resumed_host", "resumed_hbm", "recomputed", "tracked")] + \
               [("gpu_cost", C.c_double), ("t2", C.c_double), ("branch", C.c_int32), ("reserved", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("blocks_total", "blocks_free", "blocks_active", "blocks_pinned")] + \
               [(n, C.c_uint64) for n in ("host_capacity", "host_used", "host_largest_hole")] + \
               [(n, C.c_int64) for n in ("n_active", "n_retained", "n_host", "n_expired",
                                         "suspends", "resumes", "resident_resumes", "expires",
                                         "recompute_marked", "host_full_rejects", "hbm_full_rejects")] + \
               [(n, C.c_uint64) for n in ("bytes_suspended", "bytes_resumed", "bytes_expired_from_host")] + \
               [(n, C.c_int64) for n in ("ops_in_flight", "gather_launches", "scatter_launches",
                                         "d2h_copies", "h2d_copies")] + \
               [(n, C.c_uint64) for n in ("gather_bytes", "scatter_bytes", "d2h_bytes", "h2d_bytes", "desc_bytes")] + \
               [(n, C.c_double) for n in ("gather_ms", "scatter_ms", "gather_kernel_ms", "scatter_kernel_ms")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


EXPORTS = [
    "kvr_bytes_per_token", "kvr_pool_create", "kvr_pool_destroy", "kvr_request_admit", "kvr_request_admit_into", "kvr_request_release",
    "kvr_request_admit_sharing", "kvr_request_admit_sharing_into", "kvr_request_sharing", "kvr_block_refcount", "kvr_test_fail_nth", "kvr_test_points", "kvr_test_plan",
    "kvr_pool_numa_node", "kvr_numa_lookup",
    "kvr_retain_in_hbm", "kvr_suspend_to_host", "kvr_expire", "kvr_resume_from_host",
    "kvr_resume_from_host_into", "kvr_export_to_device", "kvr_import_from_device", "kvr_request_info",
    "kvr_request_latency", "kvr_wait", "kvr_pool_stats", "kvr_free_queue", "kvr_pool_device_ptr",
    "kvr_pool_host_arena", "kvr_last_error", "kvr_gather_noalloc", "kvr_read_load", "kvr_probe_link", "kvr_selftest_bounded_wait", "kvr_selftest_block_check", "kvr_clear_device_error",
    "kvr_policy_break_evens", "kvr_policy_host_ttl", "kvr_policy_replay", "kvr_policy_select",
    "kvr_controller_create", "kvr_controller_destroy", "kvr_controller_calibrate", "kvr_controller_suspend",
    "kvr_controller_advance", "kvr_controller_resume", "kvr_controller_get_stats",
]

_lib = None


def lib():
    """Load libkvr.so (building it with nvcc if the sources are newer).  Raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    try:
        path = _build.build()
    except Exception as e:  # no silent fallback: the CUDA library is the product
        if not os.path.exists(_build.SO):
            raise ImportError("libkvr.so is missing and could not be built: %r" % (e,))
        path = _build.SO
    L = C.CDLL(path)
    i32, i64, u32, u64, vp = C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_void_p
    pi32, pu64 = C.POINTER(C.c_int32), C.POINTER(C.c_uint64)
    L.kvr_bytes_per_token.restype = u64
    L.kvr_bytes_per_token.argtypes = [C.POINTER(Geometry)]
    L.kvr_pool_create.restype = i32
    L.kvr_pool_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    L.kvr_pool_destroy.restype = i32
    L.kvr_pool_destroy.argtypes = [vp]
    L.kvr_request_admit.restype = i32
    L.kvr_request_admit.argtypes = [vp, u64, i64, pi32, i32]
    L.kvr_request_admit_into.restype = i32
    L.kvr_request_admit_into.argtypes = [vp, u64, i64, pi32, i32]
    L.kvr_request_release.restype = i32
    L.kvr_request_release.argtypes = [vp, u64]
    L.kvr_request_admit_sharing.restype = i32
    L.kvr_request_admit_sharing.argtypes = [vp, u64, i64, u64, i32, pi32, i32]
    L.kvr_request_admit_sharing_into.restype = i32
    L.kvr_request_admit_sharing_into.argtypes = [vp, u64, i64, u64, i32, pi32, i32]
    L.kvr_request_sharing.restype = i32
    L.kvr_request_sharing.argtypes = [vp, u64, pi32, pi32, i32]
    L.kvr_block_refcount.restype = i32
    L.kvr_block_refcount.argtypes = [vp, i32]
    L.kvr_test_fail_nth.restype = i32
    L.kvr_test_fail_nth.argtypes = [vp, i32, i64]
    L.kvr_test_points.restype = i64
    L.kvr_test_points.argtypes = [vp, i32]
    L.kvr_test_plan.restype = i32
    L.kvr_test_plan.argtypes = [C.POINTER(Geometry), C.POINTER(i64), i32, u64, i32, i32, i32, i32, u32, u64, u64,
                                C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), i64, C.POINTER(i64)]
    L.kvr_pool_numa_node.restype = i32
    L.kvr_pool_numa_node.argtypes = [vp]
    L.kvr_numa_lookup.restype = i32
    L.kvr_numa_lookup.argtypes = [C.c_char_p, C.c_char_p, pi32, pi32, i32]
    for name in ("kvr_retain_in_hbm", "kvr_expire"):
        f = getattr(L, name)
        f.restype = i32
        f.argtypes = [vp, pu64, i32, pi32]
    for name in ("kvr_suspend_to_host", "kvr_resume_from_host"):
        f = getattr(L, name)
        f.restype = i32
        f.argtypes = [vp, pu64, i32, u32, pi32]
    L.kvr_resume_from_host_into.restype = i32
    L.kvr_resume_from_host_into.argtypes = [vp, u64, pi32, i32, u32]
    for name in ("kvr_export_to_device", "kvr_import_from_device"):
        f = getattr(L, name)
        f.restype = i32
        f.argtypes = [vp, pu64, i32, vp, u64, pu64, u32]
    L.kvr_request_info.restype = i32
    L.kvr_request_info.argtypes = [vp, u64, pi32, C.POINTER(i64), pi32, pi32, i32, C.POINTER(vp), pu64, pu64]
    L.kvr_request_latency.restype = i32
    L.kvr_request_latency.argtypes = [vp, u64, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.kvr_wait.restype = i32
    L.kvr_wait.argtypes = [vp, u64, i64]
    L.kvr_pool_stats.restype = i32
    L.kvr_pool_stats.argtypes = [vp, C.POINTER(Stats)]
    L.kvr_free_queue.restype = i64
    L.kvr_free_queue.argtypes = [vp, pi32, i64]
    L.kvr_pool_device_ptr.restype = vp
    L.kvr_pool_device_ptr.argtypes = [vp]
    L.kvr_pool_host_arena.restype = vp
    L.kvr_pool_host_arena.argtypes = [vp]
    L.kvr_last_error.restype = C.c_char_p
    L.kvr_last_error.argtypes = []
    pd = C.POINTER(C.c_double)
    L.kvr_policy_break_evens.restype = i32
    L.kvr_policy_break_evens.argtypes = [C.POINTER(Prices), pd, pd]
    L.kvr_policy_host_ttl.restype = i32
    L.kvr_policy_host_ttl.argtypes = [C.POINTER(Prices), C.c_double, C.c_double, C.c_double, pd, pd]
    L.kvr_policy_replay.restype = i32
    L.kvr_policy_replay.argtypes = [C.POINTER(Prices), pd, pd, i64, i64, C.c_double, pd, pd]
    L.kvr_policy_select.restype = i32
    L.kvr_policy_select.argtypes = [C.POINTER(Prices), pd, pd, i64, C.c_double, i64, C.c_double, pi32, pd, pd, pd]
    L.kvr_controller_create.restype = i32
    L.kvr_controller_create.argtypes = [vp, C.POINTER(ControllerConfig), C.POINTER(vp)]
    L.kvr_controller_destroy.restype = i32
    L.kvr_controller_destroy.argtypes = [vp]
    L.kvr_controller_calibrate.restype = i32
    L.kvr_controller_calibrate.argtypes = [vp, pd, pd, i64, pi32]
    L.kvr_controller_suspend.restype = i32
    L.kvr_controller_suspend.argtypes = [vp, u64, C.c_double]
    L.kvr_controller_advance.restype = i32
    L.kvr_controller_advance.argtypes = [vp, C.c_double, pi32, pi32]
    L.kvr_controller_resume.restype = i32
    L.kvr_controller_resume.argtypes = [vp, u64, C.c_double]
    L.kvr_controller_get_stats.restype = i32
    L.kvr_controller_get_stats.argtypes = [vp, C.POINTER(ControllerStats)]
    L.kvr_selftest_bounded_wait.restype = i32
    L.kvr_selftest_bounded_wait.argtypes = [vp, i32]
    L.kvr_selftest_block_check.restype = i32
    L.kvr_selftest_block_check.argtypes = [vp, i32]
    L.kvr_clear_device_error.restype = i32
    L.kvr_clear_device_error.argtypes = [vp]
    L.kvr_probe_link.restype = i32
    L.kvr_probe_link.argtypes = [vp, u64, i32, pd, pd]
    L.kvr_read_load.restype = i32
    L.kvr_read_load.argtypes = [vp, u64, i32, vp, vp]
    L.kvr_gather_noalloc.restype = i32
    L.kvr_gather_noalloc.argtypes = [vp, C.POINTER(Geometry), i32, pi32, i32, i64, vp, vp]
    _lib = L
    return L


def last_error():
    return lib().kvr_last_error().decode()


def bytes_per_token(layers, kv_heads, head_dim, dtype_bytes, block_size=16):
    g = Geometry(layers, kv_heads, head_dim, dtype_bytes, block_size)
    return int(lib().kvr_bytes_per_token(C.byref(g)))


def _check(st):
    if st != OK:
        raise KvrError(st, last_error())


def policy_break_evens(alpha1, beta2, beta3):
    p, t1, ts = Prices(alpha1, beta2, beta3), C.c_double(), C.c_double()
    _check(lib().kvr_policy_break_evens(C.byref(p), C.byref(t1), C.byref(ts)))
    return t1.value, ts.value


def policy_host_ttl(prices, lam, c2, w_ref):
    p, a2, t2 = Prices(*prices), C.c_double(), C.c_double()
    _check(lib().kvr_policy_host_ttl(C.byref(p), lam, c2, w_ref, C.byref(a2), C.byref(t2)))
    return a2.value, t2.value


def _f64p(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def policy_replay(prices, arrive, wait, c2, ttl):
    p, cost, frac = Prices(*prices), C.c_double(), C.c_double()
    arrive, wait = np.ascontiguousarray(arrive, dtype=np.float64), np.ascontiguousarray(wait, dtype=np.float64)
    _check(lib().kvr_policy_replay(C.byref(p), _f64p(arrive), _f64p(wait), len(arrive), c2, ttl, C.byref(cost), C.byref(frac)))
    return cost.value, frac.value


def policy_select(prices, arrive, wait, lam, c2, w_ref):
    p = Prices(*prices)
    use, cr, ct, t2 = C.c_int32(), C.c_double(), C.c_double(), C.c_double()
    arrive, wait = np.ascontiguousarray(arrive, dtype=np.float64), np.ascontiguousarray(wait, dtype=np.float64)
    _check(lib().kvr_policy_select(C.byref(p), _f64p(arrive), _f64p(wait), len(arrive), lam, c2, w_ref,
                                   C.byref(use), C.byref(cr), C.byref(ct), C.byref(t2)))
    return ("ttl" if use.value else "retain"), cr.value, ct.value, t2.value


BRANCH_RETAIN, BRANCH_TTL = 0, 1
ADMIT_REPLAY, ADMIT_LIVE = 0, 1


class Controller:
    """kvr_controller handle over a Pool (which must outlive it)."""

    def __init__(self, pool, prices, lam, w_ref, c2=0.0, mean_image_bytes=0.0, hbm_grace_s=0.0,
                 branch=BRANCH_RETAIN, admission=ADMIT_REPLAY):
        cfg = ControllerConfig(Prices(*prices), lam, c2, mean_image_bytes, w_ref, hbm_grace_s, branch, admission)
        h = C.c_void_p()
        _check(lib().kvr_controller_create(pool._h, C.byref(cfg), C.byref(h)))
        self._h, self.pool = h, pool

    def close(self):
        if getattr(self, "_h", None):
            lib().kvr_controller_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def calibrate(self, arrive, wait):
        arrive, wait = np.ascontiguousarray(arrive, dtype=np.float64), np.ascontiguousarray(wait, dtype=np.float64)
        b = C.c_int32()
        _check(lib().kvr_controller_calibrate(self._h, _f64p(arrive), _f64p(wait), len(arrive), C.byref(b)))
        return b.value

    def suspend(self, rid, now):
        return lib().kvr_controller_suspend(self._h, rid, now)

    def advance(self, now):
        a, b = C.c_int32(), C.c_int32()
        st = lib().kvr_controller_advance(self._h, now, C.byref(a), C.byref(b))
        return st, a.value, b.value

    def resume(self, rid, now):
        return lib().kvr_controller_resume(self._h, rid, now)

    def stats(self):
        s = ControllerStats()
        _check(lib().kvr_controller_get_stats(self._h, C.byref(s)))
        return {n: getattr(s, n) for n, _ in s._fields_ if n != "reserved"}


def read_load(device_buf, nbytes, launches, device_sink, stream=None):
    """kvr_read_load: enqueue the synthetic HBM-read load (benchmark support)."""
    return lib().kvr_read_load(device_buf, nbytes, launches, device_sink, stream)


def test_plan(geom, n_tokens, slot_bytes, slots, launch_slots, ring_next=0, resume=False, flags=0, suspend_single=0,
              resume_single=0, cap=1 << 16):
    """kvr_test_plan: the staged route's plan for one move, as numpy arrays (chunks[k, 6], copies[j, 5], segs[i, 5])
    and the ring's next slot."""
    g = Geometry(*geom)
    n = np.ascontiguousarray(n_tokens, dtype=np.int64)
    chunks, copies, segs = (np.zeros((cap, w), dtype=np.int64) for w in (6, 5, 5))
    counts = np.zeros(4, dtype=np.int64)
    p64 = lambda a: a.ctypes.data_as(C.POINTER(C.c_int64))   # noqa: E731
    st = lib().kvr_test_plan(C.byref(g), p64(n), len(n), slot_bytes, slots, launch_slots, ring_next, int(resume), flags,
                             suspend_single, resume_single, p64(chunks), p64(copies), p64(segs), cap, p64(counts))
    if st != OK:
        raise KvrError(st, last_error())
    return chunks[:counts[0]].copy(), copies[:counts[1]].copy(), segs[:counts[2]].copy(), int(counts[3])


test_plan.__test__ = False      # a library call, not a pytest test


def numa_lookup(sysfs_root, pci_bus_id, cap=4096):
    """kvr_numa_lookup: (node, [cpus]) of a PCI device under a sysfs tree (None = the machine's /sys)."""
    node = C.c_int32()
    cpus = np.zeros(cap, dtype=np.int32)
    n = lib().kvr_numa_lookup(None if sysfs_root is None else str(sysfs_root).encode(), pci_bus_id.encode(),
                              C.byref(node), cpus.ctypes.data_as(C.POINTER(C.c_int32)), cap)
    return node.value, cpus[:min(n, cap)].tolist()


NOALLOC_MAX_BLOCKS = 65536


def gather_noalloc(device_pool, geom, num_blocks, block_table, n_tokens, dst_device, stream=None):
    """kvr_gather_noalloc: one request's image, pool -> dst, with no allocation anywhere (see include/kvr.h).
    geom = (layers, kv_heads, head_dim, dtype_bytes, block_size); block_table is a host int32 array."""
    g = Geometry(*geom)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    return lib().kvr_gather_noalloc(device_pool, C.byref(g), num_blocks, _i32p(bt) if bt.size else None, bt.size,
                                    n_tokens, dst_device, stream)


def _i32p(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _u64p(a):
    return a.ctypes.data_as(C.POINTER(C.c_uint64))


class Pool:
    """kvr_pool handle.  Methods are the C calls with numpy / int marshalling; statuses are returned, not raised,
    except for errors of pool creation."""

    def __init__(self, layers, kv_heads, head_dim, dtype_bytes, block_size, num_blocks, host_capacity_bytes,
                 initial_free_order=None, device=0, chunk_bytes=0, staging_slots=0, route=0, kernel=0,
                 max_ctas=0, flags=0, device_pool=None, host_arena=None, layout=0, device_staging=None, streams=None,
                 suspend_single_bytes=0, resume_single_bytes=0, copy_piece_bytes=0, max_moves_in_flight=0,
                 bulk_shape=None):
        self.geom = (layers, kv_heads, head_dim, dtype_bytes, block_size)
        self.NB = num_blocks
        cfg = Config()
        cfg.g = Geometry(*self.geom)
        cfg.num_blocks, cfg.device = num_blocks, device
        cfg.host_capacity_bytes, cfg.chunk_bytes, cfg.staging_slots = host_capacity_bytes, chunk_bytes, staging_slots
        cfg.route, cfg.kernel, cfg.max_ctas, cfg.flags, cfg.layout = route, kernel, max_ctas, flags, layout
        self.layout = layout
        cfg.device_pool = device_pool
        cfg.host_arena = host_arena
        cfg.device_staging = device_staging
        if streams is not None:
            if len(streams) != 4:
                raise ValueError("streams: gather, d2h, h2d, scatter")
            for i, st in enumerate(streams):
                cfg.streams[i] = st
        cfg.suspend_single_bytes, cfg.resume_single_bytes = suspend_single_bytes, resume_single_bytes
        cfg.copy_piece_bytes, cfg.max_moves_in_flight = copy_piece_bytes, max_moves_in_flight
        if bulk_shape is not None:
            cfg.bulk_warps, cfg.bulk_stages, cfg.bulk_piece_bytes = bulk_shape
        order = None
        if initial_free_order is not None:
            order = np.ascontiguousarray(initial_free_order, dtype=np.int32)
            if order.size != num_blocks:
                raise ValueError("initial_free_order must have num_blocks entries")
            cfg.initial_free_order = _i32p(order)
        h = C.c_void_p()
        st = lib().kvr_pool_create(C.byref(cfg), C.byref(h))
        if st != OK:
            raise KvrError(st, last_error())
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            st = lib().kvr_pool_destroy(self._h)
            self._h = None
            return st
        return OK

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # -- lifecycle
    def admit(self, rid, n_tokens):
        nb = max(0, -(-n_tokens // self.geom[4]))
        out = np.zeros(max(nb, 1), dtype=np.int32)
        st = lib().kvr_request_admit(self._h, rid, n_tokens, _i32p(out), nb)
        return st, (out[:nb].copy() if st == OK else None)

    def admit_into(self, rid, n_tokens, blocks):
        blocks = np.ascontiguousarray(blocks, dtype=np.int32)
        return lib().kvr_request_admit_into(self._h, rid, n_tokens, _i32p(blocks), len(blocks))

    def release(self, rid):
        return lib().kvr_request_release(self._h, rid)

    def admit_sharing(self, rid, n_tokens, donor, n_shared):
        nb = max(0, -(-n_tokens // self.geom[4]))
        out = np.zeros(max(nb, 1), dtype=np.int32)
        st = lib().kvr_request_admit_sharing(self._h, rid, n_tokens, donor, n_shared, _i32p(out), nb)
        return st, (out[:nb].copy() if st == OK else None)

    def admit_sharing_into(self, rid, n_tokens, donor, n_shared, private_blocks):
        blocks = np.ascontiguousarray(private_blocks, dtype=np.int32)
        return lib().kvr_request_admit_sharing_into(self._h, rid, n_tokens, donor, n_shared, _i32p(blocks), len(blocks))

    def sharing(self, rid):
        """(status, shared-prefix block ids the request refers to)."""
        ns = C.c_int32()
        st = lib().kvr_request_sharing(self._h, rid, C.byref(ns), None, 0)
        if st != OK:
            return st, None
        out = np.zeros(max(ns.value, 1), dtype=np.int32)
        lib().kvr_request_sharing(self._h, rid, None, _i32p(out), ns.value)
        return st, out[:ns.value].copy()

    def refcount(self, blk):
        return int(lib().kvr_block_refcount(self._h, blk))

    def test_fail_nth(self, kind, n):
        return lib().kvr_test_fail_nth(self._h, kind, n)

    def test_points(self, kind):
        return int(lib().kvr_test_points(self._h, kind))

    @property
    def numa_node(self):
        return int(lib().kvr_pool_numa_node(self._h))

    # -- the named calls
    def _batch(self, fn, ids, *flags):
        ids = np.ascontiguousarray(ids, dtype=np.uint64)
        per = np.zeros(max(len(ids), 1), dtype=np.int32)
        st = fn(self._h, _u64p(ids), len(ids), *flags, _i32p(per))
        return st, per[:len(ids)].tolist()

    def retain_in_hbm(self, ids):
        return self._batch(lib().kvr_retain_in_hbm, ids)

    def suspend_to_host(self, ids, flags=0):
        return self._batch(lib().kvr_suspend_to_host, ids, flags)

    def expire(self, ids):
        return self._batch(lib().kvr_expire, ids)

    def resume_from_host(self, ids, flags=0):
        return self._batch(lib().kvr_resume_from_host, ids, flags)

    def resume_from_host_into(self, rid, blocks, flags=0):
        blocks = np.ascontiguousarray(blocks, dtype=np.int32)
        return lib().kvr_resume_from_host_into(self._h, rid, _i32p(blocks), len(blocks), flags)

    def _device_copy(self, fn, ids, ptr, capacity, flags):
        ids = np.ascontiguousarray(ids, dtype=np.uint64)
        offs = np.zeros(max(len(ids), 1), dtype=np.uint64)
        st = fn(self._h, _u64p(ids), len(ids), ptr, capacity, _u64p(offs), flags)
        return st, offs[:len(ids)].copy()

    def export_to_device(self, ids, device_ptr, capacity, flags=0):
        return self._device_copy(lib().kvr_export_to_device, ids, device_ptr, capacity, flags)

    def import_from_device(self, ids, device_ptr, capacity, flags=0):
        return self._device_copy(lib().kvr_import_from_device, ids, device_ptr, capacity, flags)

    # -- observation
    def info(self, rid):
        state, n, nb = C.c_int32(), C.c_int64(), C.c_int32()
        img, nbytes, off = C.c_void_p(), C.c_uint64(), C.c_uint64()
        st = lib().kvr_request_info(self._h, rid, C.byref(state), C.byref(n), C.byref(nb), None, 0,
                                    C.byref(img), C.byref(nbytes), C.byref(off))
        if st != OK:
            return st, None
        d = dict(state=state.value, n_tokens=n.value, nb=nb.value, image_bytes=nbytes.value,
                 arena_offset=off.value, blocks=None, image_ptr=img.value)
        if nb.value >= 0:
            blocks = np.zeros(max(nb.value, 1), dtype=np.int32)
            st2 = lib().kvr_request_info(self._h, rid, None, None, None, _i32p(blocks), nb.value, None, None, None)
            if st2 == OK and state.value in (ACTIVE, RETAINED, RESUMING):
                d["blocks"] = blocks[:nb.value].copy()
        return st, d

    def host_image(self, rid):
        """Borrowed uint8 numpy view of a HOST request's image in the pinned arena (wait for the suspend first)."""
        st, d = self.info(rid)
        if st != OK or not d["image_ptr"]:
            return None
        if d["image_bytes"] == 0:
            return np.zeros(0, dtype=np.uint8)
        buf = (C.c_uint8 * d["image_bytes"]).from_address(d["image_ptr"])
        return np.frombuffer(buf, dtype=np.uint8)

    def latency(self, rid):
        h, dv = C.c_double(), C.c_double()
        st = lib().kvr_request_latency(self._h, rid, C.byref(h), C.byref(dv))
        return st, h.value, dv.value

    def wait(self, rid=ALL, timeout_ms=-1):
        return lib().kvr_wait(self._h, rid, timeout_ms)

    def stats(self):
        s = Stats()
        st = lib().kvr_pool_stats(self._h, C.byref(s))
        if st != OK:
            raise KvrError(st, last_error())
        return s.as_dict()

    def selftest_bounded_wait(self, leave_error_set=False):
        return lib().kvr_selftest_bounded_wait(self._h, int(leave_error_set))

    def selftest_block_check(self, leave_error_set=False):
        return lib().kvr_selftest_block_check(self._h, int(leave_error_set))

    def clear_device_error(self):
        return lib().kvr_clear_device_error(self._h)

    def probe_link(self, nbytes=2 << 30, reps=10):
        """kvr_probe_link: best pinned-copy rate per direction over this pool's arena, GB/s."""
        a, b = C.c_double(), C.c_double()
        st = lib().kvr_probe_link(self._h, nbytes, reps, C.byref(a), C.byref(b))
        return st, a.value, b.value

    def free_queue(self):
        n = int(lib().kvr_free_queue(self._h, None, 0))
        out = np.zeros(max(n, 1), dtype=np.int32)
        lib().kvr_free_queue(self._h, _i32p(out), n)
        return out[:n].copy()

    @property
    def device_ptr(self):
        return lib().kvr_pool_device_ptr(self._h)

    @property
    def host_arena_ptr(self):
        return lib().kvr_pool_host_arena(self._h)
