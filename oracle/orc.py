"""ctypes binding of the plain-C oracle (kvr_oracle.c).  TEST INFRASTRUCTURE ONLY.

Argument marshalling only: every rule of the method lives in the C file, where
each function names the passage of the paper it restates.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_DIR, "libkvr_oracle.so")
_SRC = [os.path.join(_DIR, "kvr_oracle.c"), os.path.join(_DIR, "kvr_oracle.h")]

OK, RESIDENT, RECOMPUTE, HOST_FULL, HBM_FULL = 0, 1, 2, 3, 4
ERR_INVALID_ARG, ERR_UNKNOWN_REQUEST, ERR_BAD_STATE, ERR_GEOMETRY, ERR_NOMEM = -1, -2, -3, -4, -7
ACTIVE, RETAINED, HOST, EXPIRED = 0, 1, 3, 5
LAYER_MAJOR, BLOCK_MAJOR = 0, 1


def build(force=False):
    """Compile the oracle with gcc (plain C11, no CUDA)."""
    stale = (not os.path.exists(_SO)) or any(os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC)
    if force or stale:
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-std=c11", "-O2", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", tmp, _SRC[0]])
        os.replace(tmp, _SO)
    return _SO


class OrcStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("blocks_total", "blocks_free", "blocks_active", "blocks_pinned")] + \
               [(n, C.c_uint64) for n in ("host_capacity", "host_used", "host_largest_hole")] + \
               [(n, C.c_int64) for n in ("n_active", "n_retained", "n_host", "n_expired",
                                         "suspends", "resumes", "resident_resumes", "expires",
                                         "recompute_marked", "host_full_rejects", "hbm_full_rejects")] + \
               [(n, C.c_uint64) for n in ("bytes_suspended", "bytes_resumed", "bytes_expired_from_host")]

    def as_dict(self):
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        i32, i64, u64, vp = C.c_int32, C.c_int64, C.c_uint64, C.c_void_p
        pi32, pu64 = C.POINTER(C.c_int32), C.POINTER(C.c_uint64)
        L = _lib
        L.orc_bytes_per_token.restype = u64
        L.orc_bytes_per_token.argtypes = [i32] * 4
        L.orc_pool_offset.restype = u64
        L.orc_pool_offset.argtypes = [i32] * 14
        L.orc_image_offset.restype = u64
        L.orc_image_offset.argtypes = [i32, i32, i32, i32, i64, i32, i32, i64, i32, i32, i32]
        L.orc_pool_create.restype = vp
        L.orc_pool_create.argtypes = [i32] * 6 + [u64, pi32, i32, i32]
        L.orc_pool_destroy.restype = None
        L.orc_pool_destroy.argtypes = [vp]
        L.orc_pool_data.restype = vp
        L.orc_pool_data.argtypes = [vp]
        L.orc_pool_bytes.restype = u64
        L.orc_pool_bytes.argtypes = [vp]
        L.orc_request_admit.restype = i32
        L.orc_request_admit.argtypes = [vp, u64, i64, pi32, i32]
        L.orc_request_admit_into.restype = i32
        L.orc_request_admit_into.argtypes = [vp, u64, i64, pi32, i32]
        L.orc_request_release.restype = i32
        L.orc_request_release.argtypes = [vp, u64]
        L.orc_request_admit_sharing.restype = i32
        L.orc_request_admit_sharing.argtypes = [vp, u64, i64, u64, i32, pi32, i32]
        L.orc_request_admit_sharing_into.restype = i32
        L.orc_request_admit_sharing_into.argtypes = [vp, u64, i64, u64, i32, pi32, i32]
        L.orc_request_sharing.restype = i32
        L.orc_request_sharing.argtypes = [vp, u64, pi32, pi32, i32]
        L.orc_block_refcount.restype = i32
        L.orc_block_refcount.argtypes = [vp, i32]
        for name in ("orc_retain_in_hbm", "orc_suspend_to_host", "orc_expire", "orc_resume_from_host"):
            f = getattr(L, name)
            f.restype = i32
            f.argtypes = [vp, pu64, i32, pi32]
        L.orc_resume_from_host_into.restype = i32
        L.orc_resume_from_host_into.argtypes = [vp, u64, pi32, i32]
        L.orc_request_info.restype = i32
        L.orc_request_info.argtypes = [vp, u64, pi32, C.POINTER(i64), pi32, pi32, i32,
                                       C.POINTER(vp), pu64, pu64]
        L.orc_pool_stats.restype = i32
        L.orc_pool_stats.argtypes = [vp, C.POINTER(OrcStats)]
        L.orc_free_queue.restype = i64
        L.orc_free_queue.argtypes = [vp, pi32, i64]
        for name in ("orc_gather", "orc_scatter"):
            f = getattr(L, name)
            f.restype = None
            f.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, pi32, i64, i32]
    return _lib


def bytes_per_token(layers, kv_heads, head_dim, dtype_bytes):
    return int(lib().orc_bytes_per_token(layers, kv_heads, head_dim, dtype_bytes))


def pool_offset(L, H, D, e, BS, NB, l, kv, blk, slot, h=0, d=0, byte=0, layout=LAYER_MAJOR):
    return int(lib().orc_pool_offset(L, H, D, e, BS, NB, l, kv, blk, slot, h, d, byte, layout))


def image_offset(L, H, D, e, n, l, kv, t, h=0, d=0, byte=0):
    return int(lib().orc_image_offset(L, H, D, e, n, l, kv, t, h, d, byte))


def _i32p(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def gather(pool, L, H, D, e, BS, NB, bt, n, layout=LAYER_MAJOR):
    """image = gather(pool) for one request; pool is a flat uint8 array."""
    bt = np.ascontiguousarray(bt, dtype=np.int32)
    image = np.zeros(n * 2 * L * H * D * e, dtype=np.uint8)
    lib().orc_gather(pool.ctypes.data, image.ctypes.data, L, H, D, e, BS, NB, _i32p(bt), n, layout)
    return image


def scatter(pool, image, L, H, D, e, BS, NB, bt, n, layout=LAYER_MAJOR):
    bt = np.ascontiguousarray(bt, dtype=np.int32)
    image = np.ascontiguousarray(image, dtype=np.uint8)
    lib().orc_scatter(pool.ctypes.data, image.ctypes.data, L, H, D, e, BS, NB, _i32p(bt), n, layout)


class OrcPool:
    """One oracle pool.  Methods mirror the C-ABI call set of the product library."""

    def __init__(self, L, H, D, e, BS, NB, host_capacity, initial_free_order=None, with_data=True,
                 layout=LAYER_MAJOR):
        self.geom = (L, H, D, e, BS)
        self.NB = NB
        self.layout = layout
        order = None
        if initial_free_order is not None:
            order = np.ascontiguousarray(initial_free_order, dtype=np.int32)
        self._h = lib().orc_pool_create(L, H, D, e, BS, NB, host_capacity,
                                        _i32p(order) if order is not None else None, int(with_data), layout)
        if not self._h:
            raise ValueError("orc_pool_create failed (geometry, free order or memory)")
        self.with_data = with_data

    def close(self):
        if self._h:
            lib().orc_pool_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    @property
    def data(self):
        """The pool bytes as a writable flat uint8 numpy view (with_data only)."""
        n = int(lib().orc_pool_bytes(self._h))
        ptr = lib().orc_pool_data(self._h)
        buf = (C.c_uint8 * n).from_address(ptr)
        return np.frombuffer(buf, dtype=np.uint8)

    def admit(self, rid, n_tokens):
        nb = (n_tokens + self.geom[4] - 1) // self.geom[4] if n_tokens >= 0 else 0
        out = np.zeros(max(nb, 1), dtype=np.int32)
        st = lib().orc_request_admit(self._h, rid, n_tokens, _i32p(out), nb)
        return st, (out[:nb].copy() if st == OK else None)

    def admit_into(self, rid, n_tokens, blocks):
        blocks = np.ascontiguousarray(blocks, dtype=np.int32)
        return lib().orc_request_admit_into(self._h, rid, n_tokens, _i32p(blocks), len(blocks))

    def release(self, rid):
        return lib().orc_request_release(self._h, rid)

    def admit_sharing(self, rid, n_tokens, donor, n_shared):
        nb = (n_tokens + self.geom[4] - 1) // self.geom[4] if n_tokens >= 0 else 0
        out = np.zeros(max(nb, 1), dtype=np.int32)
        st = lib().orc_request_admit_sharing(self._h, rid, n_tokens, donor, n_shared, _i32p(out), nb)
        return st, (out[:nb].copy() if st == OK else None)

    def admit_sharing_into(self, rid, n_tokens, donor, n_shared, private_blocks):
        blocks = np.ascontiguousarray(private_blocks, dtype=np.int32)
        return lib().orc_request_admit_sharing_into(self._h, rid, n_tokens, donor, n_shared, _i32p(blocks), len(blocks))

    def sharing(self, rid):
        """(status, shared-prefix block ids the request refers to)."""
        ns = C.c_int32()
        st = lib().orc_request_sharing(self._h, rid, C.byref(ns), None, 0)
        if st != OK:
            return st, None
        out = np.zeros(max(ns.value, 1), dtype=np.int32)
        lib().orc_request_sharing(self._h, rid, None, _i32p(out), ns.value)
        return st, out[:ns.value].copy()

    def refcount(self, blk):
        return int(lib().orc_block_refcount(self._h, blk))

    def _batch(self, fn, ids):
        ids = np.ascontiguousarray(ids, dtype=np.uint64)
        per = np.zeros(max(len(ids), 1), dtype=np.int32)
        st = fn(self._h, ids.ctypes.data_as(C.POINTER(C.c_uint64)), len(ids), _i32p(per))
        return st, per[:len(ids)].tolist()

    def retain_in_hbm(self, ids):
        return self._batch(lib().orc_retain_in_hbm, ids)

    def suspend_to_host(self, ids):
        return self._batch(lib().orc_suspend_to_host, ids)

    def expire(self, ids):
        return self._batch(lib().orc_expire, ids)

    def resume_from_host(self, ids):
        return self._batch(lib().orc_resume_from_host, ids)

    def resume_from_host_into(self, rid, blocks):
        blocks = np.ascontiguousarray(blocks, dtype=np.int32)
        return lib().orc_resume_from_host_into(self._h, rid, _i32p(blocks), len(blocks))

    def info(self, rid):
        state, n, nb = C.c_int32(), C.c_int64(), C.c_int32()
        img, nbytes, off = C.c_void_p(), C.c_uint64(), C.c_uint64()
        st = lib().orc_request_info(self._h, rid, C.byref(state), C.byref(n), C.byref(nb), None, 0,
                                    C.byref(img), C.byref(nbytes), C.byref(off))
        if st != OK:
            return st, None
        d = dict(state=state.value, n_tokens=n.value, nb=nb.value, image_bytes=nbytes.value,
                 arena_offset=off.value, blocks=None, image=None)
        if state.value in (ACTIVE, RETAINED):
            blocks = np.zeros(max(nb.value, 1), dtype=np.int32)
            lib().orc_request_info(self._h, rid, None, None, None, _i32p(blocks), nb.value, None, None, None)
            d["blocks"] = blocks[:nb.value].copy()
        if state.value == HOST and img.value and nbytes.value:
            buf = (C.c_uint8 * nbytes.value).from_address(img.value)
            d["image"] = np.frombuffer(buf, dtype=np.uint8)
        elif state.value == HOST and self.with_data:
            d["image"] = np.zeros(0, dtype=np.uint8)
        return st, d

    def stats(self):
        s = OrcStats()
        lib().orc_pool_stats(self._h, C.byref(s))
        return s.as_dict()

    def free_queue(self):
        n = int(lib().orc_free_queue(self._h, None, 0))
        out = np.zeros(max(n, 1), dtype=np.int32)
        lib().orc_free_queue(self._h, _i32p(out), n)
        return out[:n].copy()
