"""Helpers for the GPU parity tests: a library pool over torch-owned device memory next to an oracle
pool holding the same bytes."""
import numpy as np
import torch

import oracle as orc
from kvr_synth import fill_bytes
from paper_2608_30830_b200 import kvr


class Twin:
    """Oracle pool + library pool with identical geometry, free order and initial pool bytes."""

    def __init__(self, geom, NB, host_cap, seed=0, order=None, layout=0, **lib_kw):
        L, H, D, e, BS = geom
        self.geom, self.NB = geom, NB
        if order is None:
            order = np.random.default_rng(seed).permutation(NB).astype(np.int32)
        self.layout = layout
        self.o = orc.OrcPool(*geom, NB, host_cap, initial_free_order=order, with_data=True, layout=layout)
        nbytes = self.o.data.size
        self.o.data[:] = fill_bytes(seed, 0, nbytes, e)
        self.dev = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self.dev.copy_(torch.from_numpy(self.o.data))
        torch.cuda.synchronize()
        self.g = kvr.Pool(*geom, NB, host_cap, initial_free_order=order, device_pool=self.dev.data_ptr(), layout=layout, **lib_kw)

    def pool_bytes(self):
        assert self.g.wait() == kvr.OK
        torch.cuda.synchronize()
        return self.dev.cpu().numpy()

    def both(self, name, *args):
        a = getattr(self.o, name)(*args)
        b = getattr(self.g, name)(*args)
        return a, b

    def assert_same_images(self, ids):
        assert self.g.wait() == kvr.OK
        for rid in ids:
            st, d = self.o.info(rid)
            if st != orc.OK or d["state"] != orc.HOST:
                continue
            got = self.g.host_image(rid)
            assert got is not None and np.array_equal(got, d["image"]), "image of request %d differs" % rid

    def assert_same_pool(self):
        got = self.pool_bytes()
        if not np.array_equal(got, self.o.data):
            bad = np.flatnonzero(got != self.o.data)
            raise AssertionError("pool differs at %d bytes, first at %d" % (bad.size, bad[0]))

    def close(self):
        self.g.close()
        self.o.close()
        del self.dev
