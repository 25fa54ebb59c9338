"""Helpers for the GPU parity tests: run a workload through the C ABI and hand back numpy."""
from __future__ import annotations

import numpy as np

from paper_2502_07021_b200 import binding as fs


class GpuSolver:
    """Owns the device copies of one workload and a solver handle (freed on close)."""

    def __init__(self, M, kind, eps, a, b, offsets, domain, ld=None, misalign=0):
        import torch
        self.torch = torch
        M = np.asarray(M, dtype=np.float32)
        n = M.shape[0]
        a = np.asarray(a, dtype=np.float32)
        b = np.asarray(b, dtype=np.float32)
        self.n = n
        self.nbatch = 1 if a.ndim == 1 else a.shape[0]
        self.domain = domain
        self.ld = int(ld or n)
        dev = torch.device("cuda:0")
        # optional padding of the leading dimension and a deliberately misaligned base pointer
        store = torch.zeros(n * self.ld + misalign + 8, dtype=torch.float32, device=dev)
        self.M_store = store
        self.M_dev = store[misalign:misalign + n * self.ld].view(n, self.ld)
        self.M_dev[:, :n].copy_(torch.from_numpy(M))
        if self.ld > n:
            self.M_dev[:, n:] = float("nan")   # padding must never be read into a result
        self.a_dev = torch.from_numpy(a).to(dev).contiguous()
        self.b_dev = torch.from_numpy(b).to(dev).contiguous()
        self.offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        self.c = self.offsets.size - 1
        self.stream = torch.cuda.Stream(device=dev)
        torch.cuda.synchronize()
        self.h = fs.fs_create(n, self.c, self.offsets, self.M_dev.data_ptr(), self.ld, kind, eps, self.a_dev,
                              self.b_dev, self.nbatch, domain, self.stream)

    def iterate(self, k):
        fs.fs_iterate(self.h, k, self.stream)

    def scalings(self):
        torch = self.torch
        shape = (self.n,) if self.nbatch == 1 else (self.nbatch, self.n)
        u = torch.empty(shape, dtype=torch.float32, device="cuda:0")
        v = torch.empty(shape, dtype=torch.float32, device="cuda:0")
        fs.fs_scalings(self.h, u, v, self.stream)
        return u.cpu().numpy(), v.cpu().numpy()

    def set_scalings(self, u=None, v=None):
        torch = self.torch
        ud = None if u is None else torch.from_numpy(np.ascontiguousarray(u, dtype=np.float32)).to("cuda:0")
        vd = None if v is None else torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).to("cuda:0")
        fs.fs_set_scalings(self.h, ud, vd, self.stream)
        self.stream.synchronize()

    def errors(self, norm=1):
        return fs.fs_marginal_error(self.h, norm, self.nbatch, self.stream)

    def cost(self, C=None):
        if C is None:
            return fs.fs_transport_cost(self.h, None, 0, self.nbatch, self.stream)
        Cd = self.torch.from_numpy(np.ascontiguousarray(C, dtype=np.float32)).to("cuda:0")
        return fs.fs_transport_cost(self.h, Cd, C.shape[1], self.nbatch, self.stream)

    def close(self):
        if self.h is not None:
            fs.fs_destroy(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def rel_err(x, ref):
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(np.asarray(x, dtype=np.float64) - ref) / np.abs(ref)))
