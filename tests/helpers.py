"""Shared plumbing for the GPU parity tests: run the library's four calls on a
synthetic layer and compute the oracle's answer for the same stored inputs."""
import numpy as np
import torch

from conftest import f64
from oracle import ffsplit_oracle as orc

TOL = {"bf16": (1e-2, 2e-2), "f32": (1e-5, 1e-5)}   # (relative Frobenius, max-abs / max|Y*|)
SCORE_RTOL = {"bf16": 2e-3, "f32": 1e-4}


def to_dev(t, dev="cuda"):
    return None if t is None else t.to(dev).contiguous()


def oracle_factors(L, heavy, r):
    """Rank-r light factors from the oracle's SVD, rounded once to the storage dtype."""
    sw = orc.split_weights(f64(L.W1), f64(L.b1), f64(L.W2), heavy, f64(L.W1u))
    dt = L.cfg.torch_dtype
    cast = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dt).contiguous()
    f = {}
    a, b = orc.light_factors(sw["U2"], r); f["A1"], f["B1"] = cast(a), cast(b)
    a, b = orc.light_factors(sw["V2"], r); f["A2"], f["B2"] = cast(a), cast(b)
    if L.W1u is not None:
        a, b = orc.light_factors(sw["U2u"], r); f["A1u"], f["B1u"] = cast(a), cast(b)
    return f


def oracle_split(L, heavy, factors, X):
    fac = None if factors is None else {k: f64(v) for k, v in factors.items()}
    return orc.split_ffn(f64(X), f64(L.W1), f64(L.b1), f64(L.W2), f64(L.b2), heavy, fac, L.cfg.act, f64(L.W1u))


class GpuLayer:
    """Device copies of one layer and the library context driving it."""

    def __init__(self, ctx, L):
        import paper_2401_04044_b200 as ff
        self.ff, self.ctx, self.L = ff, ctx, L
        self.shape = ff.make_shape(L.cfg.d, L.cfg.m, L.cfg.act, L.cfg.torch_dtype)
        self.W1, self.W1u, self.b1 = to_dev(L.W1), to_dev(L.W1u), to_dev(L.b1)
        self.W2, self.b2 = to_dev(L.W2), to_dev(L.b2)

    def reserve(self, T_fwd, T_cal, k, r):
        self.ctx.ensure_workspace(self.ctx.workspace_size(self.shape, T_fwd, T_cal, k, r))

    def score(self, X, mode=0, batches=1):
        m = self.L.cfg.m
        energy = torch.empty(m, dtype=torch.float32, device="cuda")
        scores = torch.empty(m, dtype=torch.float32, device="cuda")
        Xd = to_dev(X)
        chunks = torch.chunk(Xd, batches, dim=0)
        for i, xc in enumerate(chunks):
            xc = xc.clone()      # own allocation: chunk views of an odd-width X are not 16-byte aligned
            self.ctx.score(self.shape, self.W1, self.b1, self.W2, xc, energy,
                           scores if i == len(chunks) - 1 else None, mode=mode, accumulate=i > 0, W1u=self.W1u)
        self.ctx.poll()
        return energy, scores

    def select(self, scores, k):
        m = scores.numel()
        heavy = torch.full((max(k, 1),), -1, dtype=torch.int32, device="cuda")
        light = torch.full((max(m - k, 1),), -1, dtype=torch.int32, device="cuda")
        self.ctx.select(scores, k, heavy, light)
        self.ctx.poll()
        return heavy[:k], light[:m - k]

    def pack(self, heavy, factors):
        k = int(heavy.numel())
        r = 0 if factors is None else int(factors["A1"].shape[1])
        padded, logical = self.ctx.pack_size(self.shape, k, r)
        blob = torch.empty(padded, dtype=torch.uint8, device="cuda")
        fd = None if factors is None else {n: to_dev(v) for n, v in factors.items()}
        self._keep = fd
        self.ctx.pack(self.shape, self.W1, self.b1, self.W2, self.b2, heavy.to(torch.int32).cuda().contiguous(), k, fd,
                      blob, W1u=self.W1u)
        self.ctx.poll()
        return blob, logical

    def forward(self, blob, X):
        Xd = to_dev(X)
        Y = torch.empty_like(Xd)
        self.ctx.forward(blob, Xd, Y)
        self.ctx.poll()
        return Y


def assert_close(Y, Yref, dtype_name, what=""):
    fro = orc.rel_frobenius(f64(Y), Yref)
    mx = orc.normalised_max_abs(f64(Y), Yref)
    tf, tm = TOL[dtype_name]
    assert fro <= tf and mx <= tm, f"{what}: rel-Frobenius {fro:.3e} (<= {tf}), max-abs {mx:.3e} (<= {tm})"
    return fro, mx
