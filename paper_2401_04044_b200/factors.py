"""Host-side helper for the step between selection and packing: rank-r factors
of the light slices by truncated SVD (Section 5.1.1: SVD is applied to U2 and V2
only).  This is set-up work done with torch.linalg, not a library call; the
library consumes the factors through ffsplit_pack.
"""
from __future__ import annotations

import torch


def truncated_factors(W: torch.Tensor, r: int, out_dtype: torch.dtype):
    """W [p, q] -> A [p, r], B [r, q] with A @ B the best rank-r approximation,
    singular values split evenly between the factors.  The decomposition is taken in
    float64 on whichever device holds W; only the factors are rounded to out_dtype."""
    Wf = W.to(torch.float64)
    U, S, Vh = torch.linalg.svd(Wf, full_matrices=False)
    root = S[:r].sqrt()
    A = (U[:, :r] * root[None, :]).to(out_dtype).contiguous()
    B = (root[:, None] * Vh[:r, :]).to(out_dtype).contiguous()
    return A, B


def light_factors(W1, W2, light_idx, r: int, W1u=None) -> dict:
    """Factors of U2 = W1[:, light], V2 = W2[light, :] (and the SwiGLU up slice)."""
    li = light_idx.long()
    dt = W1.dtype
    f = {}
    f["A1"], f["B1"] = truncated_factors(W1[:, li], r, dt)
    f["A2"], f["B2"] = truncated_factors(W2[li, :], r, dt)
    if W1u is not None:
        f["A1u"], f["B1u"] = truncated_factors(W1u[:, li], r, dt)
    return f
