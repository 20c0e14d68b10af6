"""The host-side factorisation helper (Section 5.1.1: truncated SVD of the light slices U2, V2) against what
the mathematics fixes and against the oracle's own factors.  Factors are not unique (signs, rotations inside
equal singular values), so only the products A @ B are compared."""
import numpy as np
import torch

from ffsplit_synth import custom_config, make_layer
from oracle import ffsplit_oracle as orc
from paper_2401_04044_b200.factors import light_factors, truncated_factors


def test_truncated_factors_meet_eckart_young():
    g = torch.Generator().manual_seed(7)
    W = torch.randn(48, 130, generator=g, dtype=torch.float64) * torch.linspace(2.0, 0.1, 130, dtype=torch.float64)
    sv2 = np.sort(np.linalg.eigvalsh((W @ W.T).numpy()))[::-1]          # squared singular values, another route
    for r in (0, 1, 7, 48):
        A, B = truncated_factors(W, r, torch.float64)
        assert A.shape == (48, r) and B.shape == (r, 130)
        res = float(torch.linalg.norm(W - A @ B) ** 2)
        assert abs(res - sv2[r:].sum()) <= 1e-9 * sv2.sum()             # best rank-r residual = tail of the spectrum
    A, B = truncated_factors(W, 48, torch.float64)
    assert torch.allclose(A @ B, W, atol=1e-12)
    # singular values are split evenly: the Gram matrices of the two factors carry the same spectrum
    A, B = truncated_factors(W, 5, torch.float64)
    assert np.allclose(np.linalg.eigvalsh((A.T @ A).numpy()), np.linalg.eigvalsh((B @ B.T).numpy()), rtol=1e-9)


def test_light_factors_agree_with_the_oracle_in_the_product():
    for act in ("gelu_erf", "swiglu"):
        cfg = custom_config(64, 256, 20, 24, act=act, dtype="f32")
        L = make_layer(cfg, 3)
        heavy = L.planted
        mask = torch.ones(cfg.m, dtype=torch.bool)
        mask[heavy] = False
        light = torch.nonzero(mask).flatten()
        f = light_factors(L.W1, L.W2, light, cfg.r, L.W1u)
        sw = orc.split_weights(L.W1.double().numpy(), None, L.W2.double().numpy(), heavy.numpy(),
                               None if L.W1u is None else L.W1u.double().numpy())
        pairs = [("A1", "B1", "U2"), ("A2", "B2", "V2")] + ([("A1u", "B1u", "U2u")] if act == "swiglu" else [])
        for a, b, name in pairs:
            Ao, Bo = orc.light_factors(sw[name], cfg.r)
            ours = f[a].double().numpy() @ f[b].double().numpy()
            scale = np.abs(Ao @ Bo).max()
            # the helper rounds its factors to the storage type (fp32 here): agreement to that rounding
            assert np.abs(ours - Ao @ Bo).max() <= 1e-5 * scale
            assert f[a].dtype == L.W1.dtype and f[a].shape == (sw[name].shape[0], cfg.r)
