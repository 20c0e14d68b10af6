"""Parity at the full sizes of the Llama-2-7B-shaped (SwiGLU) and OPT-13B-shaped configurations,
through the same launch configurations the sweep tool times: scoring + selection against the
oracle (indices bit-exact), then the split forward at prefill and decode sizes, every output
element compared.  Light factors are seeded random matrices here: parity is taken against the
factors actually packed, and an fp64 SVD of these shapes would take minutes."""
import numpy as np
import pytest
import torch

from conftest import f64
from ffsplit_synth import CONFIGS, cfg5_point, make_layer
from helpers import GpuLayer, assert_close, oracle_split
from oracle import ffsplit_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2401_04044_b200 import Context, build
    build.build()
    c = Context(0)
    yield c
    c.close()


def seeded_factors(cfg, seed):
    g = torch.Generator().manual_seed(seed)
    d, ml, r, dt = cfg.d, cfg.m - cfg.k, cfg.r, cfg.torch_dtype
    mk = lambda *s: (torch.randn(*s, generator=g) * 0.02).to(dt)
    f = {"A1": mk(d, r), "B1": mk(r, ml), "A2": mk(ml, r), "B2": mk(r, d)}
    if cfg.act == "swiglu":
        f["A1u"], f["B1u"] = mk(d, r), mk(r, ml)
    return f


@pytest.mark.parametrize("name,cfg,t_cal,tokens", [
    ("llama2_7b", CONFIGS[4], 8192, (2048, 32, 1)),
    ("opt_13b_5pct_r512", cfg5_point(5, 512), 4096, (4096, 32, 1)),
    ("opt_13b_1pct_r256", cfg5_point(1, 256), 2048, (512,)),      # r = 256: fused light chain at d = 5120
])
def test_full_size_layer(ctx, name, cfg, t_cal, tokens):
    L = make_layer(cfg, 0)
    G = GpuLayer(ctx, L)
    G.reserve(max(tokens), t_cal, cfg.k, cfg.r)
    Xc = L.tokens(t_cal)
    _, scores = G.score(Xc, batches=2)
    heavy, light = G.select(scores, cfg.k)
    _, _, s_ref = orc.neuron_scores(f64(Xc), f64(L.W1), f64(L.b1), f64(L.W2), cfg.act, orc.SCORE_EQ3, f64(L.W1u))
    heavy_ref, light_ref = orc.select_heavy(s_ref, cfg.k)
    assert np.array_equal(heavy.cpu().numpy(), heavy_ref) and np.array_equal(light.cpu().numpy(), light_ref)
    assert np.array_equal(heavy_ref, L.planted.numpy())
    assert np.allclose(f64(scores), s_ref, rtol=2e-3)
    del s_ref
    fac = seeded_factors(cfg, 99)
    blob, logical = G.pack(heavy, fac)
    es = 2
    assert logical == es * (orc.split_weight_params(cfg.d, cfg.m, cfg.k, cfg.r, cfg.n_in) + cfg.m + cfg.d)
    for T in tokens:
        X = L.tokens(T)
        Y = G.forward(blob, X)
        assert_close(Y, oracle_split(L, heavy_ref, fac, X), "bf16", f"{name} T={T}")
