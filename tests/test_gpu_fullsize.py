"""Parity at the full sizes of the Llama-2-7B-shaped (SwiGLU) and OPT-13B-shaped configurations,
through the same launch configurations the benchmark and the sweep tool time: scoring + selection
against the oracle (indices bit-exact), then the split forward at prefill and decode sizes, and the
dense layer (every neuron heavy) through the same kernels.

Few-token outputs are compared element by element.  At prefill sizes the GPU runs the full token
count (the launch configuration that is timed) and the oracle computes a sample of the token rows
one by one -- every eighth row, so that every 128-token tile of the GPU kernels contributes rows:
tokens are independent in an FFN, so a row of the full-size call is checked exactly as it would be in
a smaller one.  Light factors are seeded random matrices here: parity is taken against the factors
actually packed, and an fp64 SVD of these shapes would take minutes."""
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


def sampled_rows(T):
    """All rows of a few-token batch; every eighth row of a prefill batch (each 128-row tile gives 16)."""
    return slice(None) if T <= 512 else slice(3, None, 8)


def check_score_and_select(G, L, cfg, t_cal):
    """GPU scores and indices against the oracle on the same calibration tokens.  Planted layers have a gap of
    about 100x at the k-th score, so index equality is required; for an unplanted layer equality is required
    only when the oracle's relative gap at the boundary exceeds the score tolerance, otherwise both sets are
    correct and the GPU's set must agree with the oracle's on every neuron outside the ambiguous band."""
    Xc = L.tokens(t_cal)
    _, scores = G.score(Xc, batches=2)
    heavy, light = G.select(scores, cfg.k)
    _, _, s_ref = orc.neuron_scores(f64(Xc), f64(L.W1), f64(L.b1), f64(L.W2), cfg.act, orc.SCORE_EQ3, f64(L.W1u))
    heavy_ref, light_ref = orc.select_heavy(s_ref, cfg.k)
    rtol = 2e-3
    assert np.allclose(f64(scores), s_ref, rtol=rtol)
    order = np.sort(s_ref)[::-1]
    gap = (order[cfg.k - 1] - order[cfg.k]) / order[cfg.k - 1]
    h_gpu = heavy.cpu().numpy()
    if gap > 1e-2:
        assert np.array_equal(h_gpu, heavy_ref) and np.array_equal(light.cpu().numpy(), light_ref)
    else:
        # boundary inside the score error: neurons clearly above the k-th score must be in, clearly below out
        thr = order[cfg.k - 1]
        sure_in = np.nonzero(s_ref > thr * (1 + 2 * rtol))[0]
        sure_out = np.nonzero(s_ref < thr * (1 - 2 * rtol))[0]
        assert np.isin(sure_in, h_gpu).all() and not np.isin(sure_out, h_gpu).any()
        assert h_gpu.size == cfg.k and np.all(np.diff(h_gpu) > 0)
        # the GPU's own decision is exact on its own scores
        own_ref, _ = orc.select_heavy(f64(scores).astype(np.float32), cfg.k)
        assert np.array_equal(h_gpu, own_ref)
    return heavy_ref, gap


CASES = [
    # name, config, calibration tokens, planted, forward token counts
    ("llama2_7b", CONFIGS[4], 8192, True, (2048, 32, 8, 1)),
    ("llama2_7b_unplanted", CONFIGS[4], 2048, False, (32,)),
    ("opt_13b_5pct_r512", cfg5_point(5, 512), 4096, True, (4096, 32, 1)),
    ("opt_13b_1pct_r256", cfg5_point(1, 256), 2048, True, (4096, 32, 1)),     # r = 256: fused light chain at d = 5120
    ("opt_13b_1pct_r1280", cfg5_point(1, 1280), 1024, True, (4096, 32, 1)),   # r_pad > 1024: stage 2a with K = 1280
    ("opt_13b_10pct_r256", cfg5_point(10, 256), 1024, True, (4096, 32, 1)),   # stage 3 with K = 2304: 256-row tiles
    ("opt_13b_10pct_r1280", cfg5_point(10, 1280), 1024, True, (4096, 32, 1)),
]


@pytest.mark.parametrize("name,cfg,t_cal,planted,tokens", CASES, ids=[c[0] for c in CASES])
def test_full_size_layer(ctx, name, cfg, t_cal, planted, tokens):
    L = make_layer(cfg, 0, plant=planted)
    G = GpuLayer(ctx, L)
    G.reserve(max(tokens), t_cal, cfg.k, cfg.r)
    heavy_ref, gap = check_score_and_select(G, L, cfg, t_cal)
    if planted:
        assert gap > 1e-2 and np.array_equal(heavy_ref, L.planted.numpy())
    fac = seeded_factors(cfg, 99)
    blob, logical = G.pack(torch.from_numpy(heavy_ref), fac)
    assert logical == 2 * (orc.split_weight_params(cfg.d, cfg.m, cfg.k, cfg.r, cfg.n_in) + cfg.m + cfg.d)
    for T in tokens:
        X = L.tokens(T)
        Y = G.forward(blob, X)
        rows = sampled_rows(T)
        assert_close(Y[rows], oracle_split(L, heavy_ref, fac, X[rows]), "bf16", f"{name} T={T}")


@pytest.mark.parametrize("cid,tokens", [(4, (2048, 1)), (5, (4096, 32, 1))], ids=["llama2_7b_dense", "opt_13b_dense"])
def test_full_size_dense_layer(ctx, cid, tokens):
    """The dense comparator (k = m) at the sizes its throughput is quoted on: the 256-row-tile GEMMs at prefill,
    the weight-streaming kernel at few tokens."""
    cfg = CONFIGS[cid]
    L = make_layer(cfg, 1)
    G = GpuLayer(ctx, L)
    G.reserve(max(tokens), 0, cfg.m, 0)
    blob, _ = G.pack(torch.arange(cfg.m), None)
    for T in tokens:
        X = L.tokens(T)
        Y = G.forward(blob, X)
        rows = sampled_rows(T)
        ref = orc.dense_ffn(f64(X[rows]), f64(L.W1), f64(L.b1), f64(L.W2), f64(L.b2), cfg.act, f64(L.W1u))
        assert_close(Y[rows], ref, "bf16", f"config {cid} dense T={T}")
