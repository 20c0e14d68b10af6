"""On-device factorisation of the light slices (Section 5.1.1: low-rank decomposition of U2 and V2) against the
oracle: the truncated SVD (Eckart-Young) fixes the best possible residual, the oracle's orthogonal iteration
from the same starting basis fixes what the device routine should reach, and the factors it returns go through
pack and forward like any others."""
import numpy as np
import pytest
import torch

from conftest import f64
from ffsplit_synth import CONFIGS, custom_config, make_layer
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


def start_basis(n, r, d, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(n, r, d, generator=g).to(dtype)


def slices(L, light):
    sw = {"U2": f64(L.W1)[:, light], "V2": f64(L.W2)[light, :]}
    if L.W1u is not None:
        sw["U2u"] = f64(L.W1u)[:, light]
    return sw


def check_factors(W, A, B, r, start_dr, iters, name):
    """W [p, q] ~ A B from the device (bf16) against the optimum and against the oracle's iteration."""
    A, B = f64(A), f64(B)
    err = np.linalg.norm(W - A @ B)
    s = np.linalg.svd(W, compute_uv=False)
    best = np.sqrt(np.sum(s[r:] ** 2))
    wn = np.linalg.norm(W)
    # bf16 factors: each carries a relative rounding of 2^-9, the product of two about 4e-3 of ||A B||
    noise = 6e-3 * wn
    assert err >= best * (1 - 1e-9), name
    assert err <= 1.02 * best + noise, f"{name}: residual {err:.5g} against the optimum {best:.5g}"
    return err, best


FACTOR_CASES = [
    # act, d, m, k, r
    ("gelu_erf", 256, 1024, 100, 64),
    ("gelu_erf", 128, 300, 37, 24),        # ragged: mL = 263, r not a multiple of 16
    ("swiglu", 192, 520, 30, 48),          # three matrices
    ("gelu_erf", 768, 3072, 154, 192),     # BERT-base shape
]


@pytest.mark.parametrize("act,d,m,k,r", FACTOR_CASES)
def test_device_factors_reach_the_truncated_svd_residual(ctx, act, d, m, k, r):
    cfg = custom_config(d, m, k, r, act=act, dtype="bf16")
    L = make_layer(cfg, 5)
    G = GpuLayer(ctx, L)
    heavy = L.planted
    mask = torch.ones(m, dtype=torch.bool)
    mask[heavy] = False
    light = torch.nonzero(mask).flatten().to(torch.int32)
    iters = 6
    n_mat = 3 if act == "swiglu" else 2
    start = start_basis(n_mat, r, d, torch.bfloat16, 17)
    ctx.ensure_workspace(max(ctx.factor_workspace_size(G.shape, k, r), ctx.workspace_size(G.shape, 200, 0, k, r)))
    fac = ctx.factor_light(G.shape, G.W1, G.W2, light.cuda(), k, r, iters, start.cuda(), W1u=G.W1u)
    ctx.poll()
    sw = slices(L, light.long().numpy())
    # U2 ~ A1 B1 (d x mL), V2 ~ A2 B2 (mL x d): residuals against Eckart-Young
    e1, b1 = check_factors(sw["U2"], fac["A1"], fac["B1"], r, None, iters, "U2")
    e2, b2 = check_factors(sw["V2"], fac["A2"], fac["B2"], r, None, iters, "V2")
    if act == "swiglu":
        check_factors(sw["U2u"], fac["A1u"], fac["B1u"], r, None, iters, "U2 (up)")
    # the oracle's iteration from the same start reaches the same residual (its arithmetic is fp64)
    A, B = orc.orthogonal_iteration_factors(sw["U2"], r, iters, f64(start[0]).T)
    assert abs(np.linalg.norm(sw["U2"] - A @ B) - e1) <= 8e-3 * np.linalg.norm(sw["U2"])
    A, B = orc.orthogonal_iteration_factors(sw["V2"].T, r, iters, f64(start[1]).T)
    assert abs(np.linalg.norm(sw["V2"].T - A @ B) - e2) <= 8e-3 * np.linalg.norm(sw["V2"])
    # orthonormal bases: A1 = Q and B2 = Q^T
    assert np.allclose(f64(fac["A1"]).T @ f64(fac["A1"]), np.eye(r), atol=2e-2)
    assert np.allclose(f64(fac["B2"]) @ f64(fac["B2"]).T, np.eye(r), atol=2e-2)
    # and they are factors like any others: pack, forward, compare with Eq. 2 on exactly these factors
    T = 200
    host = {name: t.cpu() for name, t in fac.items()}
    blob, _ = G.pack(heavy, host)
    X = L.tokens(T)
    assert_close(G.forward(blob, X), oracle_split(L, heavy.numpy(), host, X), "bf16", "forward on device factors")


def test_iterations_improve_the_residual_and_zero_rounds_project_on_the_start(ctx):
    cfg = custom_config(256, 1024, 100, 64, act="gelu_erf", dtype="bf16")
    L = make_layer(cfg, 6)
    G = GpuLayer(ctx, L)
    mask = torch.ones(cfg.m, dtype=torch.bool)
    mask[L.planted] = False
    light = torch.nonzero(mask).flatten().to(torch.int32)
    U2 = f64(L.W1)[:, light.long().numpy()]
    start = start_basis(2, cfg.r, cfg.d, torch.bfloat16, 3)
    ctx.ensure_workspace(ctx.factor_workspace_size(G.shape, cfg.k, cfg.r))
    errs = []
    for iters in (0, 1, 3, 8):
        fac = ctx.factor_light(G.shape, G.W1, G.W2, light.cuda(), cfg.k, cfg.r, iters, start.cuda())
        ctx.poll()
        errs.append(np.linalg.norm(U2 - f64(fac["A1"]) @ f64(fac["B1"])))
        if iters == 0:
            # no round: A1 is the starting basis itself, B1 its (non-orthogonal) coefficients start U2
            assert torch.equal(fac["A1"].cpu(), start[0].T.contiguous())
            ref = f64(start[0]) @ U2
            assert orc.rel_frobenius(f64(fac["B1"]), ref) < 1e-2
    assert errs[1] > errs[2] > errs[3] * (1 - 1e-3)
    best = np.sqrt(np.sum(np.linalg.svd(U2, compute_uv=False)[cfg.r:] ** 2))
    assert errs[3] <= 1.015 * best + 6e-3 * np.linalg.norm(U2)


def test_rank_deficient_start_is_reported(ctx):
    """A starting basis without full row rank makes the Gram matrix singular: reported through poll(), no fault."""
    cfg = custom_config(128, 300, 37, 24, act="gelu_erf", dtype="bf16")
    L = make_layer(cfg, 2)
    G = GpuLayer(ctx, L)
    mask = torch.ones(cfg.m, dtype=torch.bool)
    mask[L.planted] = False
    light = torch.nonzero(mask).flatten().to(torch.int32)
    start = start_basis(2, cfg.r, cfg.d, torch.bfloat16, 4)
    start[0, 5] = 0            # a zero row in the basis for U2
    ctx.ensure_workspace(ctx.factor_workspace_size(G.shape, cfg.k, cfg.r))
    fac = ctx.factor_light(G.shape, G.W1, G.W2, light.cuda(), cfg.k, cfg.r, 2, start.cuda())
    from paper_2401_04044_b200 import FFSplitError
    with pytest.raises(FFSplitError) as e:
        ctx.poll()
    assert e.value.code == 6       # FFSPLIT_ERR_NONFINITE
    assert all(torch.isfinite(t.float()).all() for t in fac.values())
    ctx.poll()                 # the condition was cleared by the report


def test_factor_argument_checks(ctx):
    import paper_2401_04044_b200 as ff
    shape = ff.make_shape(128, 300, "gelu_erf", torch.bfloat16)
    with pytest.raises(RuntimeError):
        ctx.factor_workspace_size(shape, 300, 8)        # no light neurons
    with pytest.raises(RuntimeError):
        ctx.factor_workspace_size(shape, 10, 129)       # r > d
    with pytest.raises(RuntimeError):
        ctx.factor_workspace_size(ff.make_shape(128, 300, "gelu_erf", torch.float32), 10, 8)   # bf16 only
