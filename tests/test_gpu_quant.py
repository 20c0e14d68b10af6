"""Quantised split (Section 5.2: heavy-hitter neurons 8 bits, everything else 3 bits, round to nearest, group size
128) against the oracle: the packed codes and group parameters bit for bit, the few-token forward element by
element against Eq. 2 evaluated in float64 on the oracle's dequantised weights, at the bf16 tolerances."""
import numpy as np
import pytest
import torch

from conftest import f64
from ffsplit_synth import CONFIGS, cfg5_point, custom_config, make_layer
from helpers import GpuLayer, assert_close
from oracle import ffsplit_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2401_04044_b200 import Context, build
    build.build()
    c = Context(0)
    c.ensure_workspace(1 << 20)
    yield c
    c.close()


def light_of(m, heavy):
    mask = torch.ones(m, dtype=torch.bool)
    mask[heavy] = False
    return torch.nonzero(mask).flatten()


def quant_pack(ctx, G, L, heavy):
    cfg = L.cfg
    k = int(heavy.numel())
    ctx.ensure_workspace(ctx.quant_workspace_size(G.shape, k))
    padded, logical = ctx.quant_pack_size(G.shape, k)
    blob = torch.empty(padded, dtype=torch.uint8, device="cuda")
    light = light_of(cfg.m, heavy)
    ctx.quant_pack(G.shape, G.W1, G.b1, G.W2, G.b2, heavy.to(torch.int32).cuda(), k, light.to(torch.int32).cuda(), blob,
                   W1u=G.W1u)
    ctx.poll()
    return blob, logical


QUANT_CASES = [
    # act, d, m, k      (d and the part sizes around and across group and double-group boundaries)
    ("gelu_erf", 256, 1024, 52),
    ("gelu_erf", 72, 300, 37),         # one ragged group everywhere
    ("gelu_tanh", 384, 700, 130),      # 3 groups along d (padded to 4), heavy part just over one group
    ("swiglu", 256, 520, 40),
    ("gelu_erf", 1024, 4096, 205),     # GPT-2-medium shape
    ("gelu_erf", 128, 512, 0),         # no heavy neurons: all 3 bits
    ("gelu_erf", 128, 300, 300),       # every neuron heavy: all 8 bits
]


@pytest.mark.parametrize("act,d,m,k", QUANT_CASES)
def test_quant_pack_codes_and_parameters_are_bit_exact(ctx, act, d, m, k):
    cfg = custom_config(d, m, k, 0, act=act, dtype="bf16")
    L = make_layer(cfg, 4)
    G = GpuLayer(ctx, L)
    heavy = L.planted
    blob, logical = quant_pack(ctx, G, L, heavy)
    Q = orc.quantize_split(f64(L.W1).astype(np.float32), f64(L.W2).astype(np.float32), heavy.numpy(),
                           W1u=None if L.W1u is None else f64(L.W1u).astype(np.float32))
    ml = m - k
    names = [("U1", 0, k, d), ("U2", 1, ml, d), ("V1", 4, d, k), ("V2", 5, d, ml)]
    if act == "swiglu":
        names += [("U1u", 2, k, d), ("U2u", 3, ml, d)]
    for name, which, rows, cols in names:
        if rows == 0 or cols == 0:
            continue
        codes, scale, lo = ctx.quant_unpack(blob, which, rows, cols)
        ctx.poll()
        qc, qs, ql = Q[name]
        assert np.array_equal(codes.cpu().numpy(), qc), f"{name}: codes differ from the oracle"
        assert np.array_equal(scale.cpu().numpy(), qs) and np.array_equal(lo.cpu().numpy(), ql), f"{name}: parameters differ"
    n_in = 2 if act == "swiglu" else 1
    assert logical == orc.quant_weight_bytes(d, m, k, n_in=n_in) + 4 * (m + d)


@pytest.mark.parametrize("act,d,m,k", QUANT_CASES)
@pytest.mark.parametrize("T", [1, 3, 8, 13])
def test_quant_forward_matches_oracle(ctx, act, d, m, k, T):
    cfg = custom_config(d, m, k, 0, act=act, dtype="bf16")
    L = make_layer(cfg, 4)
    G = GpuLayer(ctx, L)
    heavy = L.planted
    blob, _ = quant_pack(ctx, G, L, heavy)
    Q = orc.quantize_split(f64(L.W1).astype(np.float32), f64(L.W2).astype(np.float32), heavy.numpy(),
                           W1u=None if L.W1u is None else f64(L.W1u).astype(np.float32))
    X = L.tokens(T)
    Xd = X.cuda()
    Y = torch.full_like(Xd, float("nan"))
    ctx.quant_forward(blob, Xd, Y)
    ctx.poll()
    ref = orc.quant_split_ffn(f64(X), f64(L.b1), f64(L.b2), Q, d, m, act)
    assert_close(Y, ref, "bf16", f"quantised forward T={T}")
    Y2 = torch.empty_like(Xd)
    ctx.quant_forward(blob, Xd, Y2)
    ctx.poll()
    assert torch.equal(Y, Y2), "quantised forward is not bitwise reproducible"


def test_quant_blob_registry(ctx):
    from paper_2401_04044_b200 import Context, FFSplitError
    cfg = custom_config(128, 512, 26, 0, dtype="bf16")
    L = make_layer(cfg, 5)
    G = GpuLayer(ctx, L)
    blob, _ = quant_pack(ctx, G, L, L.planted)
    Xd = L.tokens(2).cuda()
    Y = torch.empty_like(Xd)
    ctx.quant_forward(blob, Xd, Y)
    ctx.poll()
    c2 = Context(0)
    try:
        c2.ensure_workspace(c2.quant_workspace_size(G.shape, cfg.k))
        with pytest.raises(FFSplitError) as e:
            c2.quant_forward(blob, Xd, torch.empty_like(Xd))
        assert e.value.code == 7
        copy = blob.clone()
        c2.quant_blob_open(copy)
        Y2 = torch.empty_like(Xd)
        c2.quant_forward(copy, Xd, Y2)
        c2.poll()
        assert torch.equal(Y2, Y)
        with pytest.raises(FFSplitError) as e:
            c2.quant_blob_open(torch.zeros(4096, dtype=torch.uint8, device="cuda"))
        assert e.value.code == 7
        # a bf16 blob is not a quantised one, and fp32 layers are refused
        with pytest.raises(FFSplitError) as e:
            c2.quant_pack_size(c2_shape_f32(), 4)
        assert e.value.code == 4
    finally:
        c2.close()


def c2_shape_f32():
    from paper_2401_04044_b200 import make_shape
    return make_shape(64, 256, "gelu_erf", torch.float32)


@pytest.mark.parametrize("name,cfg,tokens", [("opt_13b_5pct", cfg5_point(5, 512), (1, 8)), ("llama2_7b", CONFIGS[4], (1,))])
def test_quant_full_size_layer(ctx, name, cfg, tokens):
    """The OPT-13B- and Llama-2-7B-shaped layers at full size: sampled packed rows bit for bit, the forward on every
    output element against the oracle's dequantised weights."""
    L = make_layer(cfg, 0)
    G = GpuLayer(ctx, L)
    heavy = L.planted
    blob, logical = quant_pack(ctx, G, L, heavy)
    W1, W2 = f64(L.W1).astype(np.float32), f64(L.W2).astype(np.float32)
    W1u = None if L.W1u is None else f64(L.W1u).astype(np.float32)
    Q = orc.quantize_split(W1, W2, heavy.numpy(), W1u=W1u)
    d, m, k = cfg.d, cfg.m, cfg.k
    assert logical == orc.quant_weight_bytes(d, m, k, n_in=cfg.n_in) + 4 * (m + d)
    for nm, which, rows, cols in (("U2", 1, m - k, d), ("V1", 4, d, k)):
        codes, scale, lo = ctx.quant_unpack(blob, which, rows, cols)
        ctx.poll()
        pick = np.arange(0, rows, 97)
        assert np.array_equal(codes.cpu().numpy()[pick], Q[nm][0][pick])
        assert np.array_equal(scale.cpu().numpy()[pick], Q[nm][1][pick]) and np.array_equal(lo.cpu().numpy()[pick], Q[nm][2][pick])
    for T in tokens:
        X = L.tokens(T)
        Xd = X.cuda()
        Y = torch.empty_like(Xd)
        ctx.quant_forward(blob, Xd, Y)
        ctx.poll()
        assert_close(Y, orc.quant_split_ffn(f64(X), f64(L.b1), f64(L.b2), Q, d, m, cfg.act), "bf16", f"{name} quantised T={T}")
