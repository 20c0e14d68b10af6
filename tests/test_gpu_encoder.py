"""The transformer block around the FFN (Section 5.1.2 / Table 2: whole BERT-base layers) against the oracle:
attention, the two LayerNorms and the packed FFN (split and dense) through `ffsplit_encoder_forward`."""
import numpy as np
import pytest
import torch

from conftest import f64
from ffsplit_synth import custom_config, make_layer
from helpers import GpuLayer, oracle_factors
from oracle import ffsplit_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2401_04044_b200 import Context, build
    build.build()
    c = Context(0)
    yield c
    c.close()


def block_weights(d, seed):
    """Seeded attention and LayerNorm parameters in the oracle's layout, rounded to what the device stores."""
    g = torch.Generator().manual_seed(seed)
    rn = lambda *s, std=1.0: torch.randn(*s, generator=g) * std
    w = {"Wqkv": rn(d, 3 * d, std=0.05).to(torch.bfloat16), "bqkv": rn(3 * d, std=0.02),
         "Wo": rn(d, d, std=0.05).to(torch.bfloat16), "bo": rn(d, std=0.02),
         "g1": 1 + rn(d, std=0.1), "b1": rn(d, std=0.05), "g2": 1 + rn(d, std=0.1), "b2": rn(d, std=0.05)}
    return w


def run_block(ctx, G, w, blob, X, batch, seq, heads, eps):
    dev = lambda t: t.cuda().contiguous()
    keep = {"Wqkv_t": dev(w["Wqkv"].T), "bqkv": dev(w["bqkv"]), "Wo_t": dev(w["Wo"].T), "bo": dev(w["bo"]),
            "g1": dev(w["g1"]), "b1": dev(w["b1"]), "g2": dev(w["g2"]), "b2": dev(w["b2"])}
    desc = ctx.encoder_desc(batch, seq, heads, keep["Wqkv_t"], keep["bqkv"], keep["Wo_t"], keep["bo"],
                            (keep["g1"], keep["b1"]), (keep["g2"], keep["b2"]), eps, blob)
    ctx.ensure_workspace(ctx.encoder_workspace_size(desc))
    Xd = X.cuda()
    Y = torch.empty_like(Xd)
    ctx.encoder_forward(desc, Xd, Y)
    ctx.poll()
    Y2 = torch.empty_like(Xd)
    ctx.encoder_forward(desc, Xd, Y2)
    ctx.poll()
    assert torch.equal(Y, Y2), "the block is not bitwise reproducible"
    return Y


def oracle_block(L, w, X, batch, seq, heads, eps, heavy, fac):
    attn = (f64(w["Wqkv"]), f64(w["bqkv"]), f64(w["Wo"]), f64(w["bo"]))
    if fac is None:
        ffn = lambda Z: orc.dense_ffn(Z, f64(L.W1), f64(L.b1), f64(L.W2), f64(L.b2), L.cfg.act)
    else:
        facd = {k: f64(v) for k, v in fac.items()}
        ffn = lambda Z: orc.split_ffn(Z, f64(L.W1), f64(L.b1), f64(L.W2), f64(L.b2), heavy, facd, L.cfg.act)
    return orc.encoder_layer(f64(X), attn, (f64(w["g1"]), f64(w["b1"])), (f64(w["g2"]), f64(w["b2"])), eps, batch, seq,
                             heads, ffn)


BLOCK_CASES = [
    # heads, m, k, r, batch, seq
    (2, 512, 26, 32, 3, 128),       # d = 128: the smallest width, full tiles
    (4, 1024, 52, 64, 2, 77),       # ragged sequences: keys past 77 masked, the next sequence's rows in the tile
    (12, 3072, 154, 192, 4, 128),   # BERT-base width
    (3, 600, 30, 48, 5, 1),         # one token per sequence: attention is the identity on V
]


@pytest.mark.parametrize("heads,m,k,r,batch,seq", BLOCK_CASES)
@pytest.mark.parametrize("split", [True, False], ids=["split_ffn", "dense_ffn"])
def test_encoder_block_matches_oracle(ctx, heads, m, k, r, batch, seq, split):
    d = 64 * heads
    cfg = custom_config(d, m, k, r, act="gelu_erf", dtype="bf16")
    L = make_layer(cfg, 9)
    G = GpuLayer(ctx, L)
    T = batch * seq
    G.reserve(T, 0, k, r)
    G.reserve(T, 0, m, 0)
    if split:
        heavy = L.planted
        fac = oracle_factors(L, heavy.numpy(), r)
        blob, _ = G.pack(heavy, fac)
    else:
        heavy, fac = None, None
        blob, _ = G.pack(torch.arange(m), None)
    w = block_weights(d, 100 + heads)
    g = torch.Generator().manual_seed(5)
    X = torch.randn(T, d, generator=g).to(torch.bfloat16)
    eps = 1e-12
    Y = run_block(ctx, G, w, blob, X, batch, seq, heads, eps)
    ref = oracle_block(L, w, X, batch, seq, heads, eps, None if heavy is None else heavy.numpy(), fac)
    # the block's output is a LayerNorm: entries of order one; bf16 intermediates (projections, P, attention output,
    # X1, the FFN) each carry 2^-9 relative rounding
    err = orc.rel_frobenius(f64(Y), ref)
    mx = np.abs(f64(Y) - ref).max()
    assert err < 1.5e-2 and mx < 0.15, f"rel-Frobenius {err:.3e}, max-abs {mx:.3e}"


def test_attention_alone_through_the_block(ctx):
    """With LayerNorm gains that kill the FFN branch's visibility impossible to build, test attention directly: zero
    FFN weights and unit LayerNorms leave Y = LN(LN(X + A)), so an error in A shows at full size."""
    heads, batch, seq = 4, 3, 100
    d, m = 64 * heads, 256
    cfg = custom_config(d, m, 16, 16, act="gelu_erf", dtype="bf16")
    L = make_layer(cfg, 1)
    L.W2.zero_()
    L.b2.zero_()
    G = GpuLayer(ctx, L)
    T = batch * seq
    G.reserve(T, 0, m, 0)
    blob, _ = G.pack(torch.arange(m), None)
    w = block_weights(d, 7)
    w["Wqkv"] = (w["Wqkv"].float() * 6).to(torch.bfloat16)      # sharper softmax rows
    for n in ("g1", "g2"):
        w[n] = torch.ones(d)
    for n in ("b1", "b2"):
        w[n] = torch.zeros(d)
    g = torch.Generator().manual_seed(8)
    X = (torch.randn(T, d, generator=g) * 0.3).to(torch.bfloat16)
    Y = run_block(ctx, G, w, blob, X, batch, seq, heads, 1e-12)
    ref = oracle_block(L, w, X, batch, seq, heads, 1e-12, None, None)
    assert orc.rel_frobenius(f64(Y), ref) < 1.5e-2


def test_encoder_argument_checks(ctx):
    from paper_2401_04044_b200 import FFSplitError
    d = 128
    cfg = custom_config(d, 256, 16, 16, act="gelu_erf", dtype="bf16")
    L = make_layer(cfg, 2)
    G = GpuLayer(ctx, L)
    G.reserve(256, 0, 256, 0)
    blob, _ = G.pack(torch.arange(256), None)
    w = block_weights(d, 3)
    dev = lambda t: t.cuda().contiguous()
    args = (dev(w["Wqkv"].T), dev(w["bqkv"]), dev(w["Wo"].T), dev(w["bo"]), (dev(w["g1"]), dev(w["b1"])),
            (dev(w["g2"]), dev(w["b2"])), 1e-12)
    with pytest.raises(FFSplitError):
        ctx.encoder_workspace_size(ctx.encoder_desc(2, 129, 2, *args, blob))     # sequence longer than a tile
    with pytest.raises(FFSplitError):
        ctx.encoder_workspace_size(ctx.encoder_desc(2, 64, 2, *args, torch.empty(1024, dtype=torch.uint8, device="cuda")))  # unknown blob
