"""ffsplit_forward_noalloc: the decode-size forward for callers that cannot allocate device memory
(a serving loop whose host application owns all of HBM, a plug-in inside another runtime's step).
The entry point keeps its scratch in an array built into the library, so this test gives the
context it calls through NO workspace at all, and checks the result against ffsplit_forward()
-- the same kernels fed from a caller-owned workspace -- on two calls in a row (the second call
finds the first call's leftovers in the shared array).  Collected last on purpose."""
import pytest
import torch

from ffsplit_synth import custom_config, make_layer
from helpers import GpuLayer, assert_close, oracle_factors, oracle_split

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("act,d,m,k,r", [("gelu_erf", 1024, 4096, 205, 256), ("swiglu", 512, 1400, 70, 128)])
def test_noalloc_forward_equals_workspace_forward(act, d, m, k, r):
    from paper_2401_04044_b200 import Context, FFSplitError, build
    build.build()
    cfg = custom_config(d, m, k, r, act=act, dtype="bf16")
    L = make_layer(cfg, 11)
    ctx = Context(0)              # has a workspace: packs the layer and gives the reference output
    bare = Context(0)             # never given a workspace: only the no-alloc entry point can run on it
    try:
        G = GpuLayer(ctx, L)
        G.reserve(8, 0, k, r)
        fac = oracle_factors(L, L.planted.numpy(), r)
        blob, _ = G.pack(L.planted, fac)
        X = L.tokens(8).cuda()
        # a blob packed on another context has to be registered first
        with pytest.raises(FFSplitError) as e:
            bare.forward_noalloc(blob, X, torch.empty_like(X))
        assert e.value.code == 7
        bare.blob_open(blob)
        for T in (8, 3, 1):       # calls in a row, each with fewer tokens than the one before
            X = L.tokens(T)
            want = G.forward(blob, X)
            Xd = X.cuda()
            got = torch.full_like(Xd, float("nan"))
            bare.forward_noalloc(blob, Xd, got)
            bare.poll()           # works without a workspace; nothing to report
            assert torch.equal(got, want), "no-alloc forward differs from the workspace forward"
            assert_close(got, oracle_split(L, L.planted.numpy(), fac, X), "bf16", "no-alloc forward vs oracle")
        # beyond the built-in scratch: more than 8 tokens is refused, nothing is launched
        n0 = bare.launch_count()
        X = L.tokens(9).cuda()
        with pytest.raises(FFSplitError) as e:
            bare.forward_noalloc(blob, X, torch.empty_like(X))
        assert e.value.code == 2 and bare.launch_count() == n0
        # and the ordinary entry point does need a workspace on that context
        with pytest.raises(FFSplitError) as e:
            bare.forward(blob, X, torch.empty_like(X))
        assert e.value.code == 5
    finally:
        ctx.close()
        bare.close()


def test_noalloc_dense_blob_refusals_and_second_context(monkeypatch):
    """A dense (k = m) blob through the built-in scratch; the documented refusals (fp32 layer, a layer whose
    intermediates exceed the built-in 2 MiB) launch nothing; a second bare context, in the single-launch mode
    whose barrier words live in the shared array, finds the array as the first one left it."""
    from paper_2401_04044_b200 import Context, FFSplitError, build
    build.build()
    ctx, bare = Context(0), Context(0)
    monkeypatch.setenv("FFSPLIT_DECODE_LAYER", "1")
    bare2 = Context(0)
    try:
        cfg = custom_config(256, 1024, 16, 16, act="gelu_erf", dtype="bf16")
        L = make_layer(cfg, 12)
        G = GpuLayer(ctx, L)
        G.reserve(8, 0, cfg.m, 0)
        G.reserve(8, 0, cfg.k, cfg.r)
        blob, _ = G.pack(torch.arange(cfg.m), None)
        fac = oracle_factors(L, L.planted.numpy(), cfg.r)
        blob_s, _ = G.pack(L.planted, fac)
        for c in (bare, bare2):
            c.blob_open(blob)
            c.blob_open(blob_s)
        for T in (1, 5):
            Xd = L.tokens(T).cuda()
            want = torch.empty_like(Xd)
            ctx.forward(blob, Xd, want)
            ctx.poll()
            for c in (bare, bare2, bare):
                got = torch.full_like(Xd, float("nan"))
                c.forward_noalloc(blob, Xd, got)
                c.poll()
                assert torch.equal(got, want)
            want_s = torch.empty_like(Xd)
            ctx.forward(blob_s, Xd, want_s)
            ctx.poll()
            got = torch.full_like(Xd, float("nan"))
            bare2.forward_noalloc(blob_s, Xd, got)
            bare2.poll()
            assert torch.equal(got, want_s)
        # fp32 layers are refused
        cfg32 = custom_config(64, 256, 16, 16, act="gelu_erf", dtype="f32")
        L32 = make_layer(cfg32, 12)
        G32 = GpuLayer(ctx, L32)
        G32.reserve(8, 0, 16, 0)
        blob32, _ = G32.pack(L32.planted, None)
        bare.blob_open(blob32)
        n0 = bare.launch_count()
        X32 = L32.tokens(2).cuda()
        with pytest.raises(FFSplitError) as e:
            bare.forward_noalloc(blob32, X32, torch.empty_like(X32))
        assert e.value.code == 4 and bare.launch_count() == n0
        # a layer too wide for the built-in intermediates: 8 tokens x (mL_pad + ...) x 2 bytes > 2 MiB
        wide = custom_config(64, 140000, 16, 16, act="gelu_erf", dtype="bf16")
        Lw = make_layer(wide, 12)
        Gw = GpuLayer(ctx, Lw)
        Gw.reserve(8, 0, 16, 16)
        g = torch.Generator().manual_seed(3)
        mk = lambda *s: (torch.randn(*s, generator=g) * 0.02).to(torch.bfloat16)
        facw = {"A1": mk(64, 16), "B1": mk(16, wide.m - 16), "A2": mk(wide.m - 16, 16), "B2": mk(16, 64)}
        blobw, _ = Gw.pack(Lw.planted, facw)
        bare.blob_open(blobw)
        Xw = Lw.tokens(8).cuda()
        with pytest.raises(FFSplitError) as e:
            bare.forward_noalloc(blobw, Xw, torch.empty_like(Xw))
        assert e.value.code == 5 and bare.launch_count() == n0
    finally:
        ctx.close()
        bare.close()
        bare2.close()
