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
        for T in (8, 3):          # two calls in a row, the second with fewer tokens than the first
            X = L.tokens(T)
            want = G.forward(blob, X)
            Xd = X.cuda()
            got = torch.full_like(Xd, float("nan"))
            bare.forward_noalloc(blob, Xd, got)
            torch.cuda.synchronize()
            assert torch.equal(got, want), "no-alloc forward differs from the workspace forward"
            assert_close(got, oracle_split(L, L.planted.numpy(), fac, X), "bf16", "no-alloc forward vs oracle")
        # beyond the built-in scratch: more than 8 tokens is refused, nothing is launched
        X = L.tokens(9).cuda()
        with pytest.raises(FFSplitError) as e:
            bare.forward_noalloc(blob, X, torch.empty_like(X))
        assert e.value.code == 2
        # and the ordinary entry point does need a workspace on that context
        with pytest.raises(FFSplitError) as e:
            bare.forward(blob, X, torch.empty_like(X))
        assert e.value.code == 5
    finally:
        ctx.close()
        bare.close()
