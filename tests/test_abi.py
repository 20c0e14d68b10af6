"""Host-only checks of the C-ABI library: it builds, loads and exports every
symbol the header declares; size queries and argument errors need no GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2401_04044_b200 import build, binding
    build.build()
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ffsplit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ffsplit_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    from paper_2401_04044_b200 import binding
    names = declared_symbols()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), f"{n} declared in ffsplit.h but not exported"
    assert sorted(binding.EXPORTS) == names
    assert lib.ffsplit_version() >= 100


def test_pack_size_matches_closed_form(lib):
    from paper_2401_04044_b200 import binding as b
    for (d, m, k, r, act, dt, es) in [(768, 3072, 154, 192, b.GELU_ERF, b.BF16, 2), (256, 1024, 32, 64, b.GELU_ERF, b.F32, 4),
                                      (4096, 11008, 551, 1024, b.SWIGLU, b.BF16, 2), (64, 256, 256, 0, b.GELU_TANH, b.F32, 4)]:
        shape = b.Shape(d, m, act, dt)
        padded, logical = C.c_size_t(), C.c_size_t()
        assert lib.ffsplit_pack_size(C.byref(shape), k, r, C.byref(padded), C.byref(logical)) == 0
        n_in = 2 if act == b.SWIGLU else 1
        params = (n_in + 1) * (d * k + r * (d + m - k))
        assert logical.value == es * (params + m + d)
        assert padded.value >= logical.value - es * (m + d) and padded.value % 256 == 0
        assert padded.value < 1.15 * logical.value + 65536


def test_host_side_argument_errors(lib):
    from paper_2401_04044_b200 import binding as b
    n = C.c_size_t()
    bad = b.Shape(100, 64, b.GELU_ERF, b.BF16)             # bf16 needs d % 8 == 0
    assert lib.ffsplit_pack_size(C.byref(bad), 8, 8, C.byref(n), None) == 2
    ok = b.Shape(64, 256, b.GELU_ERF, b.BF16)
    assert lib.ffsplit_pack_size(C.byref(ok), 257, 0, C.byref(n), None) == 2      # k > m
    assert lib.ffsplit_pack_size(C.byref(ok), 250, 7, C.byref(n), None) == 2      # r > m - k
    assert lib.ffsplit_pack_size(C.byref(ok), 8, 65, C.byref(n), None) == 2       # r > d
    assert lib.ffsplit_workspace_size(C.byref(ok), 128, 256, 8, 16, C.byref(n)) == 0 and n.value >= 65536
    assert lib.ffsplit_workspace_size(C.byref(ok), 0, 0, 8, 16, C.byref(n)) == 0 and n.value == 65536
    assert lib.ffsplit_workspace_size(C.byref(b.Shape(64, 256, 7, b.BF16)), 1, 1, 8, 16, C.byref(n)) == 1
    assert lib.ffsplit_workspace_size(C.byref(b.Shape(64, 256, 0, 5)), 1, 1, 8, 16, C.byref(n)) == 4
    assert lib.ffsplit_last_error(None) == b"no context"


def test_create_without_a_gpu_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    h = C.c_void_p()
    assert lib.ffsplit_create(C.byref(h), 0) != 0 and not h.value


def test_missing_library_is_an_error(tmp_path):
    from paper_2401_04044_b200 import binding
    with pytest.raises(FileNotFoundError):
        binding.load_library(str(tmp_path / "nope.so"))
