"""ctypes binding of libffsplit (include/ffsplit.h).

Argument marshalling only: every step of the path (scoring, selection, packing,
forward) runs in the library's CUDA kernels.  torch is used for device memory
and streams.  There is no CPU fallback: loading fails loudly when the shared
library has not been built, and every call raises on a non-zero status.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libffsplit.so")

OK = 0
ERR_NAMES = {
    1: "INVALID_ARG", 2: "SHAPE", 3: "ALIGN", 4: "DTYPE", 5: "BUFFER_TOO_SMALL", 6: "NONFINITE",
    7: "BAD_BLOB", 8: "ARCH", 9: "CUDA", 10: "TIMEOUT", 11: "BAD_INDEX",
}
F32, BF16 = 0, 1
GELU_ERF, GELU_TANH, SWIGLU = 0, 1, 2
SCORE_EQ3, SCORE_ACT_ONLY, SCORE_SUM_NORM = 0, 1, 2
ACT_IDS = {"gelu_erf": GELU_ERF, "gelu_tanh": GELU_TANH, "swiglu": SWIGLU}
DTYPE_IDS = {torch.float32: F32, torch.bfloat16: BF16}
SCORE_IDS = {"eq3": SCORE_EQ3, "act_only": SCORE_ACT_ONLY, "sum_norm": SCORE_SUM_NORM}

EXPORTS = [
    "ffsplit_create", "ffsplit_destroy", "ffsplit_workspace_size", "ffsplit_set_workspace", "ffsplit_score",
    "ffsplit_select", "ffsplit_pack_size", "ffsplit_pack", "ffsplit_blob_open", "ffsplit_blob_section",
    "ffsplit_forward", "ffsplit_forward_host", "ffsplit_poll", "ffsplit_launch_count", "ffsplit_last_error",
    "ffsplit_version", "ffsplit_profile_begin", "ffsplit_profile_end", "ffsplit_forward_noalloc",
    "ffsplit_forward_dense", "ffsplit_score_activations", "ffsplit_score_host", "ffsplit_score_finalize",
    "ffsplit_blob_close", "ffsplit_stack_workspace_size", "ffsplit_forward_stack", "ffsplit_forward_stack_host",
    "ffsplit_debug_wait_timeout", "ffsplit_quant_pack_size", "ffsplit_quant_workspace_size", "ffsplit_quant_pack",
    "ffsplit_quant_blob_open", "ffsplit_quant_unpack", "ffsplit_quant_forward",
    "ffsplit_factor_workspace_size", "ffsplit_factor_light", "ffsplit_encoder_workspace_size", "ffsplit_encoder_forward",
]


class EncoderLayer(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq", C.c_int32), ("heads", C.c_int32), ("Wqkv_t", C.c_void_p), ("bqkv", C.c_void_p),
                ("Wo_t", C.c_void_p), ("bo", C.c_void_p), ("ln1_gamma", C.c_void_p), ("ln1_beta", C.c_void_p),
                ("ln2_gamma", C.c_void_p), ("ln2_beta", C.c_void_p), ("ln_eps", C.c_float), ("ffn_blob", C.c_void_p)]


class Shape(C.Structure):
    _fields_ = [("d", C.c_int32), ("m", C.c_int32), ("act", C.c_int32), ("dtype", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [("W1", C.c_void_p), ("W1u", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p), ("b2", C.c_void_p)]


class Factors(C.Structure):
    _fields_ = [("A1", C.c_void_p), ("B1", C.c_void_p), ("A1u", C.c_void_p), ("B1u", C.c_void_p),
                ("A2", C.c_void_p), ("B2", C.c_void_p), ("r", C.c_int32)]


class FFSplitError(RuntimeError):
    def __init__(self, code: int, where: str, text: str = ""):
        self.code = code
        super().__init__(f"{where}: FFSPLIT_ERR_{ERR_NAMES.get(code, code)} {text}".strip())


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Load libffsplit.so (built in-tree by paper_2401_04044_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(
            f"{p} not found: build it with `python -m paper_2401_04044_b200.build` (there is no fallback path)")
    lib = C.CDLL(p)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    P = C.POINTER
    lib.ffsplit_create.argtypes = [P(vp), C.c_int]
    lib.ffsplit_destroy.argtypes = [vp]
    lib.ffsplit_workspace_size.argtypes = [P(Shape), i64, i64, i32, i32, P(sz)]
    lib.ffsplit_set_workspace.argtypes = [vp, vp, sz]
    lib.ffsplit_score.argtypes = [vp, P(Shape), P(Weights), vp, i64, i32, i32, vp, vp, vp]
    lib.ffsplit_select.argtypes = [vp, vp, i32, i32, vp, vp, vp]
    lib.ffsplit_pack_size.argtypes = [P(Shape), i32, i32, P(sz), P(sz)]
    lib.ffsplit_pack.argtypes = [vp, P(Shape), P(Weights), vp, i32, P(Factors), vp, sz, vp]
    lib.ffsplit_blob_open.argtypes = [vp, vp, sz, vp]
    lib.ffsplit_blob_close.argtypes = [vp, vp]
    lib.ffsplit_score_host.argtypes = [vp, P(Shape), P(Weights), vp, i64, i32, i32, vp, vp, vp]
    lib.ffsplit_score_finalize.argtypes = [vp, P(Shape), vp, i32, vp, vp, vp]
    lib.ffsplit_score_activations.argtypes = [vp, P(Shape), vp, i64, vp, i32, i32, vp, vp, vp]
    lib.ffsplit_forward_dense.argtypes = [vp, P(Shape), P(Weights), vp, i64, vp, vp]
    lib.ffsplit_stack_workspace_size.argtypes = [vp, P(vp), i32, i64, P(sz)]
    lib.ffsplit_forward_stack.argtypes = [vp, P(vp), i32, vp, i64, vp, vp]
    lib.ffsplit_forward_stack_host.argtypes = [vp, P(vp), i32, vp, i64, vp, vp]
    lib.ffsplit_debug_wait_timeout.argtypes = [vp, i64, vp]
    lib.ffsplit_quant_pack_size.argtypes = [P(Shape), i32, P(sz), P(sz)]
    lib.ffsplit_quant_workspace_size.argtypes = [P(Shape), i32, P(sz)]
    lib.ffsplit_quant_pack.argtypes = [vp, P(Shape), P(Weights), vp, i32, vp, vp, sz, vp]
    lib.ffsplit_quant_blob_open.argtypes = [vp, vp, sz, vp]
    lib.ffsplit_quant_unpack.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.ffsplit_quant_forward.argtypes = [vp, vp, vp, i64, vp, vp]
    lib.ffsplit_encoder_workspace_size.argtypes = [vp, vp, P(sz)]
    lib.ffsplit_encoder_forward.argtypes = [vp, vp, vp, vp, vp]
    lib.ffsplit_factor_workspace_size.argtypes = [vp, i32, i32, P(sz)]
    lib.ffsplit_factor_light.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.ffsplit_blob_section.argtypes = [vp, vp, i32, P(sz), P(i64), P(i64), P(i64)]
    lib.ffsplit_forward.argtypes = [vp, vp, vp, i64, vp, vp]
    lib.ffsplit_forward_host.argtypes = [vp, vp, vp, i64, vp, vp]
    lib.ffsplit_forward_noalloc.argtypes = [vp, vp, vp, i64, vp, vp]
    lib.ffsplit_poll.argtypes = [vp, vp]
    lib.ffsplit_profile_begin.argtypes = [vp]
    lib.ffsplit_profile_end.argtypes = [vp, vp, i32, P(i32), P(C.c_double), P(C.c_double)]
    lib.ffsplit_launch_count.argtypes = [vp]
    lib.ffsplit_launch_count.restype = i64
    lib.ffsplit_last_error.argtypes = [vp]
    lib.ffsplit_last_error.restype = C.c_char_p
    lib.ffsplit_version.argtypes = []
    lib.ffsplit_version.restype = i32
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("ffsplit_launch_count", "ffsplit_last_error", "ffsplit_version"):
            fn.restype = C.c_int
    if path is None:
        _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_shape(d: int, m: int, act, dtype) -> Shape:
    a = ACT_IDS[act] if isinstance(act, str) else int(act)
    t = DTYPE_IDS[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return Shape(d, m, a, t)


class Context:
    """One ffsplit_ctx bound to a CUDA device, plus the torch tensors that back
    its workspace.  Methods mirror the C entry points one to one."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        self.device = device
        torch.cuda.set_device(device)
        h = C.c_void_p()
        rc = self.lib.ffsplit_create(C.byref(h), device)
        if rc != OK:
            raise FFSplitError(rc, "ffsplit_create")
        self.h = h
        self._ws = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.ffsplit_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != OK:
            raise FFSplitError(rc, where, (self.lib.ffsplit_last_error(self.h) or b"").decode())

    # ------------------------------------------------------------------ workspace
    def workspace_size(self, shape: Shape, T_fwd: int, T_cal: int, k: int, r: int) -> int:
        n = C.c_size_t()
        self._check(self.lib.ffsplit_workspace_size(C.byref(shape), T_fwd, T_cal, k, r, C.byref(n)),
                    "ffsplit_workspace_size")
        return n.value

    def set_workspace(self, tensor: torch.Tensor):
        self._check(self.lib.ffsplit_set_workspace(self.h, _ptr(tensor), tensor.numel() * tensor.element_size()),
                    "ffsplit_set_workspace")
        self._ws = tensor

    def ensure_workspace(self, nbytes: int):
        """Allocate (with torch) and install a workspace of at least nbytes."""
        have = 0 if self._ws is None else self._ws.numel()
        if have < nbytes:
            self.set_workspace(torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{self.device}"))

    # ------------------------------------------------------------------ entry points
    def score(self, shape: Shape, W1, b1, W2, X, energy, scores=None, mode=SCORE_EQ3, accumulate=False, W1u=None,
              stream=None):
        w = Weights(_ptr(W1), _ptr(W1u), _ptr(b1), _ptr(W2), None)
        self._check(self.lib.ffsplit_score(self.h, C.byref(shape), C.byref(w), _ptr(X), X.shape[0], int(mode),
                                           int(bool(accumulate)), _ptr(energy), _ptr(scores), _stream_ptr(stream)),
                    "ffsplit_score")

    def score_activations(self, shape: Shape, H, W2, energy, scores=None, mode=SCORE_EQ3, accumulate=False,
                          stream=None):
        """ffsplit_score_activations: Eq. 3 from a stored activation matrix H [T, m]."""
        self._check(self.lib.ffsplit_score_activations(self.h, C.byref(shape), _ptr(H), H.shape[0], _ptr(W2), mode,
                                                       1 if accumulate else 0, _ptr(energy), _ptr(scores),
                                                       _stream_ptr(stream)), "ffsplit_score_activations")

    def select(self, scores, k: int, heavy_idx, light_idx=None, stream=None):
        self._check(self.lib.ffsplit_select(self.h, _ptr(scores), scores.numel(), k, _ptr(heavy_idx), _ptr(light_idx),
                                            _stream_ptr(stream)), "ffsplit_select")

    def pack_size(self, shape: Shape, k: int, r: int):
        a, b = C.c_size_t(), C.c_size_t()
        self._check(self.lib.ffsplit_pack_size(C.byref(shape), k, r, C.byref(a), C.byref(b)), "ffsplit_pack_size")
        return a.value, b.value

    def pack(self, shape: Shape, W1, b1, W2, b2, heavy_idx, k: int, factors: Optional[dict], blob, W1u=None,
             stream=None):
        w = Weights(_ptr(W1), _ptr(W1u), _ptr(b1), _ptr(W2), _ptr(b2))
        fp = None
        if factors is not None:
            f = Factors(_ptr(factors["A1"]), _ptr(factors["B1"]), _ptr(factors.get("A1u")), _ptr(factors.get("B1u")),
                        _ptr(factors["A2"]), _ptr(factors["B2"]), int(factors["A1"].shape[1]))
            fp = C.byref(f)
        self._check(self.lib.ffsplit_pack(self.h, C.byref(shape), C.byref(w), _ptr(heavy_idx), k, fp, _ptr(blob),
                                          blob.numel() * blob.element_size(), _stream_ptr(stream)), "ffsplit_pack")

    def blob_open(self, blob, stream=None):
        self._check(self.lib.ffsplit_blob_open(self.h, _ptr(blob), blob.numel() * blob.element_size(),
                                               _stream_ptr(stream)), "ffsplit_blob_open")

    def blob_close(self, blob):
        self._check(self.lib.ffsplit_blob_close(self.h, _ptr(blob)), "ffsplit_blob_close")

    def score_host(self, shape: Shape, W1, b1, W2, X_host, energy, scores=None, mode=SCORE_EQ3, accumulate=False,
                   W1u=None, stream=None):
        """ffsplit_score_host: calibration tokens in (pinned) host memory, staged through the workspace in chunks."""
        w = Weights(_ptr(W1), _ptr(W1u), _ptr(b1), _ptr(W2), None)
        self._check(self.lib.ffsplit_score_host(self.h, C.byref(shape), C.byref(w), _ptr(X_host), X_host.shape[0],
                                                int(mode), int(bool(accumulate)), _ptr(energy), _ptr(scores),
                                                _stream_ptr(stream)), "ffsplit_score_host")

    def score_finalize(self, shape: Shape, W2, energy, scores, mode=SCORE_EQ3, stream=None):
        """ffsplit_score_finalize: scores from a complete energy vector (after a sharded or multi-call accumulation)."""
        self._check(self.lib.ffsplit_score_finalize(self.h, C.byref(shape), _ptr(W2), int(mode), _ptr(energy),
                                                    _ptr(scores), _stream_ptr(stream)), "ffsplit_score_finalize")

    @staticmethod
    def _blob_array(blobs):
        arr = (C.c_void_p * len(blobs))(*[b.data_ptr() for b in blobs])
        return arr

    def stack_workspace_size(self, blobs, T: int) -> int:
        n = C.c_size_t()
        self._check(self.lib.ffsplit_stack_workspace_size(self.h, self._blob_array(blobs), len(blobs), T, C.byref(n)),
                    "ffsplit_stack_workspace_size")
        return n.value

    def forward_stack(self, blobs, X, Y, stream=None):
        self._check(self.lib.ffsplit_forward_stack(self.h, self._blob_array(blobs), len(blobs), _ptr(X), X.shape[0],
                                                   _ptr(Y), _stream_ptr(stream)), "ffsplit_forward_stack")

    def forward_stack_host(self, blobs, X_host, Y_host, stream=None):
        self._check(self.lib.ffsplit_forward_stack_host(self.h, self._blob_array(blobs), len(blobs), _ptr(X_host),
                                                        X_host.shape[0], _ptr(Y_host), _stream_ptr(stream)),
                    "ffsplit_forward_stack_host")

    # ------------------------------------------------------------------ the transformer block around the FFN
    def encoder_desc(self, batch: int, seq: int, heads: int, Wqkv_t, bqkv, Wo_t, bo, ln1, ln2, eps: float, ffn_blob):
        """ffsplit_encoder_layer from device tensors; ln1, ln2 = (gamma, beta).  The tensors must stay alive."""
        return EncoderLayer(batch, seq, heads, Wqkv_t.data_ptr(), bqkv.data_ptr(), Wo_t.data_ptr(), bo.data_ptr(),
                            ln1[0].data_ptr(), ln1[1].data_ptr(), ln2[0].data_ptr(), ln2[1].data_ptr(), eps,
                            ffn_blob.data_ptr())

    def encoder_workspace_size(self, layer: "EncoderLayer") -> int:
        n = C.c_size_t()
        self._check(self.lib.ffsplit_encoder_workspace_size(self.h, C.byref(layer), C.byref(n)), "ffsplit_encoder_workspace_size")
        return n.value

    def encoder_forward(self, layer: "EncoderLayer", X, Y, stream=None):
        self._check(self.lib.ffsplit_encoder_forward(self.h, C.byref(layer), _ptr(X), _ptr(Y), _stream_ptr(stream)),
                    "ffsplit_encoder_forward")

    # ------------------------------------------------------------------ on-device light factors (Section 5.1.1)
    def factor_workspace_size(self, shape: Shape, k: int, r: int) -> int:
        n = C.c_size_t()
        self._check(self.lib.ffsplit_factor_workspace_size(C.byref(shape), k, r, C.byref(n)), "ffsplit_factor_workspace_size")
        return n.value

    def factor_light(self, shape: Shape, W1, W2, light_idx, k: int, r: int, iters: int, start, W1u=None, stream=None) -> dict:
        """ffsplit_factor_light: rank-r factors of the light slices as a dict ready for pack().  `start` is the
        [n, r, d] starting basis (n = 2, or 3 with W1u) in the layer's dtype."""
        d, m = shape.d, shape.m
        ml = m - k
        dev, dt = W1.device, W1.dtype
        f = {"A1": torch.empty(d, r, dtype=dt, device=dev), "B1": torch.empty(r, ml, dtype=dt, device=dev),
             "A2": torch.empty(ml, r, dtype=dt, device=dev), "B2": torch.empty(r, d, dtype=dt, device=dev)}
        if W1u is not None:
            f["A1u"] = torch.empty(d, r, dtype=dt, device=dev)
            f["B1u"] = torch.empty(r, ml, dtype=dt, device=dev)
        w = Weights(_ptr(W1), _ptr(W1u), None, _ptr(W2), None)
        self._check(self.lib.ffsplit_factor_light(self.h, C.byref(shape), C.byref(w), _ptr(light_idx), k, r, iters,
                                                  _ptr(start), _ptr(f["A1"]), _ptr(f["B1"]), _ptr(f["A2"]), _ptr(f["B2"]),
                                                  _ptr(f.get("A1u")), _ptr(f.get("B1u")), _stream_ptr(stream)),
                    "ffsplit_factor_light")
        return f

    # ------------------------------------------------------------------ quantised split (Section 5.2)
    def quant_pack_size(self, shape: Shape, k: int):
        a, b = C.c_size_t(), C.c_size_t()
        self._check(self.lib.ffsplit_quant_pack_size(C.byref(shape), k, C.byref(a), C.byref(b)), "ffsplit_quant_pack_size")
        return a.value, b.value

    def quant_workspace_size(self, shape: Shape, k: int) -> int:
        n = C.c_size_t()
        self._check(self.lib.ffsplit_quant_workspace_size(C.byref(shape), k, C.byref(n)), "ffsplit_quant_workspace_size")
        return n.value

    def quant_pack(self, shape: Shape, W1, b1, W2, b2, heavy_idx, k: int, light_idx, blob, W1u=None, stream=None):
        w = Weights(_ptr(W1), _ptr(W1u), _ptr(b1), _ptr(W2), _ptr(b2))
        self._check(self.lib.ffsplit_quant_pack(self.h, C.byref(shape), C.byref(w), _ptr(heavy_idx), k, _ptr(light_idx),
                                                _ptr(blob), blob.numel() * blob.element_size(), _stream_ptr(stream)),
                    "ffsplit_quant_pack")

    def quant_blob_open(self, blob, stream=None):
        self._check(self.lib.ffsplit_quant_blob_open(self.h, _ptr(blob), blob.numel() * blob.element_size(),
                                                     _stream_ptr(stream)), "ffsplit_quant_blob_open")

    def quant_unpack(self, blob, which: int, rows: int, cols: int, stream=None):
        """-> (codes uint8 [rows, cols], scale float32 [rows, ceil(cols / 128)], lo likewise) of one packed matrix."""
        dev = blob.device
        codes = torch.zeros(rows, cols, dtype=torch.uint8, device=dev)
        ng = (cols + 127) // 128
        scale = torch.zeros(rows, ng, dtype=torch.float32, device=dev)
        lo = torch.zeros(rows, ng, dtype=torch.float32, device=dev)
        self._check(self.lib.ffsplit_quant_unpack(self.h, _ptr(blob), which, _ptr(codes), _ptr(scale), _ptr(lo),
                                                  _stream_ptr(stream)), "ffsplit_quant_unpack")
        return codes, scale, lo

    def quant_forward(self, blob, X, Y, stream=None):
        self._check(self.lib.ffsplit_quant_forward(self.h, _ptr(blob), _ptr(X), X.shape[0], _ptr(Y), _stream_ptr(stream)),
                    "ffsplit_quant_forward")

    def debug_wait_timeout(self, limit_cycles: int, stream=None):
        self._check(self.lib.ffsplit_debug_wait_timeout(self.h, int(limit_cycles), _stream_ptr(stream)),
                    "ffsplit_debug_wait_timeout")

    def blob_section(self, blob, which: int):
        off, r, c, ld = C.c_size_t(), C.c_int64(), C.c_int64(), C.c_int64()
        self._check(self.lib.ffsplit_blob_section(self.h, _ptr(blob), which, C.byref(off), C.byref(r), C.byref(c),
                                                  C.byref(ld)), "ffsplit_blob_section")
        return off.value, r.value, c.value, ld.value

    def forward(self, blob, X, Y, stream=None):
        self._check(self.lib.ffsplit_forward(self.h, _ptr(blob), _ptr(X), X.shape[0], _ptr(Y), _stream_ptr(stream)),
                    "ffsplit_forward")

    def forward_dense(self, shape: Shape, W1, b1, W2, b2, X, Y, W1u=None, stream=None):
        """ffsplit_forward_dense: the unsplit FFN from the row-major weights (packed into the workspace per call)."""
        w = Weights(_ptr(W1), _ptr(W1u), _ptr(b1), _ptr(W2), _ptr(b2))
        self._check(self.lib.ffsplit_forward_dense(self.h, C.byref(shape), C.byref(w), _ptr(X), X.shape[0], _ptr(Y),
                                                   _stream_ptr(stream)), "ffsplit_forward_dense")

    def forward_noalloc(self, blob, X, Y, stream=None):
        """ffsplit_forward_noalloc: up to 8 tokens, bf16, scratch built into the library (no workspace needed)."""
        self._check(self.lib.ffsplit_forward_noalloc(self.h, _ptr(blob), _ptr(X), X.shape[0], _ptr(Y),
                                                     _stream_ptr(stream)), "ffsplit_forward_noalloc")

    def forward_host(self, blob, X_host, Y_host, stream=None):
        self._check(self.lib.ffsplit_forward_host(self.h, _ptr(blob), _ptr(X_host), X_host.shape[0], _ptr(Y_host),
                                                  _stream_ptr(stream)), "ffsplit_forward_host")

    def poll(self, stream=None):
        self._check(self.lib.ffsplit_poll(self.h, _stream_ptr(stream)), "ffsplit_poll")

    def profile_begin(self):
        self._check(self.lib.ffsplit_profile_begin(self.h), "ffsplit_profile_begin")

    def profile_end(self, kernel_class: int = 0, stream=None):
        """-> (launches, total milliseconds, total algorithmic work) of one kernel class."""
        n, ms, work = C.c_int32(), C.c_double(), C.c_double()
        self._check(self.lib.ffsplit_profile_end(self.h, _stream_ptr(stream), kernel_class, C.byref(n), C.byref(ms),
                                                 C.byref(work)), "ffsplit_profile_end")
        return n.value, ms.value, work.value

    def launch_count(self) -> int:
        return int(self.lib.ffsplit_launch_count(self.h))


def read_section(ctx: Context, blob: torch.Tensor, which: int, dtype: torch.dtype) -> torch.Tensor:
    """View of one matrix inside a packed blob (for inspection and tests)."""
    off, rows, cols, ld = ctx.blob_section(blob, which)
    es = torch.empty((), dtype=dtype).element_size()
    raw = blob.view(torch.uint8)[off: off + rows * ld * es]
    return raw.view(dtype).view(rows, ld)[:, :cols]
