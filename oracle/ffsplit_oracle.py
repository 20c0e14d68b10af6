"""CPU fp64 oracle for the split feed-forward network (FFSplit, arXiv 2401.04044).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import it; the product never does, and this
module imports nothing from the product.

Every function takes numpy arrays (any real dtype), up-casts them exactly to
float64 and applies the paper's definition with no blocking, fusion or
intermediate rounding.  Library primitives used as single steps: ``numpy``
matmul, ``numpy`` stable argsort, ``numpy.linalg.svd`` and ``scipy.special.erf``.

Notation follows the paper: X in R^{s x d} (tokens by hidden width), U = W1 in
R^{d x d_ff}, V = W2 in R^{d_ff x d}, h2 = the heavy-hitter index set
(Section 2).  Biases b1, b2 and the SwiGLU form are not in the paper's FFN
(Section 2 writes FFN(X) = sigma(XU)V); they follow the usual transformer
definitions and are documented where they enter.

Pins (tests that tie each function to something other than itself):
  activations ........ closed forms x*Phi(x) via erfc, symmetry identities
  dense_ffn .......... Eq. 1 rank-one sum written with explicit loops
  neuron_scores ...... Eq. 3 removal identity (materialise both FFNs, subtract)
  select_heavy ....... arg-max rounds, exhaustive tie patterns, planted recovery
  light_factors ...... Eckart-Young residual, full rank reproduces the slice
  orthogonal_iteration_factors ... exact for rank(W) <= r after one round, residual never below Eckart-Young's and
                       within 1 % of it after 6 rounds on gapped and on flat spectra, Q orthonormal, A B = Q Q^T W
  split_ffn .......... Eq. 2 (k = d_ff, exact light part, full-rank factors all
                       reproduce the dense FFN), permutation / padding invariance
  param counts ....... the 43.1 % reduction printed in Section 5.1.1
  rtn_quantize ....... |w - dq(q(w))| <= step / 2, grid end points, constant groups and on-grid values exact,
                       round-to-nearest on hand-placed values, independence of groups and of output channels
  quantize_split ..... group axes and bit widths per part, reassembly; quant_split_ffn against Eq. 2 written
                       neuron by neuron on the dequantised weights, error halving per extra bit; byte formula
  layer_norm, multi_head_attention, encoder_layer ... attention written token by token with explicit loops,
                       uniform attention when Q = 0 (output = mean of V), constant V passes through, sequences and
                       heads independent, permutation equivariance inside a sequence; LayerNorm moments, shift
                       invariance; the block with zero attention and zero FFN weights is LN2(LN1(X)) in closed form
Parity unpinned: the error of a *truncated* light part against the dense FFN
(the paper reports task accuracy only, Table 1); it is reported, never gated.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import erf as _erf

ACT_GELU_ERF = "gelu_erf"
ACT_GELU_TANH = "gelu_tanh"
ACT_SWIGLU = "swiglu"

SCORE_EQ3 = "eq3"            # ||sigma(X U_j)||^2 * ||V_j||^2   (Eq. 3, last line)
SCORE_ACT_ONLY = "act_only"  # ||sigma(X U_j)||^2               (Section 2 / Figure 1 ranking)
SCORE_SUM_NORM = "sum_norm"  # sum_t ||sigma(x_t U_j) V_j||     (unsquared reading)


def _f64(a):
    return None if a is None else np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# Activations (Section 2: "sigma is the activation function, e.g., GeLU";
# SwiGLU is named there as the other dominant family).
# --------------------------------------------------------------------------
def gelu_erf(z):
    """GELU(z) = z * Phi(z) = 0.5 z (1 + erf(z / sqrt 2))  (Hendrycks & Gimpel)."""
    z = _f64(z)
    return 0.5 * z * (1.0 + _erf(z / math.sqrt(2.0)))


def gelu_tanh(z):
    """Tanh form: 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))."""
    z = _f64(z)
    return 0.5 * z * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))


def silu(z):
    """SiLU(z) = z / (1 + exp(-z))."""
    z = _f64(z)
    return z / (1.0 + np.exp(-z))


def neuron_activations(X, W1, b1, act, W1u=None):
    """sigma(X U) of Section 2, one column per neuron: H in R^{s x d_ff}.

    GELU variants: H = sigma(X W1 + b1).
    SwiGLU: H = SiLU(X W1) * (X W1u)  (gate W1, up W1u; no bias).
    """
    X, W1, b1, W1u = _f64(X), _f64(W1), _f64(b1), _f64(W1u)
    Z = X @ W1
    if act == ACT_SWIGLU:
        if W1u is None:
            raise ValueError("SwiGLU needs the up projection W1u")
        return silu(Z) * (X @ W1u)
    if b1 is not None:
        Z = Z + b1[None, :]
    if act == ACT_GELU_ERF:
        return gelu_erf(Z)
    if act == ACT_GELU_TANH:
        return gelu_tanh(Z)
    raise ValueError(f"unknown activation {act!r}")


def dense_ffn(X, W1, b1, W2, b2, act, W1u=None):
    """FFN(X) = sigma(X U) V (+ b2)  -- the unnumbered FFN equation of Section 2."""
    H = neuron_activations(X, W1, b1, act, W1u)
    Y = H @ _f64(W2)
    if b2 is not None:
        Y = Y + _f64(b2)[None, :]
    return Y


# --------------------------------------------------------------------------
# Heavy-hitter score (Eq. 3) and selection (Sections 4.1, 5.1.1).
# --------------------------------------------------------------------------
def neuron_scores(X, W1, b1, W2, act, mode=SCORE_EQ3, W1u=None):
    """Per-neuron importance over a calibration token set.

    Eq. 3: removing neuron j changes the FFN output by
    ||sigma(X U_{:,j})||_F^2 * ||V_{j,:}||_F^2 in squared Frobenius norm.
    Returns (energy e, row_energy w, score s):
      e_j = sum_t H[t,j]^2   (sum_t |H[t,j]| for the unsquared reading)
      w_j = sum_c V[j,c]^2
      s_j = e_j w_j (eq3) | e_j (act_only) | e_j sqrt(w_j) (sum_norm)
    """
    H = neuron_activations(X, W1, b1, act, W1u)
    W2 = _f64(W2)
    w = np.sum(W2 * W2, axis=1)
    if mode == SCORE_SUM_NORM:
        e = np.sum(np.abs(H), axis=0)
        return e, w, e * np.sqrt(w)
    e = np.sum(H * H, axis=0)
    if mode == SCORE_EQ3:
        return e, w, e * w
    if mode == SCORE_ACT_ONLY:
        return e, w, e.copy()
    raise ValueError(f"unknown score mode {mode!r}")


def select_heavy(scores, k):
    """h2 = the k neurons with the highest score (Section 4.1: neurons are
    sorted by output norm, the highest are the heavy hitters).  Equal scores
    go to the lower index.  Returns (heavy ascending, light ascending), int32.
    """
    s = np.asarray(scores)
    m = s.shape[0]
    if not (0 <= k <= m):
        raise ValueError("k out of range")
    if not np.all(np.isfinite(s)):
        raise ValueError("non-finite score")
    order = np.argsort(-s, kind="stable")        # stable: ties keep index order
    heavy = np.sort(order[:k]).astype(np.int32)
    mask = np.ones(m, dtype=bool)
    mask[heavy] = False
    light = np.nonzero(mask)[0].astype(np.int32)
    return heavy, light


def select_heavy_argmax_rounds(scores, k):
    """Same set by k rounds of 'take the largest remaining, lowest index first'."""
    s = [float(v) for v in np.asarray(scores)]
    taken = []
    alive = [True] * len(s)
    for _ in range(k):
        best = -1
        for j in range(len(s)):
            if alive[j] and (best < 0 or s[j] > s[best]):
                best = j
        alive[best] = False
        taken.append(best)
    heavy = np.array(sorted(taken), dtype=np.int32)
    light = np.array([j for j in range(len(s)) if alive[j]], dtype=np.int32)
    return heavy, light


# --------------------------------------------------------------------------
# Split weights (Figure 3 caption) and light-part compression (Section 5.1.1).
# --------------------------------------------------------------------------
def split_weights(W1, b1, W2, heavy, W1u=None):
    """U1 = U[:, h2], V1 = V[h2, :]; U2, V2 = the remaining neurons, in
    ascending index order.  Returns a dict of float64 arrays."""
    W1, b1, W2, W1u = _f64(W1), _f64(b1), _f64(W2), _f64(W1u)
    m = W1.shape[1]
    heavy = np.asarray(heavy, dtype=np.int64)
    mask = np.ones(m, dtype=bool)
    mask[heavy] = False
    light = np.nonzero(mask)[0]
    out = {
        "heavy": heavy, "light": light,
        "U1": W1[:, heavy], "V1": W2[heavy, :],
        "U2": W1[:, light], "V2": W2[light, :],
        "b1_heavy": None if b1 is None else b1[heavy],
        "b1_light": None if b1 is None else b1[light],
    }
    if W1u is not None:
        out["U1u"] = W1u[:, heavy]
        out["U2u"] = W1u[:, light]
    return out


def light_factors(W, r):
    """Rank-r factors of a light slice by truncated SVD (Section 5.1.1: SVD on
    U2 and V2 only).  W = P S Q^T; returns A = P_r S_r^{1/2}, B = S_r^{1/2} Q_r^T
    so that A @ B is the best rank-r approximation of W."""
    W = _f64(W)
    P, S, Qt = np.linalg.svd(W, full_matrices=False)
    r = int(r)
    if not (0 <= r <= S.shape[0]):
        raise ValueError("rank out of range")
    root = np.sqrt(S[:r])
    return P[:, :r] * root[None, :], root[:, None] * Qt[:r, :]


def orthogonal_iteration_factors(W, r, iters, start):
    """Rank-r factors of W [d, n] from `iters` rounds of block power (orthogonal) iteration on the left singular
    subspace: Q <- orth(W W^T Q), starting from start [d, r]; returns A = Q, B = Q^T W, so that A @ B is the
    orthogonal projection of W's columns onto span(Q).  This is the textbook iteration the on-device routine
    follows (its own choice of algorithm for the rank-r decomposition of Section 5.1.1); orth is numpy's
    Householder QR here.  As span(Q) converges to the leading singular subspace A @ B converges to
    light_factors' product; for rank(W) <= r one round reproduces W exactly."""
    W = _f64(W)
    Q = _f64(start)
    if Q.shape != (W.shape[0], int(r)):
        raise ValueError("start must be [d, r]")
    for _ in range(int(iters)):
        Q, _ = np.linalg.qr(W @ (W.T @ Q))
    return Q, Q.T @ W


def split_ffn(X, W1, b1, W2, b2, heavy, factors, act, W1u=None):
    """Eq. 2: FFN(X) = FFN_1(X) + FFN_2(X) with FFN_1 over h2 kept dense and
    FFN_2 over the remaining neurons using compressed weights.

    factors: None (FFN_2 uses the exact light slices U2, V2 -- Eq. 2 as
    printed), or a dict with 'A1','B1' (U2 ~ A1 B1), 'A2','B2' (V2 ~ A2 B2)
    and for SwiGLU 'A1u','B1u' (up-projection light slice); an empty light set
    or rank 0 contributes nothing.  b1 enters both parts inside sigma; b2 is
    added once.
    """
    X = _f64(X)
    sw = split_weights(W1, b1, W2, heavy, W1u)

    def part(U, Uu, bias, V):
        if U.shape[1] == 0:
            return np.zeros((X.shape[0], _f64(W2).shape[1]))
        return dense_ffn(X, U, bias, V, None, act, Uu)

    Y = part(sw["U1"], sw.get("U1u"), sw["b1_heavy"], sw["V1"])
    if sw["light"].shape[0] > 0:
        if factors is None:
            Y = Y + part(sw["U2"], sw.get("U2u"), sw["b1_light"], sw["V2"])
        else:
            A1, B1 = _f64(factors["A1"]), _f64(factors["B1"])
            A2, B2 = _f64(factors["A2"]), _f64(factors["B2"])
            if A1.shape[1] > 0:
                Z = (X @ A1) @ B1
                if act == ACT_SWIGLU:
                    Zu = (X @ _f64(factors["A1u"])) @ _f64(factors["B1u"])
                    Hl = silu(Z) * Zu
                else:
                    if sw["b1_light"] is not None:
                        Z = Z + sw["b1_light"][None, :]
                    Hl = gelu_erf(Z) if act == ACT_GELU_ERF else gelu_tanh(Z)
                Y = Y + (Hl @ A2) @ B2
    if b2 is not None:
        Y = Y + _f64(b2)[None, :]
    return Y


# --------------------------------------------------------------------------
# Model size (Section 5.1.1: top 25 % heavy + rank 10 % => 43.1 % fewer
# parameters, embeddings excluded).
# --------------------------------------------------------------------------
def ffn_weight_params(d, m, n_in=1):
    """Weights of one dense FFN: n_in up-projections and one down-projection."""
    return (n_in + 1) * d * m


def split_weight_params(d, m, k, r, n_in=1):
    """Weights of one split FFN: dense heavy slices plus rank-r factor pairs of
    every light slice."""
    return (n_in + 1) * (d * k + r * (d + (m - k)))


# --------------------------------------------------------------------------
# Error metrics used by the parity tests.
# --------------------------------------------------------------------------
def rel_frobenius(Y, Yref):
    Y, Yref = _f64(Y), _f64(Yref)
    den = np.linalg.norm(Yref)
    return float(np.linalg.norm(Y - Yref) / den) if den > 0 else float(np.linalg.norm(Y))


def normalised_max_abs(Y, Yref):
    Y, Yref = _f64(Y), _f64(Yref)
    den = np.max(np.abs(Yref)) if Yref.size else 0.0
    num = np.max(np.abs(Y - Yref)) if Yref.size else 0.0
    return float(num / den) if den > 0 else float(num)


# --------------------------------------------------------------------------
# Quantised split (Section 5.2): round-to-nearest with a group size of 128, 8 bits for the heavy-hitter
# neurons and 3 bits for everything else.  The paper fixes the bit widths, the group size and "round to
# nearest"; it does not say along which axis the groups run, whether the grid is symmetric, or how codes
# are stored.  Reading taken here (the usual "wB-g128" convention of weight-only quantisation):
#   * each of the four matrices of the split (U1, V1 heavy; U2, V2 light) is quantised on its own;
#   * a group is 128 consecutive weights along the INPUT dimension of the linear map, for one output
#     channel: along d for a column of U (one neuron's input weights), along the neuron axis of the part
#     (heavy neurons, or light neurons, in ascending index order) for a column of V; a last, shorter group
#     takes what is left;
#   * asymmetric min/max grid: lo = min, scale = (max - lo) / (2^b - 1), code q = round((w - lo) / scale)
#     clamped to [0, 2^b - 1], dequantised value lo + q * scale; a constant group has scale 0, code 0 and is
#     reproduced exactly;
#   * the decisions (min, max, scale, the rounding) are taken in float32 arithmetic, round-half-to-even --
#     the precision the CUDA path takes them in -- so that codes can be compared bit for bit; the
#     dequantised value is lo + q * scale evaluated exactly from the stored float32 (lo, scale);
#   * biases are not quantised.
# --------------------------------------------------------------------------
QUANT_GROUP = 128
QUANT_BITS_HEAVY = 8
QUANT_BITS_LIGHT = 3


def rtn_quantize_groups(w, bits, group=QUANT_GROUP):
    """Round-to-nearest quantisation of the LAST axis of `w` in groups of `group` (the last one may be
    shorter).  Returns (codes uint8 with w's shape, scale float32 [..., n_groups], lo float32 [..., n_groups])."""
    w = np.asarray(w, dtype=np.float32)
    n = w.shape[-1]
    ng = (n + group - 1) // group
    qmax = np.float32((1 << bits) - 1)
    codes = np.zeros(w.shape, dtype=np.uint8)
    scale = np.zeros(w.shape[:-1] + (ng,), dtype=np.float32)
    lo = np.zeros_like(scale)
    for g in range(ng):
        seg = w[..., g * group:(g + 1) * group]
        mn = seg.min(axis=-1).astype(np.float32)
        mx = seg.max(axis=-1).astype(np.float32)
        sc = ((mx - mn).astype(np.float32) / qmax).astype(np.float32)
        lo[..., g] = mn
        scale[..., g] = sc
        safe = np.where(sc > 0, sc, np.float32(1.0)).astype(np.float32)
        q = np.rint(((seg - mn[..., None]).astype(np.float32) / safe[..., None]).astype(np.float32))
        q = np.clip(q, 0, float(qmax))
        q = np.where(sc[..., None] > 0, q, 0.0)
        codes[..., g * group:(g + 1) * group] = q.astype(np.uint8)
    return codes, scale, lo


def rtn_dequantize_groups(codes, scale, lo, group=QUANT_GROUP):
    """lo + q * scale per group, in float64 (exact for the stored float32 parameters and integer codes)."""
    codes = np.asarray(codes)
    n = codes.shape[-1]
    idx = np.arange(n) // group
    return _f64(lo)[..., idx] + codes.astype(np.float64) * _f64(scale)[..., idx]


def quantize_split(W1, W2, heavy, bits_heavy=QUANT_BITS_HEAVY, bits_light=QUANT_BITS_LIGHT, group=QUANT_GROUP,
                   W1u=None):
    """The four (SwiGLU: six) quantised matrices of the split.  Every entry of the result is a triple
    (codes, scale, lo) laid out with the grouped (input) axis last:
      'U1', 'U2' (and 'U1u', 'U2u'): [neurons of the part, d]        groups along d
      'V1', 'V2':                    [d, neurons of the part]        groups along the part's neuron axis
    """
    sw = split_weights(W1, None, W2, heavy, W1u)
    out = {"heavy": sw["heavy"], "light": sw["light"]}
    out["U1"] = rtn_quantize_groups(sw["U1"].T, bits_heavy, group)
    out["U2"] = rtn_quantize_groups(sw["U2"].T, bits_light, group)
    out["V1"] = rtn_quantize_groups(sw["V1"].T, bits_heavy, group)
    out["V2"] = rtn_quantize_groups(sw["V2"].T, bits_light, group)
    if W1u is not None:
        out["U1u"] = rtn_quantize_groups(sw["U1u"].T, bits_heavy, group)
        out["U2u"] = rtn_quantize_groups(sw["U2u"].T, bits_light, group)
    return out


def dequantized_weights(Q, d, m, group=QUANT_GROUP):
    """Reassemble the full matrices W1~ [d, m], W2~ [m, d] (and W1u~) from the quantised parts."""
    heavy, light = Q["heavy"], Q["light"]
    W1 = np.zeros((d, m))
    W2 = np.zeros((m, d))
    W1[:, heavy] = rtn_dequantize_groups(*Q["U1"], group).T
    W1[:, light] = rtn_dequantize_groups(*Q["U2"], group).T
    W2[heavy, :] = rtn_dequantize_groups(*Q["V1"], group).T
    W2[light, :] = rtn_dequantize_groups(*Q["V2"], group).T
    W1u = None
    if "U1u" in Q:
        W1u = np.zeros((d, m))
        W1u[:, heavy] = rtn_dequantize_groups(*Q["U1u"], group).T
        W1u[:, light] = rtn_dequantize_groups(*Q["U2u"], group).T
    return W1, W2, W1u


def quant_split_ffn(X, b1, b2, Q, d, m, act, group=QUANT_GROUP):
    """Eq. 2 with FFN_1 on the 8-bit heavy matrices and FFN_2 on the 3-bit light ones: the dense FFN of
    Section 2 evaluated on the dequantised weights (both parts use their own neurons' biases)."""
    W1, W2, W1u = dequantized_weights(Q, d, m, group)
    return dense_ffn(X, W1, b1, W2, b2, act, W1u)


def quant_weight_bytes(d, m, k, bits_heavy=QUANT_BITS_HEAVY, bits_light=QUANT_BITS_LIGHT, group=QUANT_GROUP,
                       n_in=1, param_bytes=8):
    """Bytes of the quantised weights: codes at their bit width plus one (scale, lo) pair of float32 per group
    (param_bytes = 8).  U-type matrices have ceil(d / group) groups per neuron, V-type ceil(neurons / group)
    per output column."""
    ml = m - k
    gd = -(-d // group)
    def part(n, bits):
        if n == 0:
            return 0
        gv = -(-n // group)
        u_bits = n_in * n * d * bits
        v_bits = n * d * bits
        return (u_bits + v_bits) / 8 + param_bytes * (n_in * n * gd + d * gv)
    return part(k, bits_heavy) + part(ml, bits_light)


# ---------------------------------------------------------------------------------------------------
# The transformer block around the FFN (Section 5.1.2 / Table 2 time whole BERT-base models).  The paper gives no
# formulas for it; these are the standard post-LayerNorm encoder definitions (Vaswani et al. 2017, Devlin et al.
# 2019): scaled dot-product attention over whole sequences without a padding mask, heads of equal width.
# ---------------------------------------------------------------------------------------------------
def layer_norm(x, gamma, beta, eps):
    """Per row: (x - mean) / sqrt(var + eps) * gamma + beta, var the biased variance over the features."""
    x = _f64(x)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * _f64(gamma) + _f64(beta)


def multi_head_attention(X, Wqkv, bqkv, Wo, bo, batch, seq, heads):
    """X [batch * seq, d], sequence after sequence; Wqkv [d, 3 d] = [Wq | Wk | Wv], head h owning columns
    h dh .. (h + 1) dh - 1 of each; per sequence and head softmax(Q K^T / sqrt(dh)) V, heads concatenated, times Wo."""
    X, Wqkv, bqkv, Wo, bo = _f64(X), _f64(Wqkv), _f64(bqkv), _f64(Wo), _f64(bo)
    T, d = X.shape
    if T != batch * seq or d % heads:
        raise ValueError("shape mismatch")
    dh = d // heads
    qkv = X @ Wqkv + bqkv
    out = np.empty((T, d))
    for b in range(batch):
        rows = slice(b * seq, (b + 1) * seq)
        for h in range(heads):
            q = qkv[rows, h * dh:(h + 1) * dh]
            k = qkv[rows, d + h * dh:d + (h + 1) * dh]
            v = qkv[rows, 2 * d + h * dh:2 * d + (h + 1) * dh]
            s = q @ k.T / math.sqrt(dh)
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p = p / p.sum(axis=1, keepdims=True)
            out[rows, h * dh:(h + 1) * dh] = p @ v
    return out @ Wo + bo


def encoder_layer(X, attn, ln1, ln2, eps, batch, seq, heads, ffn):
    """Y = LN2(X1 + ffn(X1)), X1 = LN1(X + MHA(X)); attn = (Wqkv, bqkv, Wo, bo), ln = (gamma, beta), ffn a function
    of the token matrix (dense_ffn or split_ffn with its weights bound)."""
    X = _f64(X)
    A = multi_head_attention(X, *attn, batch, seq, heads)
    X1 = layer_norm(X + A, ln1[0], ln1[1], eps)
    return layer_norm(X1 + _f64(ffn(X1)), ln2[0], ln2[1], eps)

