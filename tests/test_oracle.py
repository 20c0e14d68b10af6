"""Pins for the CPU oracle: each function is tied to something other than
itself -- closed forms, the paper's identities (Eq. 1, Eq. 2, Eq. 3), textbook
theorems (Eckart-Young) and brute force on tiny inputs."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import ffsplit_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ACTS = [orc.ACT_GELU_ERF, orc.ACT_GELU_TANH, orc.ACT_SWIGLU]


def _tiny(rng, s=5, d=4, m=7, act=orc.ACT_GELU_ERF, bias=True):
    X = rng.normal(size=(s, d))
    W1 = rng.normal(size=(d, m)) * 0.7
    W1u = rng.normal(size=(d, m)) * 0.7 if act == orc.ACT_SWIGLU else None
    W2 = rng.normal(size=(m, d + 1))          # non-square output on purpose
    b1 = rng.normal(size=m) if (bias and act != orc.ACT_SWIGLU) else None
    b2 = rng.normal(size=d + 1) if bias else None
    return X, W1, W1u, b1, W2, b2


# ---------------------------------------------------------------- activations
def test_activation_golden_values():
    fn = {"gelu_erf": orc.gelu_erf, "silu": orc.silu}
    n = 0
    for line in open(os.path.join(GOLDEN, "activation_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, x, v = line.split()
        assert abs(float(fn[name](np.array([float(x)]))[0]) - float(v)) < 1e-14
        n += 1
    assert n == 7


def test_gelu_erf_is_x_times_normal_cdf():
    for x in np.linspace(-6, 6, 49):
        phi = 0.5 * math.erfc(-x / math.sqrt(2.0))
        assert abs(orc.gelu_erf(np.array([x]))[0] - x * phi) < 1e-14


def test_activation_symmetries():
    x = np.linspace(-5, 5, 101)
    # x*Phi(x) - (-x)*Phi(-x) = x
    assert np.allclose(orc.gelu_erf(x) - orc.gelu_erf(-x), x, atol=1e-14)
    assert np.allclose(orc.gelu_tanh(x) - orc.gelu_tanh(-x), x, atol=1e-14)
    # SiLU(x) + SiLU(-x) = x tanh(x/2)
    assert np.allclose(orc.silu(x) + orc.silu(-x), x * np.tanh(x / 2), atol=1e-14)
    # tanh form tracks the erf form to < 1e-3 everywhere, and is not identical
    gap = np.max(np.abs(orc.gelu_tanh(x) - orc.gelu_erf(x)))
    assert 1e-5 < gap < 1e-3
    # value of the tanh form at 1 written out term by term
    inner = math.sqrt(2 / math.pi) * (1 + 0.044715)
    assert abs(orc.gelu_tanh(np.array([1.0]))[0] - 0.5 * (1 + math.tanh(inner))) < 1e-15


# ---------------------------------------------------------------- dense FFN
def test_dense_ffn_hand_worked_example():
    # one token x = (1, 0): z = first row of W1 = (0, 1, -1); GELU = (0, Phi(1), -Phi(-1))
    X = np.array([[1.0, 0.0]])
    W1 = np.array([[0.0, 1.0, -1.0], [5.0, 6.0, 7.0]])
    W2 = np.array([[9.0, 9.0], [1.0, 2.0], [3.0, 4.0]])
    p1, pm1 = 0.8413447460685429, 0.15865525393145707
    want = np.array([[p1 * 1 - pm1 * 3, p1 * 2 - pm1 * 4]])
    got = orc.dense_ffn(X, W1, None, W2, None, orc.ACT_GELU_ERF)
    assert np.allclose(got, want, atol=1e-14)
    # bias shifts: b1 = (1, 0, 0) makes z_0 = 1; b2 adds (10, 20)
    got = orc.dense_ffn(X, W1, np.array([1.0, 0, 0]), W2, np.array([10.0, 20.0]), orc.ACT_GELU_ERF)
    assert np.allclose(got, want + p1 * 9 + np.array([[10.0, 20.0]]), atol=1e-13)


@pytest.mark.parametrize("act", ACTS)
def test_dense_ffn_equals_rank_one_sum(rng, act):
    """Eq. 1: FFN(X) = sum_j sigma(X U_{:,j}) V_{j,:}, written with scalar loops."""
    X, W1, W1u, b1, W2, b2 = _tiny(rng, act=act)
    s, d = X.shape
    m, dout = W2.shape
    Y = np.zeros((s, dout))
    for j in range(m):
        col = np.zeros(s)
        for t in range(s):
            z = sum(X[t, i] * W1[i, j] for i in range(d))
            if act == orc.ACT_SWIGLU:
                u = sum(X[t, i] * W1u[i, j] for i in range(d))
                col[t] = z / (1 + math.exp(-z)) * u
            else:
                z += b1[j]
                if act == orc.ACT_GELU_ERF:
                    col[t] = z * 0.5 * math.erfc(-z / math.sqrt(2))
                else:
                    col[t] = 0.5 * z * (1 + math.tanh(math.sqrt(2 / math.pi) * (z + 0.044715 * z ** 3)))
        Y += np.outer(col, W2[j, :])
    Y += b2[None, :]
    assert np.allclose(orc.dense_ffn(X, W1, b1, W2, b2, act, W1u), Y, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- score
@pytest.mark.parametrize("act", ACTS)
def test_score_is_the_removal_residual(rng, act):
    """Eq. 3: ||FFN(X) - FFN_{without j}(X)||_F^2 = ||sigma(X U_j)||^2 ||V_j||^2."""
    X, W1, W1u, b1, W2, b2 = _tiny(rng, s=9, act=act)
    e, w, sc = orc.neuron_scores(X, W1, b1, W2, act, orc.SCORE_EQ3, W1u)
    full = orc.dense_ffn(X, W1, b1, W2, b2, act, W1u)
    for j in range(W1.shape[1]):
        W1r = np.delete(W1, j, axis=1)
        W1ur = None if W1u is None else np.delete(W1u, j, axis=1)
        b1r = None if b1 is None else np.delete(b1, j)
        W2r = np.delete(W2, j, axis=0)
        less = orc.dense_ffn(X, W1r, b1r, W2r, b2, act, W1ur)
        resid = np.sum((full - less) ** 2)
        assert abs(resid - sc[j]) <= 1e-10 * max(resid, 1e-30)
    assert np.allclose(e * w, sc)


def test_score_modes_by_explicit_contributions(rng):
    X, W1, W1u, b1, W2, b2 = _tiny(rng, s=6)
    H = orc.neuron_activations(X, W1, b1, orc.ACT_GELU_ERF)
    _, _, s_act = orc.neuron_scores(X, W1, b1, W2, orc.ACT_GELU_ERF, orc.SCORE_ACT_ONLY)
    _, _, s_sum = orc.neuron_scores(X, W1, b1, W2, orc.ACT_GELU_ERF, orc.SCORE_SUM_NORM)
    for j in range(W1.shape[1]):
        contrib = np.outer(H[:, j], W2[j, :])                  # s x d_out
        assert abs(s_act[j] - np.linalg.norm(H[:, j]) ** 2) < 1e-12
        assert abs(s_sum[j] - sum(np.linalg.norm(contrib[t]) for t in range(X.shape[0]))) < 1e-12
    # ranking by Eq. 3 is unchanged by a square root; the unsquared sum may differ
    _, _, s3 = orc.neuron_scores(X, W1, b1, W2, orc.ACT_GELU_ERF, orc.SCORE_EQ3)
    assert np.array_equal(orc.select_heavy(s3, 3)[0], orc.select_heavy(np.sqrt(s3), 3)[0])


def test_score_is_additive_over_token_batches(rng):
    X, W1, W1u, b1, W2, b2 = _tiny(rng, s=10)
    e, w, _ = orc.neuron_scores(X, W1, b1, W2, orc.ACT_GELU_ERF)
    e1, _, _ = orc.neuron_scores(X[:4], W1, b1, W2, orc.ACT_GELU_ERF)
    e2, _, _ = orc.neuron_scores(X[4:], W1, b1, W2, orc.ACT_GELU_ERF)
    assert np.allclose(e, e1 + e2, rtol=1e-13)


# ---------------------------------------------------------------- select
def _select_by_python_sort(s, k):
    order = sorted(range(len(s)), key=lambda j: (-float(s[j]), j))
    heavy = sorted(order[:k])
    light = sorted(order[k:])
    return heavy, light


def test_select_exhaustive_tie_patterns():
    for m in range(1, 8):
        for pattern in itertools.product((0.0, 1.0, 2.5), repeat=m) if m <= 5 else \
                itertools.product((0.0, 1.0), repeat=m):
            s = np.array(pattern, dtype=np.float32)
            for k in range(m + 1):
                h, l = orc.select_heavy(s, k)
                hw, lw = _select_by_python_sort(s, k)
                assert list(h) == hw and list(l) == lw
                h2, l2 = orc.select_heavy_argmax_rounds(s, k)
                assert list(h2) == hw and list(l2) == lw


def test_select_random_against_argmax_rounds(rng):
    for m, k in [(1, 1), (17, 5), (64, 64), (100, 0), (257, 31)]:
        s = (rng.random(m) ** 3).astype(np.float32)
        s[rng.integers(0, m, size=m // 3)] = s[0]            # many equal keys
        h, l = orc.select_heavy(s, k)
        h2, l2 = orc.select_heavy_argmax_rounds(s, k)
        assert np.array_equal(h, h2) and np.array_equal(l, l2)
        assert h.dtype == np.int32 and len(h) == k and len(l) == m - k
        assert sorted(set(h.tolist()) | set(l.tolist())) == list(range(m))
        if k:
            assert s[h].min() >= (s[l].max() if len(l) else -1)


def test_select_edge_cases_and_invariances(rng):
    s = rng.random(50).astype(np.float32)
    assert np.array_equal(orc.select_heavy(s, 50)[0], np.arange(50))
    assert len(orc.select_heavy(s, 0)[0]) == 0
    assert np.array_equal(orc.select_heavy(s, 7)[0], orc.select_heavy(s.astype(np.float64) ** 2, 7)[0])
    # all keys equal: the k lowest indices win
    assert np.array_equal(orc.select_heavy(np.ones(9, np.float32), 4)[0], np.arange(4))
    with pytest.raises(ValueError):
        orc.select_heavy(np.array([1.0, np.nan]), 1)
    with pytest.raises(ValueError):
        orc.select_heavy(s, 51)


def test_planted_heavy_hitters_are_recovered():
    from ffsplit_synth import custom_config, make_layer
    from conftest import f64
    for act in ("gelu_erf", "swiglu"):
        cfg = custom_config(64, 256, 13, 16, act=act, dtype="f32")
        L = make_layer(cfg, 0)
        X = L.tokens(128)
        _, _, s = orc.neuron_scores(f64(X), f64(L.W1), f64(L.b1), f64(L.W2), act, orc.SCORE_EQ3, f64(L.W1u))
        heavy, _ = orc.select_heavy(s, 13)
        assert np.array_equal(heavy, L.planted.numpy())
        # and the gap to the best light neuron is wide (x100 from the V rows)
        light_best = np.max(np.delete(s, heavy))
        assert s[heavy].min() > 10 * light_best


# ---------------------------------------------------------------- factors
def test_light_factors_eckart_young(rng):
    W = rng.normal(size=(12, 30))
    sig2 = np.sort(np.linalg.eigvalsh(W @ W.T))[::-1]         # squared singular values, another routine
    for r in (0, 1, 5, 12):
        A, B = orc.light_factors(W, r)
        assert A.shape == (12, r) and B.shape == (r, 30)
        resid = np.sum((W - A @ B) ** 2)
        assert abs(resid - np.sum(sig2[r:])) < 1e-9
    A, B = orc.light_factors(W, 12)
    assert np.allclose(A @ B, W, atol=1e-12)
    # balanced split: both factors carry sqrt(sigma)
    A, B = orc.light_factors(W, 4)
    assert np.allclose(np.linalg.norm(A, axis=0), np.linalg.norm(B, axis=1), rtol=1e-10)


def test_light_factors_known_spectrum(rng):
    Q1, _ = np.linalg.qr(rng.normal(size=(10, 10)))
    Q2, _ = np.linalg.qr(rng.normal(size=(25, 10)))
    s = np.array([9.0, 7, 5, 3, 2, 1, .5, .25, .1, .05])
    W = (Q1 * s) @ Q2.T
    A, B = orc.light_factors(W, 3)
    assert np.allclose(A @ B, (Q1[:, :3] * s[:3]) @ Q2[:, :3].T, atol=1e-12)


def test_orthogonal_iteration_factors_against_eckart_young(rng):
    """The iteration the on-device factorisation follows, pinned to what the mathematics fixes: a projection can
    never beat the truncated SVD, it equals it when the spectrum has a gap and the iteration has converged, it is
    exact for a matrix of rank <= r, and on a flat (Gaussian) spectrum six rounds come within 1 % of the optimum."""
    d, n, r = 24, 70, 6
    # gapped spectrum: known singular vectors
    P, _ = np.linalg.qr(rng.normal(size=(d, d)))
    V, _ = np.linalg.qr(rng.normal(size=(n, d)))
    sv = np.concatenate([np.linspace(10, 6, r), np.linspace(1.0, 0.1, d - r)])
    W = (P * sv) @ V.T
    start = rng.normal(size=(d, r))
    opt = np.sqrt(np.sum(sv[r:] ** 2))
    prev = np.inf
    for iters in (0, 1, 2, 6, 12):
        A, B = orc.orthogonal_iteration_factors(W, r, iters, start)
        assert A.shape == (d, r) and B.shape == (r, n)
        err = np.linalg.norm(W - A @ B)
        assert err >= opt * (1 - 1e-12) and err <= prev * (1 + 1e-12)      # never below Eckart-Young, monotone here
        prev = err
        if iters > 0:
            assert np.allclose(A.T @ A, np.eye(r), atol=1e-12)            # orthonormal basis
            assert np.allclose(A @ B, A @ (A.T @ W), atol=1e-12)          # the projection Q Q^T W
    assert abs(prev - opt) < 1e-6 * opt
    A, B = orc.orthogonal_iteration_factors(W, r, 12, start)
    assert np.allclose(A @ B, (P[:, :r] * sv[:r]) @ V[:, :r].T, atol=1e-6)  # the truncated SVD's product itself
    # rank(W) <= r: one round reproduces W
    W0 = rng.normal(size=(d, 4)) @ rng.normal(size=(4, n))
    A, B = orc.orthogonal_iteration_factors(W0, r, 1, start)
    assert np.allclose(A @ B, W0, atol=1e-10)
    # flat spectrum (the synthetic layers' light slices are Gaussian): within 1 % of the optimum after 6 rounds
    G = rng.normal(size=(64, 400))
    s2 = np.linalg.svd(G, compute_uv=False) ** 2
    for rr in (8, 16):
        A, B = orc.orthogonal_iteration_factors(G, rr, 6, rng.normal(size=(64, rr)))
        err, best = np.linalg.norm(G - A @ B), np.sqrt(np.sum(s2[rr:]))
        assert best <= err <= 1.01 * best
    with pytest.raises(ValueError):
        orc.orthogonal_iteration_factors(W, r, 1, rng.normal(size=(d, r + 1)))


# ---------------------------------------------------------------- split FFN
def _full_rank_factors(sw, act):
    f = {}
    f["A1"], f["B1"] = orc.light_factors(sw["U2"], min(sw["U2"].shape))
    f["A2"], f["B2"] = orc.light_factors(sw["V2"], min(sw["V2"].shape))
    if act == orc.ACT_SWIGLU:
        f["A1u"], f["B1u"] = orc.light_factors(sw["U2u"], min(sw["U2u"].shape))
    return f


@pytest.mark.parametrize("act", ACTS)
def test_split_reproduces_dense(rng, act):
    """Eq. 2 holds for any index set; k = d_ff, k = 0 and full-rank light factors
    all give back the dense FFN."""
    X, W1, W1u, b1, W2, b2 = _tiny(rng, s=6, d=5, m=11, act=act)
    dense = orc.dense_ffn(X, W1, b1, W2, b2, act, W1u)
    m = W1.shape[1]
    for heavy in ([], [3], [0, 4, 10], [10, 2, 7, 1], list(range(m))):
        y = orc.split_ffn(X, W1, b1, W2, b2, heavy, None, act, W1u)
        assert np.allclose(y, dense, rtol=1e-12, atol=1e-12)
        if len(heavy) < m:
            sw = orc.split_weights(W1, b1, W2, heavy, W1u)
            y = orc.split_ffn(X, W1, b1, W2, b2, heavy, _full_rank_factors(sw, act), act, W1u)
            assert np.allclose(y, dense, rtol=1e-10, atol=1e-10)
    # ascending full set is the same summation order as the dense FFN
    y = orc.split_ffn(X, W1, b1, W2, b2, np.arange(m), None, act, W1u)
    assert np.array_equal(y, dense)


@pytest.mark.parametrize("act", ACTS)
def test_split_truncated_rank_is_exact_on_low_rank_light_slices(rng, act):
    """If the light slices have rank <= r, the rank-r factors lose nothing."""
    s, d, m, r = 7, 8, 20, 3
    heavy = [1, 5, 6, 19]
    light = [j for j in range(m) if j not in heavy]
    X = rng.normal(size=(s, d))

    def low_rank_except_heavy(shape_rows, along_cols):
        W = rng.normal(size=shape_rows)
        L = rng.normal(size=(d, r)) @ rng.normal(size=(r, len(light)))
        if along_cols:
            W[:, light] = L
        else:
            W[light, :] = L.T
        return W

    W1 = low_rank_except_heavy((d, m), True)
    W1u = low_rank_except_heavy((d, m), True) if act == orc.ACT_SWIGLU else None
    W2 = low_rank_except_heavy((m, d), False)
    b1 = rng.normal(size=m) if act != orc.ACT_SWIGLU else None
    b2 = rng.normal(size=d)
    sw = orc.split_weights(W1, b1, W2, heavy, W1u)
    f = {}
    f["A1"], f["B1"] = orc.light_factors(sw["U2"], r)
    f["A2"], f["B2"] = orc.light_factors(sw["V2"], r)
    if act == orc.ACT_SWIGLU:
        f["A1u"], f["B1u"] = orc.light_factors(sw["U2u"], r)
    y = orc.split_ffn(X, W1, b1, W2, b2, heavy, f, act, W1u)
    assert np.allclose(y, orc.dense_ffn(X, W1, b1, W2, b2, act, W1u), rtol=1e-9, atol=1e-9)
    # rank 0 drops the light part: what is left is the FFN over the heavy neurons only
    f0 = {key: (v[:, :0] if key.startswith("A") else v[:0, :]) for key, v in f.items()}
    y0 = orc.split_ffn(X, W1, b1, W2, b2, heavy, f0, act, W1u)
    only = orc.dense_ffn(X, W1[:, heavy], None if b1 is None else b1[heavy], W2[heavy, :], b2, act,
                         None if W1u is None else W1u[:, heavy])
    assert np.allclose(y0, only, rtol=1e-12, atol=1e-12)


def test_split_truncation_changes_the_output_and_uses_the_given_factors(rng):
    X, W1, W1u, b1, W2, b2 = _tiny(rng, s=6, d=6, m=14)
    heavy = [0, 3, 9]
    sw = orc.split_weights(W1, b1, W2, heavy)
    f = {}
    f["A1"], f["B1"] = orc.light_factors(sw["U2"], 2)
    f["A2"], f["B2"] = orc.light_factors(sw["V2"], 2)
    y = orc.split_ffn(X, W1, b1, W2, b2, heavy, f, orc.ACT_GELU_ERF)
    # same thing spelled out with the reconstructed light matrices
    U2h, V2h = f["A1"] @ f["B1"], f["A2"] @ f["B2"]
    W1c, W2c = W1.copy(), W2.copy()
    W1c[:, sw["light"]] = U2h
    W2c[sw["light"], :] = V2h
    assert np.allclose(y, orc.dense_ffn(X, W1c, b1, W2c, b2, orc.ACT_GELU_ERF), rtol=1e-11, atol=1e-11)
    assert not np.allclose(y, orc.dense_ffn(X, W1, b1, W2, b2, orc.ACT_GELU_ERF), atol=1e-3)


@pytest.mark.parametrize("act", ACTS)
def test_split_permutation_and_padding_invariance(rng, act):
    X, W1, W1u, b1, W2, b2 = _tiny(rng, s=4, d=5, m=9, act=act)
    heavy = np.array([2, 7, 8])
    sw = orc.split_weights(W1, b1, W2, heavy, W1u)
    f = {}
    f["A1"], f["B1"] = orc.light_factors(sw["U2"], 2)
    f["A2"], f["B2"] = orc.light_factors(sw["V2"], 2)
    if act == orc.ACT_SWIGLU:
        f["A1u"], f["B1u"] = orc.light_factors(sw["U2u"], 2)
    y = orc.split_ffn(X, W1, b1, W2, b2, heavy, f, act, W1u)
    # relabel neurons: move every neuron j to position perm_inv[j]; keep the light
    # order inside the factors by permuting only heavy labels among themselves and
    # shifting the whole layer by appended zero neurons (padding)
    m = W1.shape[1]
    pad = 3
    W1p = np.concatenate([W1, np.zeros((W1.shape[0], pad))], axis=1)
    W2p = np.concatenate([W2, np.zeros((pad, W2.shape[1]))], axis=0)
    W1up = None if W1u is None else np.concatenate([W1u, np.zeros((W1u.shape[0], pad))], axis=1)
    b1p = None if b1 is None else np.concatenate([b1, np.zeros(pad)])
    heavy_p = np.concatenate([heavy, np.arange(m, m + pad)])      # zero neurons join the heavy set
    yp = orc.split_ffn(X, W1p, b1p, W2p, b2, heavy_p, f, act, W1up)
    assert np.allclose(yp, y, rtol=1e-13, atol=1e-13)
    # permutation of the whole neuron axis, exact light part (Eq. 1 is a sum over neurons)
    perm = rng.permutation(m)
    inv = np.argsort(perm)
    y_exact = orc.split_ffn(X, W1, b1, W2, b2, heavy, None, act, W1u)
    yq = orc.split_ffn(X, W1[:, perm], None if b1 is None else b1[perm], W2[perm, :], b2, inv[heavy], None, act,
                       None if W1u is None else W1u[:, perm])
    assert np.allclose(yq, y_exact, rtol=1e-12, atol=1e-12)


def test_split_weights_are_plain_gathers(rng):
    X, W1, W1u, b1, W2, b2 = _tiny(rng, m=9)
    sw = orc.split_weights(W1, b1, W2, [7, 2])
    assert np.array_equal(sw["U1"][:, 0], W1[:, 7]) and np.array_equal(sw["V1"][1], W2[2])
    assert list(sw["light"]) == [0, 1, 3, 4, 5, 6, 8]
    assert np.array_equal(sw["U2"][:, 2], W1[:, 3]) and np.array_equal(sw["V2"][6], W2[8])
    assert np.array_equal(sw["b1_light"], b1[sw["light"]])


# ---------------------------------------------------------------- model size
def test_param_reduction_matches_the_paper():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "param_reduction.txt")) if l[0] != "#" and l.strip()]
    heavy_pc, rank_pc, printed = (float(v) for v in rows[0])
    d, m, layers = 768, 3072, 12                    # BERT-base
    k = round(heavy_pc / 100 * m)
    r = round(rank_pc / 100 * min(d, m - k))
    ffn = orc.ffn_weight_params(d, m)
    split = orc.split_weight_params(d, m, k, r)
    assert ffn == 2 * d * m and split == 2 * (d * k + r * (d + m - k))
    attn = 4 * d * d
    # weights only, and with biases + LayerNorm + pooler counted: the printed figure lies between
    red_w = (ffn - split) / (ffn + attn)
    other = layers * (4 * d + m + d + 4 * d) + d * d + d
    red_all = layers * (ffn - split) / (layers * (ffn + attn) + other)
    assert red_all * 100 <= printed + 0.15 and printed - 0.15 <= red_w * 100
    assert abs(red_w * 100 - printed) < 0.5
    # k = d_ff with no light part is the dense FFN
    assert orc.split_weight_params(d, m, m, 0) == ffn
    assert orc.split_weight_params(64, 256, 16, 8, n_in=2) == 3 * (64 * 16 + 8 * (64 + 240))


def test_error_metrics():
    a = np.array([[3.0, 4.0]])
    assert orc.rel_frobenius(a, a) == 0
    assert abs(orc.rel_frobenius(a + np.array([[0.3, 0.4]]), a) - 0.1) < 1e-15
    assert abs(orc.normalised_max_abs(a + np.array([[0.0, -0.2]]), a) - 0.05) < 1e-15


# ---------------------------------------------------------------------------------------------
# Quantised split (Section 5.2): round-to-nearest, group size 128, 8 bits heavy / 3 bits light
# ---------------------------------------------------------------------------------------------
def test_rtn_error_bound_codes_and_constant_groups(rng):
    for bits in (3, 8):
        qmax = (1 << bits) - 1
        w = (rng.standard_normal((7, 300)) * 0.02).astype(np.float32)      # 2 full groups and a ragged one of 44
        w[3, 128:256] = 0.125                                               # a constant group
        q, scale, lo = orc.rtn_quantize_groups(w, bits)
        assert q.shape == w.shape and scale.shape == (7, 3) and lo.shape == (7, 3) and q.dtype == np.uint8
        assert q.max() <= qmax
        wd = orc.rtn_dequantize_groups(q, scale, lo)
        idx = np.arange(300) // 128
        # every value lies within half a step of its code (a few float32 ulps of slack for the division)
        assert np.all(np.abs(wd - w) <= 0.5 * scale[:, idx] * (1 + 1e-5) + 1e-12)
        # the grid spans the group exactly: the minimum gets code 0, the maximum the last code
        for g in range(3):
            seg, qs = w[:, 128 * g:128 * (g + 1)], q[:, 128 * g:128 * (g + 1)]
            live = scale[:, g] > 0
            assert np.all(qs[np.arange(7), seg.argmin(axis=1)] == 0)
            assert np.all(qs[np.arange(7), seg.argmax(axis=1)][live] == qmax)
            assert np.allclose(lo[:, g], seg.min(axis=1)) and np.allclose(scale[:, g] * qmax, seg.max(axis=1) - seg.min(axis=1), rtol=1e-6)
        # the constant group: scale 0, all codes 0, reproduced exactly
        assert scale[3, 1] == 0 and not q[3, 128:256].any() and np.all(wd[3, 128:256] == 0.125)


def test_rtn_values_on_the_grid_are_exact_and_rounding_is_to_nearest():
    # a group whose values sit on an 8-level grid with a power-of-two step: 3 bits reproduce it exactly
    base = np.float32(-0.25)
    step = np.float32(2.0 ** -4)
    levels = np.arange(128) % 8
    w = (base + levels * step).astype(np.float32)[None, :]
    q, scale, lo = orc.rtn_quantize_groups(w, 3)
    assert np.array_equal(q[0], levels) and scale[0, 0] == step and lo[0, 0] == base
    assert np.array_equal(orc.rtn_dequantize_groups(q, scale, lo)[0], w[0].astype(np.float64))
    # a value 0.4 of a step above a grid point rounds down, 0.6 rounds up
    w2 = w.copy()
    w2[0, 8] = base + np.float32(2.4) * step
    w2[0, 9] = base + np.float32(2.6) * step
    q2, _, _ = orc.rtn_quantize_groups(w2, 3)
    assert q2[0, 8] == 2 and q2[0, 9] == 3


def test_rtn_groups_are_independent_and_run_along_the_last_axis(rng):
    w = (rng.standard_normal((4, 256)) * 0.02).astype(np.float32)
    q0, s0, l0 = orc.rtn_quantize_groups(w, 3)
    w1 = w.copy()
    w1[2, 130] = 5.0                       # an outlier in row 2, second group
    q1, s1, l1 = orc.rtn_quantize_groups(w1, 3)
    same = np.ones((4, 2), dtype=bool)
    same[2, 1] = False
    assert np.array_equal(s1[same], s0[same]) and np.array_equal(l1[same], l0[same])
    assert np.array_equal(q1[:, :128], q0[:, :128]) and np.array_equal(q1[[0, 1, 3]], q0[[0, 1, 3]])
    assert s1[2, 1] > 10 * s0[2, 1]        # only that group's step widened
    # each row (output channel) has its own parameters: scaling one row scales only its own steps
    w2 = w.copy()
    w2[1] *= 4
    _, s2, _ = orc.rtn_quantize_groups(w2, 3)
    assert np.allclose(s2[1], 4 * s0[1]) and np.array_equal(s2[[0, 2, 3]], s0[[0, 2, 3]])


def test_quantize_split_axes_and_reassembly(rng):
    """U-type matrices are grouped along d per neuron, V-type along the part's neuron axis per output column;
    the heavy part gets 8 bits, the light part 3; reassembly puts every neuron back in its place."""
    d, m = 160, 300
    W1 = (rng.standard_normal((d, m)) * 0.02).astype(np.float32)
    W2 = (rng.standard_normal((m, d)) * 0.02).astype(np.float32)
    heavy = np.sort(rng.choice(m, 140, replace=False))
    Q = orc.quantize_split(W1, W2, heavy)
    ml = m - 140
    assert Q["U1"][0].shape == (140, d) and Q["U1"][1].shape == (140, 2)         # ceil(160 / 128) groups along d
    assert Q["V1"][0].shape == (d, 140) and Q["V1"][1].shape == (d, 2)           # ceil(140 / 128) groups along heavy neurons
    assert Q["U2"][0].shape == (ml, d) and Q["V2"][1].shape == (d, 2)
    assert Q["U1"][0].max() > 7 and Q["V1"][0].max() > 7 and Q["U2"][0].max() <= 7 and Q["V2"][0].max() <= 7
    W1q, W2q, _ = orc.dequantized_weights(Q, d, m)
    light = Q["light"]
    # 8-bit steps are 255/7 times finer than 3-bit ones on the same kind of data
    e_h = np.abs(W1q[:, heavy] - W1[:, heavy]).max()
    e_l = np.abs(W1q[:, light] - W1[:, light]).max()
    assert e_h < e_l / 10
    step_u2 = Q["U2"][1]
    assert np.all(np.abs(W1q[:, light].T - W1[:, light].T) <= 0.5 * step_u2[:, np.arange(d) // 128] * (1 + 1e-5) + 1e-12)
    step_v1 = Q["V1"][1]
    assert np.all(np.abs(W2q[heavy, :].T - W2[heavy, :].T) <= 0.5 * step_v1[:, np.arange(140) // 128] * (1 + 1e-5) + 1e-12)
    # the V groups follow the part's own neuron order: rows of V[heavy] number 128.. form the second group
    assert np.allclose(Q["V1"][2][:, 1], W2[heavy[128:], :].min(axis=0))
    assert np.allclose(Q["U1"][2][:, 1], W1[128:, heavy].min(axis=0))


def test_quant_split_ffn_is_the_dense_ffn_of_the_dequantised_weights_and_converges_with_bits(rng):
    d, m, T = 96, 200, 9
    W1 = rng.standard_normal((d, m)) * 0.05
    W2 = rng.standard_normal((m, d)) * 0.05
    b1 = rng.standard_normal(m) * 0.1
    b2 = rng.standard_normal(d) * 0.1
    X = rng.standard_normal((T, d))
    heavy = np.sort(rng.choice(m, 30, replace=False))
    ref = orc.dense_ffn(X, W1.astype(np.float32), b1, W2.astype(np.float32), b2, "gelu_erf")
    errs = []
    for bl in (2, 3, 4, 6, 8):
        Q = orc.quantize_split(W1, W2, heavy, bits_heavy=8, bits_light=bl)
        Y = orc.quant_split_ffn(X, b1, b2, Q, d, m, "gelu_erf")
        # written out with explicit sums over the two parts (Eq. 2), neuron by neuron
        W1q, W2q, _ = orc.dequantized_weights(Q, d, m)
        Y2 = np.tile(b2, (T, 1))
        for j in range(m):
            Y2 += np.outer(orc.gelu_erf(X @ W1q[:, j] + b1[j]), W2q[j, :])
        assert np.allclose(Y, Y2, rtol=1e-12, atol=1e-12)
        errs.append(orc.rel_frobenius(Y, ref))
    assert all(errs[i + 1] < 0.75 * errs[i] for i in range(len(errs) - 1))     # about a factor two per bit
    assert errs[-1] < 0.02
    # SwiGLU: the up projection is quantised like the gate
    W1u = rng.standard_normal((d, m)) * 0.05
    Q = orc.quantize_split(W1, W2, heavy, W1u=W1u)
    W1q, W2q, W1uq = orc.dequantized_weights(Q, d, m)
    Y = orc.quant_split_ffn(X, None, None, Q, d, m, "swiglu")
    assert np.allclose(Y, (orc.silu(X @ W1q) * (X @ W1uq)) @ W2q, rtol=1e-12, atol=1e-14)


def test_quant_weight_bytes_formula_counts_codes_and_group_parameters():
    d, m, k = 5120, 20480, 1024
    got = orc.quant_weight_bytes(d, m, k)
    ml = m - k
    codes = (2 * k * d * 8 + 2 * ml * d * 3) / 8
    params = 8 * (k * 40 + d * 8 + ml * 40 + d * 152)
    assert got == codes + params
    # 3.25-3.5 bits per weight overall at 5 % heavy: about a fifth of the bf16 layer
    assert 0.21 < got / (2 * 2 * d * m) < 0.24
    assert orc.quant_weight_bytes(256, 1024, 0) == (2 * 1024 * 256 * 3) / 8 + 8 * (1024 * 2 + 256 * 8)


# ---------------------------------------------------------------- the block around the FFN
def test_layer_norm_moments_and_invariances(rng):
    x = rng.normal(size=(7, 24)) * 3 + 1.5
    y = orc.layer_norm(x, np.ones(24), np.zeros(24), 0.0)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-12) and np.allclose((y ** 2).mean(axis=1), 1, atol=1e-12)
    assert np.allclose(orc.layer_norm(x + 5.0, np.ones(24), np.zeros(24), 0.0), y, atol=1e-12)      # shift
    assert np.allclose(orc.layer_norm(2.0 * x, np.ones(24), np.zeros(24), 0.0), y, atol=1e-12)      # scale (eps = 0)
    g, b = rng.normal(size=24), rng.normal(size=24)
    assert np.allclose(orc.layer_norm(x, g, b, 0.0), y * g + b, atol=1e-12)
    # eps enters under the root: a row of variance v is divided by sqrt(v + eps)
    v = ((x - x.mean(axis=1, keepdims=True)) ** 2).mean(axis=1)
    assert np.allclose(orc.layer_norm(x, np.ones(24), np.zeros(24), 0.3), y * np.sqrt(v / (v + 0.3))[:, None], atol=1e-12)


def test_multi_head_attention_against_token_loops_and_closed_forms(rng):
    batch, seq, heads, dh = 2, 5, 3, 4
    d = heads * dh
    X = rng.normal(size=(batch * seq, d))
    Wqkv, bqkv = rng.normal(size=(d, 3 * d)) * 0.4, rng.normal(size=3 * d) * 0.1
    Wo, bo = rng.normal(size=(d, d)) * 0.4, rng.normal(size=d) * 0.1
    out = orc.multi_head_attention(X, Wqkv, bqkv, Wo, bo, batch, seq, heads)
    # the definition, one query token and one head at a time
    ref = np.zeros((batch * seq, d))
    for b in range(batch):
        for i in range(seq):
            t = b * seq + i
            for h in range(heads):
                q = X[t] @ Wqkv[:, h * dh:(h + 1) * dh] + bqkv[h * dh:(h + 1) * dh]
                w = np.zeros(seq)
                vs = []
                for j in range(seq):
                    u = b * seq + j
                    k = X[u] @ Wqkv[:, d + h * dh:d + (h + 1) * dh] + bqkv[d + h * dh:d + (h + 1) * dh]
                    vs.append(X[u] @ Wqkv[:, 2 * d + h * dh:2 * d + (h + 1) * dh] + bqkv[2 * d + h * dh:2 * d + (h + 1) * dh])
                    w[j] = math.exp(float(q @ k) / math.sqrt(dh))
                ref[t, h * dh:(h + 1) * dh] = sum(wj * vj for wj, vj in zip(w, vs)) / w.sum()
    assert np.allclose(out, ref @ Wo + bo, atol=1e-12)
    # Q = 0: uniform attention, every token gets the mean of its sequence's V
    W0, b0 = Wqkv.copy(), bqkv.copy()
    W0[:, :d] = 0
    b0[:d] = 0
    V = X @ W0[:, 2 * d:] + b0[2 * d:]
    mean_v = np.repeat(V.reshape(batch, seq, d).mean(axis=1), seq, axis=0)
    assert np.allclose(orc.multi_head_attention(X, W0, b0, Wo, bo, batch, seq, heads), mean_v @ Wo + bo, atol=1e-12)
    # V constant (Wv = 0): the softmax weights sum to one, so the output is bv Wo + bo whatever Q and K are
    W1 = Wqkv.copy()
    W1[:, 2 * d:] = 0
    assert np.allclose(orc.multi_head_attention(X, W1, bqkv, Wo, bo, batch, seq, heads),
                       np.tile(bqkv[2 * d:] @ Wo + bo, (batch * seq, 1)), atol=1e-12)
    # sequences do not see one another; tokens of a sequence are exchangeable
    X2 = X.copy()
    X2[seq:] = rng.normal(size=(seq, d))
    assert np.allclose(orc.multi_head_attention(X2, Wqkv, bqkv, Wo, bo, batch, seq, heads)[:seq], out[:seq], atol=1e-12)
    perm = rng.permutation(seq)
    Xp = X.copy()
    Xp[:seq] = X[:seq][perm]
    assert np.allclose(orc.multi_head_attention(Xp, Wqkv, bqkv, Wo, bo, batch, seq, heads)[:seq], out[:seq][perm], atol=1e-12)


def test_encoder_layer_composition(rng):
    batch, seq, heads, d, m = 2, 4, 2, 8, 20
    X = rng.normal(size=(batch * seq, d))
    attn = (rng.normal(size=(d, 3 * d)) * 0.3, rng.normal(size=3 * d) * 0.1, rng.normal(size=(d, d)) * 0.3, rng.normal(size=d) * 0.1)
    ln1, ln2 = (rng.normal(size=d), rng.normal(size=d)), (rng.normal(size=d), rng.normal(size=d))
    W1, b1, W2, b2 = rng.normal(size=(d, m)), rng.normal(size=m), rng.normal(size=(m, d)), rng.normal(size=d)
    ffn = lambda Z: orc.dense_ffn(Z, W1, b1, W2, b2, orc.ACT_GELU_ERF)
    Y = orc.encoder_layer(X, attn, ln1, ln2, 1e-5, batch, seq, heads, ffn)
    A = orc.multi_head_attention(X, *attn, batch, seq, heads)
    X1 = orc.layer_norm(X + A, *ln1, 1e-5)
    assert np.allclose(Y, orc.layer_norm(X1 + ffn(X1), *ln2, 1e-5), atol=1e-12)
    # no attention, no FFN: two LayerNorms of X in closed form (the second one of an already normalised row)
    zero_attn = (np.zeros((d, 3 * d)), np.zeros(3 * d), np.zeros((d, d)), np.zeros(d))
    one = (np.ones(d), np.zeros(d))
    Y0 = orc.encoder_layer(X, zero_attn, one, one, 0.0, batch, seq, heads, lambda Z: np.zeros_like(Z))
    xc = X - X.mean(axis=1, keepdims=True)
    assert np.allclose(Y0, xc / np.sqrt((xc ** 2).mean(axis=1, keepdims=True)), atol=1e-12)
