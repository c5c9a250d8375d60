"""Pins for the CPU oracle: closed forms, invariants, library special cases, brute force.

The paper prints no numeric worked example for any of the five programs, so the
oracle is pinned to what the mathematics fixes: hand-worked closed forms
(tests/golden/), special cases that collapse to a numpy/scipy routine, the
algebraic equalities of Table 1 that the fused kernels rely on (factor motion,
reduce refinement along K, repair fusion, MatMul reassociation and factoring),
and the M1/M2 attention forms of Figure 4 written out in the test and compared
with the oracle's M0.  No test calls the CUDA path.
"""
import itertools

import numpy as np
import pytest
from scipy.special import expit, softmax

import oracle
from conftest import load_golden

RNG = np.random.default_rng(12345)
TOL = dict(rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------
# Program 1: RMSNorm + matmul
# ----------------------------------------------------------------------------
def test_rmsnorm_hand_example():
    g = load_golden("rmsnorm_hand_example.txt")
    x = np.array([g["x"]])
    y = oracle.rmsnorm_matmul(x, np.ones(2), np.eye(2), 0.0)
    np.testing.assert_allclose(y[0], g["y"], **TOL)
    W = np.array([[1.0, 2.0, 3.0], [4.0, 5.0, 6.0]])
    y2 = oracle.rmsnorm_matmul(x, np.array([2.0, 0.5]), W, 0.0)
    np.testing.assert_allclose(y2[0], g["y2"], **TOL)
    y3 = oracle.rmsnorm_matmul(x, np.ones(2), np.eye(2), 3.5)  # eps goes on the MEAN, inside the sqrt
    np.testing.assert_allclose(y3[0], g["y3"], **TOL)


def test_rmsnorm_constant_rows_closed_form():
    # X == c, gamma == 1, eps == 0  =>  xn == sign(c), y_n = sign(c) * sum_k W[k,n]
    K, N = 7, 5
    W = RNG.standard_normal((K, N))
    for c in (2.5, -0.3):
        y = oracle.rmsnorm_matmul(np.full((3, K), c), np.ones(K), W, 0.0)
        np.testing.assert_allclose(y, np.sign(c) * np.tile(W.sum(0), (3, 1)), **TOL)
    # with eps: r = 1/sqrt(c^2 + eps) exactly (mean of a constant row is c^2, whatever K is)
    c, eps = 1.5, 0.75
    y = oracle.rmsnorm_matmul(np.full((1, K), c), np.ones(K), W, eps)
    np.testing.assert_allclose(y[0], c / np.sqrt(c * c + eps) * W.sum(0), **TOL)


def test_rmsnorm_unit_rms_rows_reduce_to_library_matmul():
    # rows with entries +-1 have mean square 1: r == 1 at eps == 0, so Y == (X*gamma) @ W (numpy)
    M, K, N = 4, 9, 6
    X = RNG.choice([-1.0, 1.0], size=(M, K))
    gamma = RNG.standard_normal(K)
    W = RNG.standard_normal((K, N))
    np.testing.assert_allclose(oracle.rmsnorm_matmul(X, gamma, W, 0.0), (X * gamma) @ W, **TOL)


def test_rmsnorm_zero_row_and_scale_invariance():
    K, N = 8, 3
    W = RNG.standard_normal((K, N))
    gamma = RNG.standard_normal(K)
    X = RNG.standard_normal((2, K))
    X[1] = 0.0
    y = oracle.rmsnorm_matmul(X, gamma, W, 1e-6)
    assert np.all(np.isfinite(y)) and np.all(y[1] == 0.0)
    # eps == 0: scaling a row by t > 0 leaves Y unchanged
    Xs = X.copy(); Xs[0] *= 37.0
    np.testing.assert_allclose(oracle.rmsnorm_matmul(Xs[:1], gamma, W, 0.0),
                               oracle.rmsnorm_matmul(X[:1], gamma, W, 0.0), **TOL)
    # gamma == 1: mean_k xn^2 == ms / (ms + eps)
    eps = 0.3
    xn = oracle.rmsnorm_matmul(X[:1], np.ones(K), np.eye(K), eps)[0]
    ms = np.mean(X[0] ** 2)
    np.testing.assert_allclose(np.mean(xn ** 2), ms / (ms + eps), **TOL)


def test_rmsnorm_factor_motion_table1():
    # MatMul(X o a, W) == MatMul(X, W) o a when a is invariant along K (Table 1, factor motion):
    # the per-row factor r moves to the epilogue; gamma varies along K and must stay inside.
    M, K, N = 3, 4, 2
    X = RNG.standard_normal((M, K)); gamma = RNG.standard_normal(K) + 2.0
    W = RNG.standard_normal((K, N)); eps = 1e-3
    r = 1.0 / np.sqrt((X ** 2).mean(1) + eps)
    y = oracle.rmsnorm_matmul(X, gamma, W, eps)
    np.testing.assert_allclose(y, r[:, None] * ((X * gamma) @ W), **TOL)
    np.testing.assert_allclose(y, r[:, None] * (X @ (gamma[:, None] * W)), **TOL)
    # negative check: gamma cannot be pulled past the contraction
    assert not np.allclose(y, r[:, None] * (X @ W) * gamma[:N])
    # Reduce refinement along K + product fusion: per-chunk partial sum-of-squares and partial
    # products, combined by +, equal the whole (Table 1, Reduce K-refinement; MatMul NK refinement)
    for split in (1, 2, 3):
        ss = (X[:, :split] ** 2).sum(1) + (X[:, split:] ** 2).sum(1)
        part = (X[:, :split] * gamma[:split]) @ W[:split] + (X[:, split:] * gamma[split:]) @ W[split:]
        np.testing.assert_allclose(y, part / np.sqrt(ss / K + eps)[:, None], **TOL)


# ----------------------------------------------------------------------------
# Program 2: gated MLP
# ----------------------------------------------------------------------------
def test_layernorm_matmul_pins():
    """LayerNorm+GEMM oracle: library special case (numpy mean/var + matmul), hand example, invariants
    (shift and positive-scale invariance at eps=0, beta enters as beta@W, constant rows give beta@W), and the
    fused form the kernel uses: r * ((x - mu) * gamma) @ W + beta @ W."""
    M, K, N = 4, 12, 5
    X = RNG.standard_normal((M, K)) + 0.7; g = 1 + 0.1 * RNG.standard_normal(K); b = 0.2 * RNG.standard_normal(K)
    W = RNG.standard_normal((K, N)); eps = 1e-5
    y = oracle.layernorm_matmul(X, g, b, W, eps)
    mu = X.mean(1, keepdims=True); var = X.var(1, keepdims=True)        # numpy: biased variance
    ref = ((X - mu) / np.sqrt(var + eps) * g + b) @ W
    np.testing.assert_allclose(y, ref, **TOL)
    # hand example: x = [1, 3] -> mu = 2, var = 1, eps = 0: xn = [-1, 1]; gamma = [2, 3], beta = [10, 20], W = I
    yh = oracle.layernorm_matmul(np.array([[1.0, 3.0]]), np.array([2.0, 3.0]), np.array([10.0, 20.0]), np.eye(2), 0.0)
    np.testing.assert_allclose(yh, [[8.0, 23.0]], **TOL)
    # eps = 0: adding a constant to a row, or scaling it by t > 0, changes nothing
    y0 = oracle.layernorm_matmul(X, g, b, W, 0.0)
    np.testing.assert_allclose(oracle.layernorm_matmul(X + 5.0, g, b, W, 0.0), y0, rtol=1e-9, atol=1e-9)
    np.testing.assert_allclose(oracle.layernorm_matmul(3.5 * X, g, b, W, 0.0), y0, rtol=1e-9, atol=1e-9)
    # beta is additive through the projection; a constant row has no deviation, so its output is beta @ W
    np.testing.assert_allclose(y - oracle.layernorm_matmul(X, g, 0 * b, W, eps), np.tile(b @ W, (M, 1)), **TOL)
    np.testing.assert_allclose(oracle.layernorm_matmul(np.full((2, K), 4.0), g, b, W, eps), np.tile(b @ W, (2, 1)), **TOL)
    # factor motion: the inverse standard deviation scales the finished projection; the mean does NOT move out
    r = 1 / np.sqrt(var + eps)
    np.testing.assert_allclose(r * (((X - mu) * g) @ W) + b @ W, y, **TOL)
    assert not np.allclose(r * ((X * g) @ W) + b @ W, y, atol=1e-3)
    # mean subtracted, unit variance: the normalised rows (gamma=1, beta=0, W=I) have mean 0 and mean square var/(var+eps)
    z = oracle.layernorm_matmul(X, np.ones(K), np.zeros(K), np.eye(K), eps)
    np.testing.assert_allclose(z.mean(1), 0, atol=1e-12)
    np.testing.assert_allclose((z ** 2).mean(1), (var / (var + eps))[:, 0], **TOL)


def test_silu_golden_values_through_one_hot_rows():
    g = load_golden("silu_constants.txt")
    # X one-hot picks row k of the weights: y_n = SiLU(Wg[k,n]) * Wu[k,n]
    Wg = np.array([[1.0, -1.0, 0.0, g["silu_argmin"][0]], [9.0, 9.0, 9.0, 9.0]])
    Wu = np.array([[1.0, 1.0, 5.0, 1.0], [9.0, 9.0, 9.0, 9.0]])
    y = oracle.gated_mlp(np.array([[1.0, 0.0]]), Wg, Wu)[0]
    np.testing.assert_allclose(y[0], g["silu_at_1"][0], **TOL)
    np.testing.assert_allclose(y[1], g["silu_at_minus_1"][0], **TOL)
    assert y[2] == 0.0
    np.testing.assert_allclose(y[3], g["silu_min"][0], rtol=0, atol=1e-13)


def test_gated_mlp_against_scipy_expit_and_numpy_matmul():
    M, K, N = 3, 5, 7
    X = RNG.standard_normal((M, K)); Wg = RNG.standard_normal((K, N)); Wu = RNG.standard_normal((K, N))
    G, U = X @ Wg, X @ Wu
    np.testing.assert_allclose(oracle.gated_mlp(X, Wg, Wu), G * expit(G) * U, **TOL)
    # which matmul is gated: swapping the weights changes the result
    assert not np.allclose(oracle.gated_mlp(X, Wu, Wg), oracle.gated_mlp(X, Wg, Wu))


def test_gated_mlp_odd_part_identity():
    # SiLU(z) - SiLU(-z) = z  =>  Y(X,Wg,Wu) - Y(X,-Wg,Wu) = (X@Wg) * (X@Wu): two library matmuls
    M, K, N = 4, 6, 5
    X = RNG.standard_normal((M, K)); Wg = RNG.standard_normal((K, N)); Wu = RNG.standard_normal((K, N))
    d = oracle.gated_mlp(X, Wg, Wu) - oracle.gated_mlp(X, -Wg, Wu)
    np.testing.assert_allclose(d, (X @ Wg) * (X @ Wu), **TOL)


def test_gated_mlp_saturation_and_lower_bound():
    g = load_golden("silu_constants.txt")
    y = oracle.gated_mlp(np.array([[1.0]]), np.array([[1e4, -1e4, 800.0, -800.0]]), np.ones((1, 4)))[0]
    assert np.all(np.isfinite(y))
    np.testing.assert_allclose(y, [1e4, 0.0, 800.0, 0.0], rtol=1e-12, atol=1e-300)
    X = RNG.standard_normal((6, 4)); Wg = 3 * RNG.standard_normal((4, 50)); Wu = np.abs(RNG.standard_normal((4, 50)))
    U = X @ Wu
    ratio = (oracle.gated_mlp(X, Wg, Wu) / U)[U > 1e-3]
    assert ratio.min() >= g["silu_min"][0] - 1e-12


def test_gated_mlp_column_combination_and_split_k():
    M, K, N = 2, 6, 8
    X = RNG.standard_normal((M, K)); Wg = RNG.standard_normal((K, N)); Wu = RNG.standard_normal((K, N))
    y = oracle.gated_mlp(X, Wg, Wu)
    # Combination over N (Table 1, MatMul N refinement + pointwise propagation)
    parts = [oracle.gated_mlp(X, Wg[:, a:b], Wu[:, a:b]) for a, b in ((0, 3), (3, 4), (4, 8))]
    np.testing.assert_allclose(np.concatenate(parts, 1), y, **TOL)
    # split-K: Reduce_+ must precede the nonlinear pointwise op ...
    G = X[:, :2] @ Wg[:2] + X[:, 2:] @ Wg[2:]; U = X[:, :2] @ Wu[:2] + X[:, 2:] @ Wu[2:]
    np.testing.assert_allclose(G * expit(G) * U, y, **TOL)
    # ... and SiLU-then-reduce is NOT equal
    wrong = oracle.gated_mlp(X[:, :2], Wg[:2], Wu[:2]) + oracle.gated_mlp(X[:, 2:], Wg[2:], Wu[2:])
    assert not np.allclose(wrong, y)


# ----------------------------------------------------------------------------
# Program 2b: RMSNorm fused into the gated MLP
# ----------------------------------------------------------------------------
def test_rmsnorm_gated_mlp_unit_rms_rows_library_case():
    # rows of +-1 have mean square 1: at eps == 0 the normalisation is the identity and
    # Y == G*expit(G)*U with G = (X*gamma)@Wg, U = (X*gamma)@Wu (numpy + scipy only)
    M, K, N = 3, 8, 5
    X = RNG.choice([-1.0, 1.0], size=(M, K)); gamma = RNG.standard_normal(K)
    Wg = RNG.standard_normal((K, N)); Wu = RNG.standard_normal((K, N))
    G, U = (X * gamma) @ Wg, (X * gamma) @ Wu
    np.testing.assert_allclose(oracle.rmsnorm_gated_mlp(X, gamma, Wg, Wu, 0.0), G * expit(G) * U, **TOL)


def test_rmsnorm_gated_mlp_factor_motion_after_each_projection():
    # Section 7.2: (s (.) X) W == s (.) (X W): the row factor applied after BOTH projections
    M, K, N = 4, 6, 7
    X = RNG.standard_normal((M, K)); gamma = 1.0 + 0.1 * RNG.standard_normal(K)
    Wg = RNG.standard_normal((K, N)); Wu = RNG.standard_normal((K, N)); eps = 1e-2
    r = 1.0 / np.sqrt((X ** 2).mean(1, keepdims=True) + eps)
    G, U = r * ((X * gamma) @ Wg), r * ((X * gamma) @ Wu)
    y = oracle.rmsnorm_gated_mlp(X, gamma, Wg, Wu, eps)
    np.testing.assert_allclose(y, G * expit(G) * U, **TOL)
    # ties to the pinned single-projection oracle: the two normalised projections, then the gate
    g1 = oracle.rmsnorm_matmul(X, gamma, Wg, eps); u1 = oracle.rmsnorm_matmul(X, gamma, Wu, eps)
    np.testing.assert_allclose(y, g1 * expit(g1) * u1, **TOL)
    # the row factor must NOT be applied once to the product (SiLU is not homogeneous)
    G0, U0 = (X * gamma) @ Wg, (X * gamma) @ Wu
    assert not np.allclose(y, r * (G0 * expit(G0) * U0))


def test_rmsnorm_gated_mlp_invariants():
    K, N = 8, 4
    X = RNG.standard_normal((2, K)); X[1] = 0.0
    gamma = RNG.standard_normal(K); Wg = RNG.standard_normal((K, N)); Wu = RNG.standard_normal((K, N))
    y = oracle.rmsnorm_gated_mlp(X, gamma, Wg, Wu, 1e-6)
    assert np.all(np.isfinite(y)) and np.all(y[1] == 0.0)          # zero row
    Xs = X.copy(); Xs[0] *= 13.0                                     # eps == 0: row scale invariance
    np.testing.assert_allclose(oracle.rmsnorm_gated_mlp(Xs[:1], gamma, Wg, Wu, 0.0),
                               oracle.rmsnorm_gated_mlp(X[:1], gamma, Wg, Wu, 0.0), **TOL)
    assert not np.allclose(oracle.rmsnorm_gated_mlp(X[:1], gamma, Wu, Wg, 0.0),
                           oracle.rmsnorm_gated_mlp(X[:1], gamma, Wg, Wu, 0.0))  # which projection is gated


# ----------------------------------------------------------------------------
# Program 3: GQA decode attention (M0 of Figure 4, one query row)
# ----------------------------------------------------------------------------
def _m2_rolling(q, K, V, scale, tile_bounds):
    """Figure 4, M2: rolling reducer over key tiles with state <max, sum, value>, identity init."""
    mx, sm, val = -np.inf, 0.0, np.zeros(V.shape[1])
    for a, b in tile_bounds:
        scaled = (K[a:b] @ q) * scale
        block_max = scaled.max()
        next_max = max(mx, block_max)
        rescale = 0.0 if mx == -np.inf else np.exp(mx - next_max)
        weights = np.exp(scaled - next_max)
        sm = rescale * sm + weights.sum()
        val = rescale * val + weights @ V[a:b]
        mx = next_max
    return val / sm


def _m1_dependent(q, K, V, scale, tile_bounds):
    """Figure 4, M1: three parallel reductions over the key tiles (max, then sum and value)."""
    scaled = [(K[a:b] @ q) * scale for a, b in tile_bounds]
    maximum = max(s.max() for s in scaled)
    weights = [np.exp(s - maximum) for s in scaled]
    normalizer = sum(w.sum() for w in weights)
    numerator = sum(w @ V[a:b] for w, (a, b) in zip(weights, tile_bounds))
    return numerator / normalizer


def _splits(L):
    """All 2^(L-1) partitions of range(L) into contiguous tiles."""
    for cuts in itertools.product([0, 1], repeat=L - 1):
        edges = [0] + [i + 1 for i, c in enumerate(cuts) if c] + [L]
        yield list(zip(edges[:-1], edges[1:]))


def test_decode_closed_form_log_weights():
    g = load_golden("softmax_log_weights.txt")
    Q = np.array([[[1.0, 0.0]]])
    K = np.array([[[[0.0, 7.0], [np.log(2.0), 7.0], [np.log(3.0), 7.0]]]])
    V = np.array([[[[6.0, 0.0], [0.0, 6.0], [6.0, 6.0]]]])
    np.testing.assert_allclose(oracle.gqa_decode(Q, K, V, 1.0)[0, 0], g["o"], **TOL)
    # scale multiplies the logits: with scale 2 the weights become [1, 4, 9] / 14
    o2 = oracle.gqa_decode(Q, K, V, 2.0)[0, 0]
    np.testing.assert_allclose(o2, (1 * V[0, 0, 0] + 4 * V[0, 0, 1] + 9 * V[0, 0, 2]) / 14.0, **TOL)


def test_decode_degenerate_cases():
    B, Hq, Hkv, L, D = 2, 4, 2, 6, 3
    Q = RNG.standard_normal((B, Hq, D)); V = RNG.standard_normal((B, Hkv, L, D))
    o = oracle.gqa_decode(Q, np.zeros((B, Hkv, L, D)), V, 0.7)       # K == 0 -> uniform weights
    for h in range(Hq):
        np.testing.assert_allclose(o[:, h], V[:, h // 2].mean(1), **TOL)
    K = RNG.standard_normal((B, Hkv, 1, D))
    o1 = oracle.gqa_decode(Q, K, V[:, :, :1], 0.7)                   # L == 1 -> o = v_0 exactly
    for h in range(Hq):
        assert np.array_equal(o1[:, h], V[:, h // 2, 0])


def test_decode_against_scipy_softmax_and_head_mapping():
    B, Hq, Hkv, L, D = 2, 6, 3, 7, 4
    Q = RNG.standard_normal((B, Hq, D)); K = RNG.standard_normal((B, Hkv, L, D)); V = RNG.standard_normal((B, Hkv, L, D))
    scale = 0.37
    o = oracle.gqa_decode(Q, K, V, scale)
    # GQA == MHA on repeat_interleave-expanded K, V (consecutive query heads share a kv head)
    Kx, Vx = np.repeat(K, Hq // Hkv, axis=1), np.repeat(V, Hq // Hkv, axis=1)
    ref = np.einsum("bhl,bhld->bhd", softmax(np.einsum("bhd,bhld->bhl", Q, Kx) * scale, axis=-1), Vx)
    np.testing.assert_allclose(o, ref, **TOL)
    np.testing.assert_allclose(oracle.gqa_decode(Q, Kx, Vx, scale), o, **TOL)
    # convexity: each output lies inside the range of the values it averages
    for h in range(Hq):
        assert np.all(o[:, h] <= V[:, h // 2].max(1) + 1e-12) and np.all(o[:, h] >= V[:, h // 2].min(1) - 1e-12)
    # joint permutation of (k_j, v_j) leaves the output unchanged
    perm = RNG.permutation(L)
    np.testing.assert_allclose(oracle.gqa_decode(Q, K[:, :, perm], V[:, :, perm], scale), o, **TOL)


def test_decode_window_and_sinks():
    """Sliding window + sinks in decode: scipy softmax over the explicitly gathered visible keys; no window (0 or
    >= L) is the plain program bit for bit; window 1 returns the last value row; sinks add exactly the first keys."""
    B, Hq, Hkv, L, D = 2, 4, 2, 11, 3
    Q = RNG.standard_normal((B, Hq, D)); K = RNG.standard_normal((B, Hkv, L, D)); V = RNG.standard_normal((B, Hkv, L, D))
    scale = 0.45
    for window, sinks in [(4, 0), (4, 2), (1, 0), (1, 3), (10, 1), (5, 9)]:
        o = oracle.gqa_decode_window(Q, K, V, scale, window, sinks)
        idx = [j for j in range(L) if j >= L - window or j < sinks]
        Kx, Vx = np.repeat(K[:, :, idx], Hq // Hkv, axis=1), np.repeat(V[:, :, idx], Hq // Hkv, axis=1)
        ref = np.einsum("bhl,bhld->bhd", softmax(np.einsum("bhd,bhld->bhl", Q, Kx) * scale, axis=-1), Vx)
        np.testing.assert_allclose(o, ref, **TOL)
    plain = oracle.gqa_decode(Q, K, V, scale)
    assert np.array_equal(oracle.gqa_decode_window(Q, K, V, scale, 0, 3), plain)
    assert np.array_equal(oracle.gqa_decode_window(Q, K, V, scale, L, 3), plain)
    assert np.array_equal(oracle.gqa_decode_window(Q, K, V, scale, L + 7, 0), plain)
    o1 = oracle.gqa_decode_window(Q, K, V, scale, 1, 0)
    for h in range(Hq):
        assert np.array_equal(o1[:, h], V[:, h // 2, L - 1])


def test_decode_varlen_against_scipy_softmax_per_entry():
    """Per-sequence lengths: entry b is plain softmax attention over its first len_b keys (library routines on the
    truncated tensors), padding rows are never read (NaN there changes nothing), an entry without keys is zero,
    lengths are clamped to [0, L], and a length-1 entry returns v_0."""
    B, Hq, Hkv, L, D = 5, 4, 2, 9, 3
    Q = RNG.standard_normal((B, Hq, D)); K = RNG.standard_normal((B, Hkv, L, D)); V = RNG.standard_normal((B, Hkv, L, D))
    lens = np.array([9, 1, 0, 4, 7], dtype=np.int32)
    scale = 0.41
    Kp, Vp = K.copy(), V.copy()
    for b in range(B):
        Kp[b, :, lens[b]:] = np.nan
        Vp[b, :, lens[b]:] = np.nan
    o = oracle.gqa_decode_varlen(Q, Kp, Vp, lens, scale)
    assert np.all(np.isfinite(o))
    for b in range(B):
        n = lens[b]
        if n == 0:
            assert np.array_equal(o[b], np.zeros((Hq, D)))
            continue
        Kx, Vx = np.repeat(K[b, :, :n], Hq // Hkv, axis=0), np.repeat(V[b, :, :n], Hq // Hkv, axis=0)
        ref = np.einsum("hl,hld->hd", softmax(np.einsum("hd,hld->hl", Q[b], Kx) * scale, axis=-1), Vx)
        np.testing.assert_allclose(o[b], ref, **TOL)
    for h in range(Hq):
        assert np.array_equal(o[1, h], V[1, h // 2, 0])           # one key: the output is that key's value row
    # all lengths equal to L: the uniform program, bit for bit (same routine on the same rows)
    full = np.full(B, L, dtype=np.int32)
    assert np.array_equal(oracle.gqa_decode_varlen(Q, K, V, full, scale), oracle.gqa_decode(Q, K, V, scale))
    # clamping: a length beyond L means L, a negative one means 0
    odd = np.array([L + 50, -2, 3, L, 0], dtype=np.int32)
    oc = oracle.gqa_decode_varlen(Q, K, V, odd, scale)
    ok = oracle.gqa_decode_varlen(Q, K, V, np.array([L, 0, 3, L, 0], dtype=np.int32), scale)
    assert np.array_equal(oc, ok)


def test_decode_max_shift_invariance():
    # adding u to every key with q.u = c shifts every logit by c*scale; softmax is invariant
    # (the basis of the repair h(c,s,s') = c*exp(s-s'), Section 4.2)
    L, D = 9, 5
    Q = RNG.standard_normal((1, 1, D)); K = RNG.standard_normal((1, 1, L, D)); V = RNG.standard_normal((1, 1, L, D))
    o = oracle.gqa_decode(Q, K, V, 1.3)
    q = Q[0, 0]
    for c in (-3.0, 5.0, 40.0):
        u = c * q / (q @ q)
        np.testing.assert_allclose(oracle.gqa_decode(Q, K + u, V, 1.3), o, rtol=1e-10, atol=1e-10)


def test_decode_rolling_m2_and_dependent_m1_equal_m0():
    D, scale = 4, 0.9
    for L in (1, 2, 5, 8):
        Q = RNG.standard_normal((1, 1, D)); K = 2 * RNG.standard_normal((1, 1, L, D)); V = RNG.standard_normal((1, 1, L, D))
        o = oracle.gqa_decode(Q, K, V, scale)[0, 0]
        for tiles in _splits(L):
            np.testing.assert_allclose(_m2_rolling(Q[0, 0], K[0, 0], V[0, 0], scale, tiles), o, rtol=1e-11, atol=1e-12)
            np.testing.assert_allclose(_m1_dependent(Q[0, 0], K[0, 0], V[0, 0], scale, tiles), o, rtol=1e-11, atol=1e-12)


def test_decode_partial_state_merge_is_associative():
    # split-KV: partial <m, l, o> states over arbitrary partitions merge to the whole
    # (Reduce K-refinement needs an associative reducer with identity init, Section 4.1)
    L, D, scale = 12, 3, 1.1
    q = RNG.standard_normal(D); K = RNG.standard_normal((L, D)); V = RNG.standard_normal((L, D))
    o = oracle.gqa_decode(q[None, None], K[None, None], V[None, None], scale)[0, 0]

    def partial(a, b):
        s = (K[a:b] @ q) * scale
        m = s.max(); w = np.exp(s - m)
        return m, w.sum(), w @ V[a:b]

    def merge(x, y):
        m = max(x[0], y[0]); ax, ay = np.exp(x[0] - m), np.exp(y[0] - m)
        return m, ax * x[1] + ay * y[1], ax * x[2] + ay * y[2]

    for edges in ([0, 5, 12], [0, 1, 2, 12], [0, 4, 8, 12]):
        parts = [partial(a, b) for a, b in zip(edges[:-1], edges[1:])]
        left = parts[0]
        for p in parts[1:]:
            left = merge(left, p)
        right = parts[-1]
        for p in parts[-2::-1]:
            right = merge(p, right)
        np.testing.assert_allclose(left[2] / left[1], o, **TOL)
        np.testing.assert_allclose(right[2] / right[1], o, **TOL)


# ----------------------------------------------------------------------------
# Program 4: QK-normalised causal prefill attention
# ----------------------------------------------------------------------------
def _qk_inputs(B=1, H=2, S=6, D=4):
    Q = RNG.standard_normal((B, H, S, D)); K = RNG.standard_normal((B, H, S, D)); V = RNG.standard_normal((B, H, S, D))
    return Q, K, V, 1.0 + 0.1 * RNG.standard_normal(D), 1.0 + 0.1 * RNG.standard_normal(D)


def test_qknorm_first_row_and_prefix_property():
    Q, K, V, gq, gk = _qk_inputs(S=7)
    o = oracle.qknorm_attn(Q, K, V, gq, gk, 1e-6, 0.5, 1)
    assert np.array_equal(o[:, :, 0], V[:, :, 0])           # row 0 sees only key 0
    o5 = oracle.qknorm_attn(Q[:, :, :5], K[:, :, :5], V[:, :, :5], gq, gk, 1e-6, 0.5, 1)
    np.testing.assert_allclose(o[:, :, :5], o5, **TOL)      # causal prefix


def test_qknorm_noncausal_library_special_case():
    Q, K, V, gq, gk = _qk_inputs(S=5)
    eps, scale = 1e-3, 0.8
    qh = Q / np.sqrt((Q ** 2).mean(-1, keepdims=True) + eps) * gq
    kh = K / np.sqrt((K ** 2).mean(-1, keepdims=True) + eps) * gk
    s = np.einsum("bhid,bhjd->bhij", qh, kh) * scale
    np.testing.assert_allclose(oracle.qknorm_attn(Q, K, V, gq, gk, eps, scale, 0),
                               softmax(s, axis=-1) @ V, **TOL)
    # causal: mask excluded entries to -inf before the library softmax
    mask = np.tril(np.ones((5, 5), dtype=bool))
    np.testing.assert_allclose(oracle.qknorm_attn(Q, K, V, gq, gk, eps, scale, 1),
                               softmax(np.where(mask, s, -np.inf), axis=-1) @ V, **TOL)


def test_qknorm_logits_side_factor_motion():
    # s_ij = scale * rq_i * rk_j * sum_d q_id (gq_d gk_d) k_jd: the inverse-RMS factors are invariant
    # along the contraction (head_dim) and move onto the logits (Table 1 factor motion; the paper's
    # MLA case study moves cached inverse-RMS factors from keys to logits the same way, Section 7.3)
    Q, K, V, gq, gk = _qk_inputs(S=6)
    eps, scale = 1e-6, 1.0 / np.sqrt(4.0)
    rq = 1.0 / np.sqrt((Q ** 2).mean(-1) + eps); rk = 1.0 / np.sqrt((K ** 2).mean(-1) + eps)
    raw = np.einsum("bhid,d,bhjd->bhij", Q, gq * gk, K)
    s = scale * rq[..., :, None] * rk[..., None, :] * raw
    mask = np.tril(np.ones((6, 6), dtype=bool))
    np.testing.assert_allclose(oracle.qknorm_attn(Q, K, V, gq, gk, eps, scale, 1),
                               softmax(np.where(mask, s, -np.inf), axis=-1) @ V, **TOL)


def test_qknorm_last_row_equals_decode_oracle():
    # cross-program tie: row S-1 of prefill == decode over all S keys with normalised q, K
    Q, K, V, gq, gk = _qk_inputs(B=2, H=3, S=6)
    eps, scale = 1e-4, 0.6
    o = oracle.qknorm_attn(Q, K, V, gq, gk, eps, scale, 1)
    qh = Q / np.sqrt((Q ** 2).mean(-1, keepdims=True) + eps) * gq
    kh = K / np.sqrt((K ** 2).mean(-1, keepdims=True) + eps) * gk
    od = oracle.gqa_decode(qh[:, :, -1], kh, V, scale)
    np.testing.assert_allclose(o[:, :, -1], od, **TOL)


def test_qknorm_scale_invariance_at_zero_eps():
    Q, K, V, gq, gk = _qk_inputs(S=5)
    o = oracle.qknorm_attn(Q, K, V, gq, gk, 0.0, 0.5, 1)
    Q2, K2 = Q.copy(), K.copy()
    Q2[0, 0, 3] *= 11.0; K2[0, 1, 2] *= 0.01
    np.testing.assert_allclose(oracle.qknorm_attn(Q2, K2, V, gq, gk, 0.0, 0.5, 1), o, rtol=1e-11, atol=1e-12)


def test_qknorm_rolling_with_causal_tile_skipping():
    # M2 over key tiles, visiting only tiles that intersect j <= i and masking inside the diagonal tile
    S, D, eps, scale = 8, 4, 1e-6, 0.5
    Q, K, V, gq, gk = _qk_inputs(B=1, H=1, S=S, D=D)
    o = oracle.qknorm_attn(Q, K, V, gq, gk, eps, scale, 1)[0, 0]
    qh = (Q / np.sqrt((Q ** 2).mean(-1, keepdims=True) + eps) * gq)[0, 0]
    kh = (K / np.sqrt((K ** 2).mean(-1, keepdims=True) + eps) * gk)[0, 0]
    for T in (1, 2, 4):
        for i in range(S):
            tiles = [(a, min(a + T, i + 1)) for a in range(0, i + 1, T)]
            np.testing.assert_allclose(_m2_rolling(qh[i], kh, V[0, 0], scale, tiles), o[i], rtol=1e-11, atol=1e-12)


# ----------------------------------------------------------------------------
# Program 5: LoRA-fused linear
# ----------------------------------------------------------------------------
def test_qknorm_attn_ex_mask_variants():
    """Window + sinks + grouped heads: equals a dense softmax under an explicitly built mask (library routines);
    no window / MHA reduces to the plain program; a window of 1 returns v_i; sinks add exactly the first keys;
    GQA equals MHA on repeat-interleaved K, V."""
    B, Hq, Hkv, S, D = 2, 4, 2, 13, 6
    Q = RNG.standard_normal((B, Hq, S, D)); K = RNG.standard_normal((B, Hkv, S, D)); V = RNG.standard_normal((B, Hkv, S, D))
    gq = 1 + 0.1 * RNG.standard_normal(D); gk = 1 + 0.1 * RNG.standard_normal(D)
    eps, scale = 1e-6, 0.6

    def dense(window, sinks):
        qh = Q / np.sqrt((Q ** 2).mean(-1, keepdims=True) + eps) * gq
        kh = K / np.sqrt((K ** 2).mean(-1, keepdims=True) + eps) * gk
        kx, vx = np.repeat(kh, Hq // Hkv, axis=1), np.repeat(V, Hq // Hkv, axis=1)
        logits = np.einsum("bhid,bhjd->bhij", qh, kx) * scale
        i, j = np.arange(S)[:, None], np.arange(S)[None, :]
        vis = (j <= i) & ((window == 0) | (j > i - window) | (j < sinks))
        logits = np.where(vis, logits, -np.inf)
        return np.einsum("bhij,bhjd->bhid", softmax(logits, axis=-1), vx)

    for window, sinks in [(0, 0), (5, 0), (5, 2), (1, 0), (1, 3), (4, 4), (13, 0), (100, 2)]:
        o = oracle.qknorm_attn_ex(Q, K, V, gq, gk, eps, scale, 1, window, sinks)
        np.testing.assert_allclose(o, dense(window, sinks), **TOL)
    # window 1, no sinks: every query sees only itself
    o1 = oracle.qknorm_attn_ex(Q, K, V, gq, gk, eps, scale, 1, 1, 0)
    np.testing.assert_allclose(o1, np.repeat(V, Hq // Hkv, axis=1), **TOL)
    # MHA, no window: the plain program (same routine family, independent code path in the oracle)
    Kx, Vx = np.repeat(K, Hq // Hkv, axis=1), np.repeat(V, Hq // Hkv, axis=1)
    np.testing.assert_allclose(oracle.qknorm_attn_ex(Q, Kx, Vx, gq, gk, eps, scale, 1, 0, 0),
                               oracle.qknorm_attn(Q, Kx, Vx, gq, gk, eps, scale, 1), **TOL)
    # grouped heads == MHA on expanded K, V, under a window as well
    np.testing.assert_allclose(oracle.qknorm_attn_ex(Q, K, V, gq, gk, eps, scale, 1, 5, 2),
                               oracle.qknorm_attn_ex(Q, Kx, Vx, gq, gk, eps, scale, 1, 5, 2), **TOL)
    # non-causal ignores window and sinks
    np.testing.assert_allclose(oracle.qknorm_attn_ex(Q, Kx, Vx, gq, gk, eps, scale, 0, 3, 1),
                               oracle.qknorm_attn(Q, Kx, Vx, gq, gk, eps, scale, 0), **TOL)


def test_lora_library_special_cases():
    M, K, N, R = 3, 7, 5, 2
    X = RNG.standard_normal((M, K)); W = RNG.standard_normal((K, N)); A = RNG.standard_normal((K, R)); B = RNG.standard_normal((R, N))
    np.testing.assert_allclose(oracle.lora_linear(X, W, A, B, 0.0), X @ W, **TOL)
    np.testing.assert_allclose(oracle.lora_linear(X, W, A, np.zeros((R, N)), 2.0), X @ W, **TOL)
    np.testing.assert_allclose(oracle.lora_linear(X, np.zeros((K, N)), A, B, 1.0), (X @ A) @ B, **TOL)


def test_lora_reassociation_and_factoring():
    # (XA)B == X(AB) (Table 1, reassociate MatMul); XW + a X(AB) == X(W + a AB) (Figure 2, factoring)
    M, K, N, R = 4, 6, 5, 3
    X = RNG.standard_normal((M, K)); W = RNG.standard_normal((K, N)); A = RNG.standard_normal((K, R)); B = RNG.standard_normal((R, N))
    alpha = 2.0
    y = oracle.lora_linear(X, W, A, B, alpha)
    np.testing.assert_allclose(y, X @ W + alpha * (X @ (A @ B)), **TOL)
    np.testing.assert_allclose(y, X @ (W + alpha * (A @ B)), **TOL)
    # concatenation identity: [X | alpha T] @ [W ; B] with T = X@A (one extra K slab of width R)
    T = X @ A
    np.testing.assert_allclose(y, np.concatenate([X, alpha * T], 1) @ np.concatenate([W, B], 0), **TOL)


def test_lora_linearity_and_one_hot_adapter():
    M, K, N, R = 3, 5, 4, 2
    X = RNG.standard_normal((M, K)); W = RNG.standard_normal((K, N)); B = RNG.standard_normal((R, N))
    A = RNG.standard_normal((K, R))
    y0, y1, y3 = (oracle.lora_linear(X, W, A, B, a) for a in (0.0, 1.0, 3.0))
    np.testing.assert_allclose(y3 - y0, 3.0 * (y1 - y0), **TOL)
    A1 = np.zeros((K, R)); A1[2, 0] = 1.0; A1[4, 1] = 1.0     # T = X[:, [2, 4]]
    np.testing.assert_allclose(oracle.lora_linear(X, W, A1, B, 1.5), X @ W + 1.5 * X[:, [2, 4]] @ B, **TOL)


# ----------------------------------------------------------------------------
# brute force on tiny inputs: explicit scalar loops, no library routine
# ----------------------------------------------------------------------------
def test_brute_force_scalar_loops():
    import math
    M, K, N, R = 2, 3, 2, 2
    X = RNG.standard_normal((M, K)); W = RNG.standard_normal((K, N)); W2 = RNG.standard_normal((K, N))
    gamma = RNG.standard_normal(K); A = RNG.standard_normal((K, R)); B = RNG.standard_normal((R, N)); eps = 0.01
    y1 = oracle.rmsnorm_matmul(X, gamma, W, eps); y2 = oracle.gated_mlp(X, W, W2); y5 = oracle.lora_linear(X, W, A, B, 2.0)
    for i in range(M):
        ms = sum(X[i, k] ** 2 for k in range(K)) / K
        for n in range(N):
            e1 = sum(X[i, k] / math.sqrt(ms + eps) * gamma[k] * W[k, n] for k in range(K))
            gg = sum(X[i, k] * W[k, n] for k in range(K)); uu = sum(X[i, k] * W2[k, n] for k in range(K))
            e2 = gg / (1.0 + math.exp(-gg)) * uu
            e5 = sum(X[i, k] * W[k, n] for k in range(K)) + 2.0 * sum(
                sum(X[i, k] * A[k, r] for k in range(K)) * B[r, n] for r in range(R))
            assert abs(y1[i, n] - e1) < 1e-12 and abs(y2[i, n] - e2) < 1e-12 and abs(y5[i, n] - e5) < 1e-12


def test_oracle_reports_threads():
    assert oracle.num_threads() >= 1
