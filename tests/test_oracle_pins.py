"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library; they run without a GPU.
"""
import math
import os

import numpy as np
import pytest

import rmm_inputs as R
from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M32 = 0xFFFFFFFF


# --------------------------------------------------------------------------- Philox
def _philox_python(ctr, key):
    """Independent big-integer transcription of the published round function."""
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & M32, p1 & M32, ((p0 >> 32) ^ c[3] ^ k[1]) & M32, p0 & M32]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert list(O.philox4x32_10(v[0:4], v[4:6])) == v[6:10]


def test_philox_matches_independent_transcription():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2**32, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 2**32, 2, dtype=np.uint64)]
        assert list(O.philox4x32_10(ctr, key)) == _philox_python(ctr, key)


# ------------------------------------------------------------------- normal transform
def test_gaussian_radius_against_box_muller_all_inputs():
    # angle word fixed at y = -1/32768 (cos ~ 1); all 2^16 radius inputs.
    worst = 0.0
    for hi in range(65536):
        ze, _ = O.gauss_pair((hi << 16) | 16383)
        r = math.sqrt(-2.0 * math.log((2 * hi + 1) / 2.0**17))
        worst = max(worst, abs(ze - r * math.cos(math.pi / 2 * (-1 / 32768))))
        assert ze > 0.0 and math.isfinite(ze)
    assert worst < 1e-3, worst


def test_gaussian_angle_against_box_muller_all_inputs():
    hi = 20000
    r = math.sqrt(-2.0 * math.log((2 * hi + 1) / 2.0**17))
    worst = 0.0
    for lo in range(65536):
        ze, zo = O.gauss_pair((hi << 16) | lo)
        y = (2 * (lo & 0x7FFF) + 1) / 32768.0 - 1.0
        sg = -1.0 if lo >> 15 else 1.0
        worst = max(worst, abs(ze - sg * r * math.cos(math.pi / 2 * y)), abs(zo - sg * r * math.sin(math.pi / 2 * y)))
    assert worst < 5e-5, worst


def test_gaussian_moments_and_tail():
    # 2^22 entries straight from the generator (fp32 storage, unscaled).
    P = O.generate_p(seed=12345, N=2048, k=2048, dist=O.DIST_GAUSSIAN, storage=O.STORE_F32).astype(np.float64).ravel()
    T = P.size
    assert abs(P.mean()) < 4.0 / math.sqrt(T)
    assert abs(P.var() - 1.0) < 4.0 * math.sqrt(2.0 / T) + 1e-4
    kurt = np.mean(P**4) / P.var() ** 2
    assert abs(kurt - 3.0) < 4.0 * math.sqrt(96.0 / T) + 2e-3, kurt
    assert abs(np.mean(P**3)) < 4.0 * math.sqrt(15.0 / T)
    assert np.abs(P).max() <= math.sqrt(2 * 17 * math.log(2)) + 1e-3   # 16-bit radius input
    # distribution function at a few points (Kolmogorov-style check)
    for z, phi in [(-2.0, 0.0227501319), (-1.0, 0.1586552539), (0.0, 0.5), (0.5, 0.6914624613), (1.5, 0.9331927987)]:
        assert abs(np.mean(P <= z) - phi) < 4.0 * math.sqrt(phi * (1 - phi) / T) + 1e-4
    # neighbouring entries (same Philox block, same word) are uncorrelated
    Q = P.reshape(2048, 2048)
    assert abs(np.mean(Q[0::2] * Q[1::2])) < 4.0 / math.sqrt(T / 2)


def test_bf16_rounding_matches_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    a = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 3,
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 65280.0, 1e-30], np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([O.bf16_round(float(x)) for x in a], dtype=np.float32)
    assert np.array_equal(got, want)
    assert np.array_equal(R.round_to_bf16(a), want)


def test_scale_is_fp32_reciprocal_sqrt():
    for k in (1, 2, 3, 256, 410, 819, 1638, 3686):
        want = np.float32(1.0) / np.sqrt(np.float32(k))
        assert np.float32(O.scale(k, O.DIST_GAUSSIAN)) == want
        assert np.float32(O.scale(k, O.DIST_RADEMACHER)) == want
    assert O.scale(5, O.DIST_IDENTITY) == 1.0


# -------------------------------------------------------------------- counter mapping
def test_gaussian_counter_mapping():
    seed, N, k = 0x1234567890ABCDEF, 37, 5
    P = O.generate_p(seed, N, k, O.DIST_GAUSSIAN, O.STORE_F32)
    key = [seed & M32, seed >> 32]
    for n in (0, 1, 7, 8, 13, 30, 36):
        for j in range(k):
            words = _philox_python([n >> 3, j, 0, 0], key)
            ze, zo = O.gauss_pair(words[(n & 7) >> 1])
            assert P[n, j] == np.float32(zo if n & 1 else ze)
    Pb = O.generate_p(seed, N, k, O.DIST_GAUSSIAN, O.STORE_BF16)
    assert np.array_equal(Pb, R.round_to_bf16(P))
    # a column range is the same as slicing the whole matrix; rows do not depend on N
    assert np.array_equal(O.generate_p(seed, N, k, O.DIST_GAUSSIAN, O.STORE_F32, 2, 4), P[:, 2:4])
    assert np.array_equal(O.generate_p(seed, 64, k, O.DIST_GAUSSIAN, O.STORE_F32)[:N], P)


def test_rademacher_counter_mapping():
    seed, N, k = 99, 300, 3
    P = O.generate_p(seed, N, k, O.DIST_RADEMACHER, O.STORE_BF16)
    assert set(np.unique(P)) == {-1.0, 1.0}
    key = [seed & M32, seed >> 32]
    for n in (0, 31, 32, 127, 128, 299):
        for j in range(k):
            words = _philox_python([n >> 7, j, 0, 1], key)
            bit = (words[(n & 127) >> 5] >> (n & 31)) & 1
            assert P[n, j] == (-1.0 if bit else 1.0)
    S = O.generate_s(seed, N, k, O.DIST_RADEMACHER, O.STORE_BF16)
    assert np.array_equal(S, P.astype(np.float64) * float(np.float32(1) / np.sqrt(np.float32(k))))


def test_sors_is_sign_flipped_hadamard_columns():
    """P[n][j] = d_n * H[n][r_j]: H against scipy's Sylvester Hadamard matrix, d_n and r_j against the
    independent Philox transcription; N not a power of two takes the first N rows of the next order."""
    from scipy.linalg import hadamard
    for seed, N, k in ((3, 64, 9), (0xABCDEF0123456789, 300, 5), (7, 1, 2), (11, 129, 4)):
        L = 1
        while L < N:
            L *= 2
        H = hadamard(L) if L > 1 else np.ones((1, 1))
        key = [seed & M32, seed >> 32]
        P = O.generate_p(seed, N, k, O.DIST_SORS, O.STORE_BF16)
        assert set(np.unique(P)) <= {-1.0, 1.0}
        d = np.array([-1.0 if (_philox_python([n >> 7, 0, 0, 2], key)[(n & 127) >> 5] >> (n & 31)) & 1 else 1.0
                      for n in range(N)])
        for j in range(k):
            r = _philox_python([j, 0, 0, 3], key)[0] % L
            assert np.array_equal(P[:, j], d * H[:N, r]), (seed, N, j)
        S = O.generate_s(seed, N, k, O.DIST_SORS, O.STORE_F32)
        assert np.array_equal(S, P.astype(np.float64) * float(np.float32(1) / np.sqrt(np.float32(k))))
    # the full orthonormal matrix: all L columns of H, each once, give S S^T = I exactly (what subsampling draws from)
    H = hadamard(32) / math.sqrt(32.0)
    assert np.allclose(H @ H.T, np.eye(32), atol=1e-12)


def test_dct_is_sign_flipped_scaled_dct2_rows():
    """P[n][j] = d_n * sqrt(L) * C[r_j][n] with C the orthonormal DCT-II matrix of order L (scipy's, an independent
    library), d_n and r_j from the independent Philox transcription; N not a power of two takes the first N
    columns of the next order.  The fp32 cosine (quadrant reduction + two cubics) stays within 2e-5 of the exact one."""
    from scipy.fft import dct
    for seed, N, k in ((3, 64, 9), (0xABCDEF0123456789, 300, 7), (7, 1, 2), (11, 129, 4), (5, 1000, 3)):
        L = 1
        while L < N:
            L *= 2
        Cm = dct(np.eye(L), type=2, norm="ortho", axis=0)          # Cm[r][n]
        assert np.allclose(Cm @ Cm.T, np.eye(L), atol=1e-12)       # the matrix the sketch subsamples is orthonormal
        key = [seed & M32, seed >> 32]
        P = O.generate_p(seed, N, k, O.DIST_DCT, O.STORE_F32).astype(np.float64)
        d = np.array([-1.0 if (_philox_python([n >> 7, 0, 0, 2], key)[(n & 127) >> 5] >> (n & 31)) & 1 else 1.0
                      for n in range(N)])
        for j in range(k):
            r = _philox_python([j, 0, 0, 3], key)[0] % L
            want = d * math.sqrt(L) * Cm[r, :N]
            assert np.abs(P[:, j] - want).max() < 2e-5, (seed, N, j, r)
        Pb = O.generate_p(seed, N, k, O.DIST_DCT, O.STORE_BF16)
        assert np.array_equal(Pb, R.round_to_bf16(P.astype(np.float32)))
        S = O.generate_s(seed, N, k, O.DIST_DCT, O.STORE_F32)
        assert np.array_equal(S, P * float(np.float32(1) / np.sqrt(np.float32(k))))
    # a column with r_j = 0 is the constant row of the DCT: entries d_n exactly
    seed, N = 0, 8
    key = [seed & M32, seed >> 32]
    js = [j for j in range(4000) if _philox_python([j, 0, 0, 3], key)[0] % 8 == 0][:3]
    assert js
    for j in js:
        col = O.generate_p(seed, N, j + 1, O.DIST_DCT, O.STORE_F32, j, j + 1)[:, 0]
        assert set(np.unique(np.abs(col))) == {1.0}


def test_identity_matrix():
    assert np.array_equal(O.generate_s(1, 6, 6, O.DIST_IDENTITY, O.STORE_BF16), np.eye(6))


# ------------------------------------------------------------- brute force, tiny shapes
def _loops_forward(X, W, b, S):
    N, Din = X.shape
    Dout, k = W.shape[0], S.shape[1]
    Y = [[sum(X[n][i] * W[o][i] for i in range(Din)) + b[o] for o in range(Dout)] for n in range(N)]
    Xp = [[sum(S[n][j] * X[n][i] for n in range(N)) for i in range(Din)] for j in range(k)]
    return np.array(Y), np.array(Xp)


def _loops_backward(dY, W, Xp, S):
    N, Dout = dY.shape
    Din, k = W.shape[1], S.shape[1]
    dX = [[sum(dY[n][o] * W[o][i] for o in range(Dout)) for i in range(Din)] for n in range(N)]
    # (dY^T S) first, then times X_proj: the association of Algorithm 1
    YtS = [[sum(dY[n][o] * S[n][j] for n in range(N)) for j in range(k)] for o in range(Dout)]
    dW = [[sum(YtS[o][j] * Xp[j][i] for j in range(k)) for i in range(Din)] for o in range(Dout)]
    db = [sum(dY[n][o] for n in range(N)) for o in range(Dout)]
    return np.array(dX), np.array(dW), np.array(db)


@pytest.mark.parametrize("dist", [O.DIST_GAUSSIAN, O.DIST_RADEMACHER])
def test_brute_force_tiny(dist):
    rng = np.random.default_rng(11)
    N, Din, Dout, k = 7, 5, 3, 4
    X, W, b, dY = rng.standard_normal((N, Din)), rng.standard_normal((Dout, Din)), rng.standard_normal(Dout), rng.standard_normal((N, Dout))
    S = O.generate_s(5, N, k, dist, O.STORE_F32)
    Y, Xp = O.forward(X, W, b, S)
    Y0, Xp0 = _loops_forward(X, W, b, S)
    assert np.allclose(Y, Y0, rtol=1e-13, atol=1e-13) and np.allclose(Xp, Xp0, rtol=1e-13, atol=1e-13)
    dX, dW, db, G = O.backward(dY, W, Xp, S)
    dX0, dW0, db0 = _loops_backward(dY, W, Xp0, S)
    assert np.allclose(dX, dX0, rtol=1e-13, atol=1e-13)
    assert np.allclose(dW, dW0, rtol=1e-12, atol=1e-13)
    assert np.allclose(db, db0, rtol=1e-13, atol=1e-13)
    assert np.allclose(G, S.T @ dY, rtol=1e-13, atol=1e-13)
    # matrix form of the same definitions (Eq. 1, 2, 4) through an independent library
    assert np.allclose(Y, X @ W.T + b) and np.allclose(Xp, S.T @ X)
    assert np.allclose(dX, dY @ W) and np.allclose(dW, (dY.T @ S) @ (S.T @ X))
    assert np.allclose(O.exact_dw(dY, X), dY.T @ X)


def test_hand_computed_two_by_two():
    # Eq. 1-3 by hand: X = [[1,2],[3,4]], W = [[1,0],[1,1]], b = [10,20], dY = [[1,0],[2,1]], S = I.
    X = np.array([[1.0, 2.0], [3.0, 4.0]])
    W = np.array([[1.0, 0.0], [1.0, 1.0]])
    b = np.array([10.0, 20.0])
    dY = np.array([[1.0, 0.0], [2.0, 1.0]])
    S = np.eye(2)
    Y, Xp = O.forward(X, W, b, S)
    assert Y.tolist() == [[11.0, 23.0], [13.0, 27.0]] and Xp.tolist() == X.tolist()
    dX, dW, db, _ = O.backward(dY, W, Xp, S)
    assert dX.tolist() == [[1.0, 0.0], [3.0, 1.0]]       # dY W
    assert dW.tolist() == [[7.0, 10.0], [3.0, 4.0]]      # dY^T X
    assert db.tolist() == [3.0, 1.0]


def test_identity_sketch_reproduces_exact_gradient():
    rng = np.random.default_rng(5)
    N, Din, Dout = 9, 6, 4
    X, W, dY = rng.standard_normal((N, Din)), rng.standard_normal((Dout, Din)), rng.standard_normal((N, Dout))
    S = O.generate_s(0, N, N, O.DIST_IDENTITY, O.STORE_F32)
    _, Xp = O.forward(X, W, None, S)
    assert np.array_equal(Xp, X)
    _, dW, _, _ = O.backward(dY, W, Xp, S)
    assert np.allclose(dW, dY.T @ X, rtol=1e-14, atol=1e-14)


# --------------------------------------------------------------- statistical properties
@pytest.mark.parametrize("dist", [O.DIST_GAUSSIAN, O.DIST_RADEMACHER, O.DIST_SORS, O.DIST_DCT])
def test_unbiasedness_of_s_st(dist):
    N, k, T = (13 if dist == O.DIST_DCT else 16), 8, 4000      # DCT: a token count that is not a power of two
    acc = np.zeros((N, N))
    for seed in range(T):
        S = O.generate_s(seed, N, k, dist, O.STORE_F32)
        acc += S @ S.T
    M = acc / T
    off = M - np.diag(np.diag(M))
    # variance of one diagonal term: 2 for normals, 0 for +-1 entries, at most 1/2 for 2 cos^2 - 1 = cos(2 theta)
    sd_diag = math.sqrt({O.DIST_GAUSSIAN: 2.0, O.DIST_DCT: 1.0}.get(dist, 0.0) / (k * T)) + 1e-6
    assert np.abs(np.diag(M) - 1.0).max() < 4.5 * sd_diag
    assert np.abs(off).max() < 4.5 * math.sqrt(1.0 / (k * T))


@pytest.mark.parametrize("dist", [O.DIST_SORS, O.DIST_DCT])
def test_sors_gradient_is_unbiased(dist):
    """E_S[dW_rmm] = dW for the subsampled Hadamard and DCT sketches (token count not a power of two)."""
    rng = np.random.default_rng(5)
    N, Din, Dout, k, T = 6, 4, 3, 3, 20000
    X = rng.standard_normal((N, Din))
    dY = X[:, :Dout] * 0.8 + 0.4 * rng.standard_normal((N, Dout))
    W = rng.standard_normal((Dout, Din))
    dW_star = O.exact_dw(dY, X)
    tot, sq = np.zeros_like(dW_star), np.zeros_like(dW_star)
    for seed in range(T):
        S = O.generate_s(500 + seed, N, k, dist, O.STORE_F32)
        _, Xp = O.forward(X, W, None, S, want_y=False)
        _, dW, _, _ = O.backward(dY, W, Xp, S, want_dx=False, want_db=False)
        tot += dW
        sq += dW * dW
    mean = tot / T
    sd = np.sqrt(np.maximum(sq / T - mean**2, 0) / T)
    assert (np.abs(mean - dW_star) / sd).max() < 4.5


@pytest.mark.parametrize("dist", [O.DIST_GAUSSIAN, O.DIST_RADEMACHER])
def test_unbiased_gradient_and_variance(dist):
    # correlated X and dY so that alpha is large and the printed Eq. 11 is far from the truth
    rng = np.random.default_rng(21)
    N, Din, Dout, k, T = 6, 4, 3, 3, 20000
    X = rng.standard_normal((N, Din))
    dY = X[:, :Dout] * 0.8 + 0.4 * rng.standard_normal((N, Dout))
    W = rng.standard_normal((Dout, Din))
    dW_star = O.exact_dw(dY, X)
    tot, sq = np.zeros_like(dW_star), np.zeros_like(dW_star)
    err2 = 0.0
    for seed in range(T):
        S = O.generate_s(1000 + seed, N, k, dist, O.STORE_F32)
        _, Xp = O.forward(X, W, None, S, want_y=False)
        _, dW, _, _ = O.backward(dY, W, Xp, S, want_dx=False, want_db=False)
        tot += dW
        sq += dW * dW
        err2 += float(np.sum((dW - dW_star) ** 2))
    mean = tot / T
    sd = np.sqrt(np.maximum(sq / T - mean**2, 0) / T)
    zscores = np.abs(mean - dW_star) / sd
    assert zscores.max() < 4.5, zscores                       # E_S[dW_rmm] = dW (Eq. 4)
    closed = (O.d2_rmm_gaussian if dist == O.DIST_GAUSSIAN else O.d2_rmm_rademacher)(X, dY, k)
    printed = O.d2_rmm_printed(X, dY, k)
    mc = err2 / T
    assert abs(mc / closed - 1.0) < 0.05, (mc, closed, printed)
    assert O.alpha(X, dY) > 0.15
    if dist == O.DIST_GAUSSIAN:
        assert abs(mc / printed - 1.0) > 0.2                   # the printed sign does not fit


def test_variance_closed_forms_against_definitions():
    rng = np.random.default_rng(2)
    B, Nx, My, k = 5, 4, 3, 7
    X, Y = rng.standard_normal((B, Nx)), rng.standard_normal((B, My))
    nx2, ny2, xty2 = np.sum(X**2), np.sum(Y**2), np.sum((X.T @ Y) ** 2)
    rows = np.sum(np.sum(X**2, 1) * np.sum(Y**2, 1))
    assert math.isclose(O.d2_rmm_printed(X, Y, k), (nx2 * ny2 - xty2) / k, rel_tol=1e-12)
    assert math.isclose(O.d2_rmm_gaussian(X, Y, k), (nx2 * ny2 + xty2) / k, rel_tol=1e-12)
    assert math.isclose(O.d2_rmm_rademacher(X, Y, k), (nx2 * ny2 + xty2 - 2 * rows) / k, rel_tol=1e-12)
    assert math.isclose(O.alpha(X, Y), xty2 / (nx2 * ny2), rel_tol=1e-12)
    # Lemma 1 from its definition: 1/(B(B-1)) sum_k |B x_k y_k^T - X^T Y|_F^2
    Z = X.T @ Y
    d = sum(np.sum((B * np.outer(X[r], Y[r]) - Z) ** 2) for r in range(B)) / (B * (B - 1))
    assert math.isclose(O.d2_sgd(X, Y), d, rel_tol=1e-12)


def test_variance_worked_example_from_paper():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "variance_worked_example.txt")) if l.strip() and l[0] != "#"]
    for eps, sgd, rmm in [(float(a), float(b), float(c)) for a, b, c in rows]:
        X = np.array([[1.0, 0.0], [-eps, 0.0]])
        Y = np.array([[1.0, 0.0], [1.0 / eps, 0.0]])
        assert np.allclose(X.T @ Y, 0.0)
        for k in (1, 3):
            assert math.isclose((2 - 1) * O.d2_sgd(X, Y), sgd, rel_tol=1e-12)
            assert math.isclose(k * O.d2_rmm_printed(X, Y, k), rmm, rel_tol=1e-12)
            # with X^T Y = 0 the Gaussian form coincides with the printed one
            assert math.isclose(k * O.d2_rmm_gaussian(X, Y, k), rmm, rel_tol=1e-12)
        assert math.isclose(rmm, 2 + eps**2 + eps**-2, rel_tol=1e-12)


# -------------------------------------------------------------------- input generators
def test_inputs_are_seeded_and_storage_exact():
    w = R.WORKLOADS["base_ffn_up_rho0.2"]
    assert w.b_proj == 819 and R.WORKLOADS["large_ffn_up_rho0.1"].b_proj == 1638
    assert [R.WORKLOADS[f"base_ffn_up_rho{r}"].b_proj for r in ("0.1", "0.5", "0.9")] == [410, 2048, 3686]
    X, W, b, dY = R.make_inputs(w, n_tokens=64)
    X2, _, _, _ = R.make_inputs(w, n_tokens=64)
    assert np.array_equal(X, X2) and np.array_equal(R.round_to_bf16(X), X)
    assert X.shape == (64, 768) and W.shape == (3072, 768) and dY.shape == (64, 3072) and not b.any()
    assert abs(W.std() - 0.02) < 1e-3 and abs(dY.std() - 0.01) < 1e-3 and abs(X.std() - 1.0) < 0.02
    assert np.array_equal(R.bf16_bits_to_f32(R.bf16_bits(X)), X)
    assert w.saved_bytes() == {"rmm": 819 * 768 * 2 + 8, "standard": 4096 * 768 * 2}
