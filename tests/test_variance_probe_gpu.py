"""Variance diagnostics on the device (Lemma 1 Eq. 9, Lemma 2 Eq. 11 and its corrected forms,
Theorem 1 Eq. 13) against the CPU oracle's own implementations of the same definitions."""
import numpy as np
import pytest
import torch

import rmm_inputs as R

pytestmark = pytest.mark.gpu


def _oracle_values(X, dY, k, dist):
    from oracle import oracle as O
    a = float((X * X).sum())
    b = float((dY * dY).sum())
    c = float(((X * X).sum(axis=1) * (dY * dY).sum(axis=1)).sum())
    dw = O.exact_dw(dY, X)
    d = float((dw * dw).sum())
    d2 = {R.DIST_GAUSSIAN: O.d2_rmm_gaussian, R.DIST_RADEMACHER: O.d2_rmm_rademacher}[dist](X, dY, k)
    return np.array([a, b, c, d, O.d2_sgd(X, dY), d2, O.d2_rmm_printed(X, dY, k), O.alpha(X, dY)]), dw


@pytest.mark.parametrize("n,d_in,d_out,k,dist,correlated", [
    (300, 264, 520, 130, R.DIST_GAUSSIAN, False),       # ragged against every tile
    (2, 8, 8, 1, R.DIST_RADEMACHER, False),             # smallest legal problem
    (1000, 768, 256, 200, R.DIST_RADEMACHER, True),     # alpha of order one: printed and corrected forms differ
    (2048, 768, 1024, 410, R.DIST_GAUSSIAN, False),     # several tiles of the contraction, many row blocks
])
def test_variance_probe_matches_oracle(n, d_in, d_out, k, dist, correlated):
    import paper_2201_13195_b200 as P
    w = R.small_case(f"variance_{n}_{d_in}_{d_out}", R.DTYPE_BF16, n, d_in, d_out, k, dist, seed=1)
    X, W, b, dY = R.make_inputs(w)
    if correlated:     # X and dY share a dominant rank-one token factor: |X^T dY|^2 is comparable to |X|^2 |dY|^2
        g = np.random.default_rng(5)
        u, v, q = g.standard_normal((n, 1)), g.standard_normal((1, d_in)), g.standard_normal((1, d_out))
        X = R.round_to_bf16((u @ v + 0.3 * X).astype(np.float32))
        dY = R.round_to_bf16((u @ q + 0.3 * g.standard_normal((n, d_out))).astype(np.float32))
    Xd = torch.from_numpy(X).cuda().to(torch.bfloat16).contiguous()
    dYd = torch.from_numpy(dY).cuda().to(torch.bfloat16).contiguous()
    dw_gpu = torch.empty(d_out, d_in, dtype=torch.bfloat16, device="cuda")
    out = P.rmm_variance_probe(Xd, dYd, k, dist, dW_exact=dw_gpu)
    out2 = P.rmm_variance_probe(Xd, dYd, k, dist)          # without the optional output; must be bit-identical
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.array_equal(got, out2.cpu().numpy()), "not reproducible"
    ref, dw = _oracle_values(X.astype(np.float64), dY.astype(np.float64), k, dist)
    rel = np.abs(got - ref) / np.maximum(np.abs(ref), 1e-300)
    assert (rel <= 1e-4).all(), dict(zip(P.VARIANCE_FIELDS, zip(got, ref)))
    from oracle import oracle as O
    assert O.rel_frobenius(dw_gpu.float().cpu().numpy(), dw) <= 1e-2
    if correlated:     # the printed form of Eq. 11 is measurably below the corrected one here
        assert got[7] > 0.3 and got[6] < 0.8 * got[5]


def test_variance_probe_identity_sketch_has_no_variance():
    import paper_2201_13195_b200 as P
    X = torch.randn(64, 32, device="cuda").to(torch.bfloat16)
    dY = torch.randn(64, 48, device="cuda").to(torch.bfloat16)
    out = P.rmm_variance_probe(X, dY, 64, P.RMM_DIST_IDENTITY).cpu().numpy()
    assert out[5] == 0.0 and out[0] > 0 and out[4] > 0


@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER])
def test_gpu_estimator_is_unbiased_and_has_the_probed_variance(dist):
    """The library's own dW over many seeds: its mean is the exact gradient dY^T X (Section 2.1,
    unbiasedness) and its mean squared error is the D^2_RMM that rmm_variance_probe reports for the
    same X and dY (Lemma 2 with the fourth moment kept)."""
    import paper_2201_13195_b200 as P
    n, d_in, d_out, k, T = 96, 16, 24, 12, 3000
    g = np.random.default_rng(11)
    u = g.standard_normal((n, 1))      # a shared token factor: |X^T dY|^2 comparable to |X|^2 |dY|^2 (alpha about 0.5)
    X = R.round_to_bf16((u @ g.standard_normal((1, d_in)) + 0.3 * g.standard_normal((n, d_in))).astype(np.float32))
    dY = R.round_to_bf16((u @ g.standard_normal((1, d_out)) + 0.3 * g.standard_normal((n, d_out))).astype(np.float32))
    Xd = torch.from_numpy(X).cuda().to(torch.bfloat16).contiguous()
    dYd = torch.from_numpy(dY).cuda().to(torch.bfloat16).contiguous()
    W = torch.zeros(d_out, d_in, dtype=torch.bfloat16, device="cuda")
    ws = P.alloc_workspace(n, d_in, d_out, k, P.RMM_DTYPE_BF16)
    Xp = torch.empty(k, d_in, dtype=torch.bfloat16, device="cuda")
    dW = torch.empty(d_out, d_in, dtype=torch.bfloat16, device="cuda")
    exact = dY.astype(np.float64).T @ X.astype(np.float64)
    acc = torch.zeros(d_out, d_in, dtype=torch.float64, device="cuda")
    acc2 = torch.zeros(d_out, d_in, dtype=torch.float64, device="cuda")
    ex = torch.from_numpy(exact).cuda()
    for seed in range(T):
        P.rmm_forward(Xd, W, None, 1000 + seed, k, dist, X_proj=Xp, workspace=ws, want_y=False)
        P.rmm_backward(dYd, W, Xp, 1000 + seed, dist, dW=dW, workspace=ws, want_dx=False, want_db=False)
        e = dW.double() - ex
        acc += e
        acc2 += e * e
    torch.cuda.synchronize()
    mean_err, mse = (acc / T).cpu().numpy(), float(acc2.sum().item()) / T
    probe = P.rmm_variance_probe(Xd, dYd, k, dist).cpu().numpy()
    # per-entry standard error of the mean; bf16 storage of X_proj, G and dW adds a bias far below it
    se = np.sqrt(np.maximum((acc2 / T).cpu().numpy() - mean_err ** 2, 1e-30) / T)
    z = np.abs(mean_err) / se
    assert (z > 4.5).mean() <= 0.01 and z.max() < 6.0, float(z.max())
    assert abs(mse / probe[5] - 1.0) < 0.08, (mse, probe[5], probe[6])
    assert probe[7] > 0.3 and mse > 1.5 * probe[6]       # Eq. 11 as printed (fourth moment dropped) is far below
