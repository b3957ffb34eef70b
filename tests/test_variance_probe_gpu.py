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
