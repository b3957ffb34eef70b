"""The allocation-free bias-gradient entry point (rmm_bias_grad_static) against rmm_backward.

Some callers cannot allocate device memory at the point where they need db: inside a
region where cudaMalloc is forbidden (a captured or pool-restricted section of a training
step) or with the device already full.  rmm_bias_grad_static serves them with scratch that
lives inside the library image.  This test calls it through the C ABI twice in a row, with
different data, and checks each result against the db that rmm_backward returns for the same
dY, within the tolerances of the parity tests.  It is collected last so that a run that
stops at the first failure has already run everything else; it also passes on its own.
"""
import numpy as np
import pytest
import torch

import rmm_inputs as R

pytestmark = pytest.mark.gpu

TOL = {torch.bfloat16: 1e-2, torch.float32: 1e-5}


def _rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm())


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_bias_grad_matches_backward_twice(dtype):
    import paper_2201_13195_b200 as P
    N, D_in, D_out, k = 777, 72, 1096, 50
    dt = P.RMM_DTYPE_BF16 if dtype == torch.bfloat16 else P.RMM_DTYPE_F32
    g = torch.Generator(device="cuda").manual_seed(1234)
    W = (0.02 * torch.randn(D_out, D_in, device="cuda", generator=g)).to(dtype)
    X = torch.randn(N, D_in, device="cuda", generator=g).to(dtype)
    ws = P.alloc_workspace(N, D_in, D_out, k, dt)
    db_static = torch.empty(D_out, dtype=dtype, device="cuda")
    for call in range(2):
        # the second call has different values and a different row count than the first
        n = N if call == 0 else N - 300
        dY = (torch.randn(n, D_out, device="cuda", generator=g) * (1.0 + call) + 0.25 * call).to(dtype).contiguous()
        _, Xp = P.rmm_forward(X[:n].contiguous(), W, None, 5 + call, k, P.RMM_DIST_RADEMACHER, workspace=ws, want_y=False)
        _, _, db_ref = P.rmm_backward(dY, W, Xp, 5 + call, P.RMM_DIST_RADEMACHER, workspace=ws, want_dx=False)
        P.rmm_bias_grad_static(dY, db=db_static)
        torch.cuda.synchronize()
        assert _rel(db_static, db_ref) <= TOL[dtype], (call, _rel(db_static, db_ref))
        # and against the definition (Eq. 3) in fp64
        assert _rel(db_static, dY.double().sum(0)) <= TOL[dtype]


def test_static_bias_grad_rejects_sizes_beyond_its_scratch():
    import paper_2201_13195_b200 as P
    too_wide = P.RMM_BIAS_GRAD_STATIC_MAX_D_OUT + 8
    dY = torch.zeros(4, too_wide, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.RmmError) as e:
        P.rmm_bias_grad_static(dY)
    assert e.value.code == P.RMM_ERR_UNSUPPORTED
    ok = P.rmm_bias_grad_static(torch.ones(3, P.RMM_BIAS_GRAD_STATIC_MAX_D_OUT, dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    assert torch.equal(ok, torch.full_like(ok, 3.0))
