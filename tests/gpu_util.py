"""Helpers shared by the GPU parity tests: upload seeded inputs, call the library through
its C ABI binding, and run the CPU oracle on the same values."""
import numpy as np
import torch

import paper_2201_13195_b200 as P
import rmm_inputs as R
from oracle import oracle as O

TOL = {R.DTYPE_BF16: 1e-2, R.DTYPE_F32: 1e-5}   # relative Frobenius error per output tensor
TORCH_DTYPE = {R.DTYPE_BF16: torch.bfloat16, R.DTYPE_F32: torch.float32}
STORE = {R.DTYPE_BF16: O.STORE_BF16, R.DTYPE_F32: O.STORE_F32}
GUARD = 1024  # elements of canary on each side of every output


def to_dev(a: np.ndarray, dtype):
    t = torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(TORCH_DTYPE[dtype])
    return t.contiguous()


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


class Guarded:
    """Output buffer with canaries before and after it."""

    def __init__(self, shape, dtype):
        n = int(np.prod(shape))
        self.buf = torch.full((n + 2 * GUARD,), 7.0, dtype=TORCH_DTYPE[dtype], device="cuda")
        self.t = self.buf[GUARD:GUARD + n].view(*shape)
        assert self.t.data_ptr() % 16 == 0

    def intact(self) -> bool:
        return bool((self.buf[:GUARD] == 7.0).all() and (self.buf[-GUARD:] == 7.0).all())


def run_layer(w: R.Workload, inputs=None, with_bias=None):
    """Forward + backward on the GPU through the binding; returns dict of numpy float64 outputs."""
    X, W, b, dY = inputs if inputs is not None else R.make_inputs(w, with_bias=with_bias)
    N, k = X.shape[0], w.b_proj
    dX_, dW_, db_ = Guarded((N, w.d_in), w.dtype), Guarded((w.d_out, w.d_in), w.dtype), Guarded((w.d_out,), w.dtype)
    Y_, Xp_ = Guarded((N, w.d_out), w.dtype), Guarded((k, w.d_in), w.dtype)
    Xd, Wd, dYd = to_dev(X, w.dtype), to_dev(W, w.dtype), to_dev(dY, w.dtype)
    bd = to_dev(b, w.dtype) if b is not None else None
    ws = P.alloc_workspace(N, w.d_in, w.d_out, k, w.dtype)
    P.rmm_forward(Xd, Wd, bd, w.seed, k, w.dist, Y=Y_.t, X_proj=Xp_.t, workspace=ws)
    torch.cuda.synchronize()
    assert P.rmm_last_device_status(ws) == P.RMM_OK
    P.rmm_backward(dYd, Wd, Xp_.t, w.seed, w.dist, dX=dX_.t, dW=dW_.t, db=db_.t, workspace=ws)
    torch.cuda.synchronize()
    assert P.rmm_last_device_status(ws) == P.RMM_OK
    for g in (Y_, Xp_, dX_, dW_, db_):
        assert g.intact(), "write outside an output buffer"
    return {"Y": to_np(Y_.t), "X_proj": to_np(Xp_.t), "dX": to_np(dX_.t), "dW": to_np(dW_.t), "db": to_np(db_.t),
            "inputs": (X, W, b, dY)}


def oracle_layer(w: R.Workload, inputs, gpu_xproj=None):
    """The oracle on the same inputs.  Backward is fed the GPU's saved X_proj when given
    (stage-wise parity, what rmm_backward itself receives), else the oracle's own."""
    X, W, b, dY = [None if a is None else a.astype(np.float64) for a in inputs]
    S = O.generate_s(w.seed, X.shape[0], w.b_proj, w.dist, STORE[w.dtype])
    Y, Xp = O.forward(X, W, b, S)
    dX, dW, db, G = O.backward(dY, W, Xp if gpu_xproj is None else gpu_xproj, S)
    return {"Y": Y, "X_proj": Xp, "dX": dX, "dW": dW, "db": db, "G": G, "S": S}


def assert_parity(got, ref, dtype, names=("Y", "X_proj", "dX", "dW", "db")):
    errs = {n: O.rel_frobenius(got[n], ref[n]) for n in names}
    bad = {n: e for n, e in errs.items() if not e <= TOL[dtype]}
    assert not bad, f"relative Frobenius error above {TOL[dtype]}: {bad} (all: {errs})"
    return errs
