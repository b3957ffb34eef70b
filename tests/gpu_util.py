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
    return {"Y": Y, "X_proj": Xp, "dX": dX, "dW": dW, "db": db, "G": G, "S": S,
            "X_proj_used": Xp if gpu_xproj is None else np.asarray(gpu_xproj, np.float64)}


# Element-wise gate beside the Frobenius one.  For an output element with fp64 reference value r, contraction
# length K and rms = root mean square of the reference tensor:
#   bf16 mode: |got - r| <= 2^-8 |r| + (2^-10 + K 2^-23) rms [+ operand term].  2^-8 |r| is the rounding of
#     the result to bf16 (half of the spacing 2^-7 of bf16 values with the magnitude of r).  The rms term
#     covers what does not scale with |r|: the fp32 accumulation of K exact bf16 x bf16 products in the tensor
#     core (each addition may lose up to 2^-23 of a partial sum whose size is of the order of rms: K 2^-23 rms
#     if every loss had the same sign) plus a floor of 2^-10 for the rounding boundary moving with that error.
#     Operand term, dW only: the operand G = S^T dY has itself been rounded to bf16 (relative error at most
#     2^-8 per entry), so element (o, i) of dW = G^T X_proj may be off by 2^-8 sum_j |G[j,o]| |X_proj[j,i]|;
#     end to end, where the oracle's X_proj is not rounded either, by twice that (first order).
#   fp32 mode: |got - r| <= 2^-20 |r| + sqrt(K) 2^-19 rms (fp32 FMA chain of length K: rounding errors of size
#     2^-24 times the partial sums, adding up like a random walk; sixteen times that as the allowance).
#   Subsampled-Hadamard sketch in bf16 mode (applied by the two-level Walsh-Hadamard transform): the first
#     level's result T is stored in bf16, so every element of X_proj and of G carries one more rounding whose
#     sum over the L/128 blocks has standard deviation 2^-9/sqrt(3) sqrt(L/N) rms <= 1.6e-3 rms (L = Hadamard
#     order < 2N), whatever the element's size: 2^-6 rms (ten standard deviations) is added for X_proj and dW.
# A wrong element (a mis-clipped store box, a stale 16-byte chunk, a missing partial tile) is off by the order
# of rms and fails this gate by an order of magnitude or more, while it passes the Frobenius gate.
SORS_FAST_PATH_EXTRA = 2.0 ** -6


def elementwise_excess(got, ref, dtype, K, operand_term=None, extra_rms=0.0):
    """max over elements of |got - ref| / bound; <= 1 passes.  Returns (excess, index of the worst element)."""
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    assert got.shape == ref.shape
    if ref.size == 0:
        return 0.0, ()
    rms = float(np.sqrt(np.mean(ref * ref)))
    if dtype == R.DTYPE_BF16:
        rel, a = 2.0 ** -8, 2.0 ** -10 + K * 2.0 ** -23
    else:
        rel, a = 2.0 ** -20, np.sqrt(K) * 2.0 ** -19
    bound = rel * np.abs(ref) + (a + extra_rms) * rms + 1e-300
    if operand_term is not None:
        bound = bound + operand_term
    ratio = np.abs(got - ref) / bound
    i = int(np.argmax(ratio))
    return float(ratio.flat[i]), np.unravel_index(i, ratio.shape)


def dw_operand_term(G, Xp, dtype, end_to_end=False):
    """Allowance for the bf16 rounding of G (and, end to end, of X_proj) in dW = G^T X_proj; zero in fp32 mode."""
    if dtype != R.DTYPE_BF16:
        return None
    return (2.0 if end_to_end else 1.0) * 2.0 ** -8 * (np.abs(G).T @ np.abs(Xp))


def contraction_lengths(N, d_in, d_out, k):
    """Length of the sum behind one element of each output tensor."""
    return {"Y": d_in, "X_proj": N, "dX": d_out, "dW": k, "db": N}


def assert_parity(got, ref, dtype, names=("Y", "X_proj", "dX", "dW", "db"), K=None, end_to_end=False, dist=None):
    """Relative Frobenius error per tensor within TOL and, when the contraction lengths K are given, every
    element within the element-wise bound above (ref must then hold the oracle's G and X_proj as well)."""
    errs = {n: O.rel_frobenius(got[n], ref[n]) for n in names}
    bad = {n: e for n, e in errs.items() if not e <= TOL[dtype]}
    assert not bad, f"relative Frobenius error above {TOL[dtype]}: {bad} (all: {errs})"
    if K is not None:
        for n in names:
            term = dw_operand_term(ref["G"], ref["X_proj_used"], dtype, end_to_end) if n == "dW" else None
            extra = SORS_FAST_PATH_EXTRA if (dist == R.DIST_SORS and dtype == R.DTYPE_BF16 and n in ("X_proj", "dW")) else 0.0
            ex, where = elementwise_excess(got[n], ref[n], dtype, K[n], term, extra)
            assert ex <= 1.0, f"{n}{list(where)}: |got - ref| is {ex:.2f} x its element-wise bound " \
                              f"(got {np.asarray(got[n])[where]}, ref {np.asarray(ref[n])[where]})"
    return errs
