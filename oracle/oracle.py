"""ctypes front end of the CPU fp64 oracle (oracle/rmm_oracle.c).

Test infrastructure, not the product: a plain restatement of Algorithm 1 and of
Eq. 1-5 / Lemmas 1-2 of the paper, used to check the CUDA library.  It imports
nothing from the product package and the product imports nothing from here.

All tensors are numpy float64, C-contiguous.  Inputs that went to the GPU as bf16
or fp32 are widened to float64 without change before they come here.
"""
import ctypes as C

import numpy as np

from . import build as _build

DIST_GAUSSIAN, DIST_RADEMACHER, DIST_IDENTITY, DIST_SORS, DIST_DCT = 0, 1, 2, 3, 4
STORE_BF16, STORE_F32 = 0, 1

_lib = C.CDLL(_build.build())
_f64p = np.ctypeslib.ndpointer(dtype=np.float64, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(dtype=np.uint32, flags="C_CONTIGUOUS")
_i64 = C.c_int64

_lib.oracle_num_threads.restype = C.c_int
_lib.oracle_set_num_threads.argtypes = [C.c_int]
_lib.oracle_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
_lib.oracle_bf16_round.argtypes = [C.c_float]
_lib.oracle_bf16_round.restype = C.c_float
_lib.oracle_gauss_pair.argtypes = [C.c_uint32, C.POINTER(C.c_float), C.POINTER(C.c_float)]
_lib.oracle_scale.argtypes = [_i64, C.c_int]
_lib.oracle_scale.restype = C.c_float
_lib.oracle_generate_p_cols.argtypes = [C.c_uint64, _i64, _i64, _i64, _i64, C.c_int, C.c_int, _f32p]
_lib.oracle_generate_s.argtypes = [C.c_uint64, _i64, _i64, C.c_int, C.c_int, _f64p]
_lib.oracle_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, _i64, _i64, _i64, C.c_void_p, _i64,
                                C.c_void_p, C.c_void_p]
_lib.oracle_backward.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, _i64, _i64, _i64, C.c_void_p, _i64,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.oracle_exact_dw.argtypes = [_f64p, _f64p, _i64, _i64, _i64, _f64p]
for _n in ("oracle_d2_sgd", "oracle_alpha"):
    getattr(_lib, _n).argtypes = [_f64p, _f64p, _i64, _i64, _i64]
    getattr(_lib, _n).restype = C.c_double
for _n in ("oracle_d2_rmm_printed", "oracle_d2_rmm_gaussian", "oracle_d2_rmm_rademacher"):
    getattr(_lib, _n).argtypes = [_f64p, _f64p, _i64, _i64, _i64, _i64]
    getattr(_lib, _n).restype = C.c_double


def _c(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def num_threads() -> int:
    return int(_lib.oracle_num_threads())


def set_num_threads(n: int) -> None:
    _lib.oracle_set_num_threads(int(n))


def philox4x32_10(ctr, key):
    """Philox4x32-10 block function: 4 counter words, 2 key words -> 4 output words."""
    out = np.zeros(4, dtype=np.uint32)
    _lib.oracle_philox4x32_10(np.asarray(ctr, dtype=np.uint32), np.asarray(key, dtype=np.uint32), out)
    return out


def bf16_round(x: float) -> float:
    return float(_lib.oracle_bf16_round(float(x)))


def gauss_pair(word: int):
    """The two normals (fp32, before storage rounding) that one Philox word gives."""
    a, b = C.c_float(), C.c_float()
    _lib.oracle_gauss_pair(int(word), C.byref(a), C.byref(b))
    return a.value, b.value


def scale(k: int, dist: int) -> float:
    """c with S = c * P (Eq. 5): fp32 1/sqrt(k), or 1 for the identity test matrix."""
    return float(_lib.oracle_scale(int(k), int(dist)))


def generate_p(seed, N, k, dist, storage, j0=0, j1=None):
    """Unscaled entries P[:, j0:j1] after rounding to the storage type (fp32 array)."""
    j1 = k if j1 is None else j1
    out = np.zeros((N, j1 - j0), dtype=np.float32)
    _lib.oracle_generate_p_cols(int(seed), N, k, j0, j1, int(dist), int(storage), out)
    return out


def generate_s(seed, N, k, dist, storage):
    """S = c * P as float64 [N, k] (Eq. 5)."""
    S = np.zeros((N, k), dtype=np.float64)
    _lib.oracle_generate_s(int(seed), N, k, int(dist), int(storage), S)
    return S


def forward(X, W, b, S, want_y=True, want_xproj=True):
    """Algorithm 1 FORWARD: (Y, X_proj) = (X W^T + 1 b^T, S^T X)."""
    X, W, S = _c(X), _c(W), _c(S)
    b = None if b is None else _c(b)
    N, Din = X.shape
    Dout = W.shape[0]
    k = S.shape[1]
    assert W.shape == (Dout, Din) and S.shape[0] == N
    Y = np.zeros((N, Dout)) if want_y else None
    Xp = np.zeros((k, Din)) if want_xproj else None
    _lib.oracle_forward(_ptr(X), _ptr(W), _ptr(b), N, Din, Dout, _ptr(S), k, _ptr(Y), _ptr(Xp))
    return Y, Xp


def backward(dY, W, Xproj, S, want_dx=True, want_dw=True, want_db=True):
    """Algorithm 1 BACKWARD: returns (dX, dW, db, G) with G = S^T dY."""
    dY, W, Xproj, S = _c(dY), _c(W), _c(Xproj), _c(S)
    N, Dout = dY.shape
    Din = W.shape[1]
    k = S.shape[1]
    assert W.shape == (Dout, Din) and Xproj.shape == (k, Din) and S.shape[0] == N
    dX = np.zeros((N, Din)) if want_dx else None
    dW = np.zeros((Dout, Din)) if want_dw else None
    db = np.zeros(Dout) if want_db else None
    G = np.zeros((k, Dout)) if want_dw else None
    _lib.oracle_backward(_ptr(dY), _ptr(W), _ptr(Xproj), N, Din, Dout, _ptr(S), k,
                         _ptr(dX), _ptr(dW), _ptr(db), _ptr(G))
    return dX, dW, db, G


def exact_dw(dY, X):
    """Exact weight gradient dY^T X (Eq. 3)."""
    dY, X = _c(dY), _c(X)
    dW = np.zeros((dY.shape[1], X.shape[1]))
    _lib.oracle_exact_dw(dY, X, X.shape[0], X.shape[1], dY.shape[1], dW)
    return dW


def d2_sgd(X, Y):
    """Lemma 1, Eq. 9."""
    X, Y = _c(X), _c(Y)
    return float(_lib.oracle_d2_sgd(X, Y, X.shape[0], X.shape[1], Y.shape[1]))


def d2_rmm_printed(X, Y, Bproj):
    """Lemma 2, Eq. 11 exactly as printed (minus sign)."""
    X, Y = _c(X), _c(Y)
    return float(_lib.oracle_d2_rmm_printed(X, Y, X.shape[0], X.shape[1], Y.shape[1], Bproj))


def d2_rmm_gaussian(X, Y, Bproj):
    """E|X^T S S^T Y - X^T Y|_F^2 for Gaussian S with the fourth moment kept."""
    X, Y = _c(X), _c(Y)
    return float(_lib.oracle_d2_rmm_gaussian(X, Y, X.shape[0], X.shape[1], Y.shape[1], Bproj))


def d2_rmm_rademacher(X, Y, Bproj):
    """The same expectation for Rademacher S."""
    X, Y = _c(X), _c(Y)
    return float(_lib.oracle_d2_rmm_rademacher(X, Y, X.shape[0], X.shape[1], Y.shape[1], Bproj))


def alpha(X, Y):
    """Theorem 1, Eq. 13."""
    X, Y = _c(X), _c(Y)
    return float(_lib.oracle_alpha(X, Y, X.shape[0], X.shape[1], Y.shape[1]))


def rel_frobenius(a, ref) -> float:
    """|a - ref|_F / |ref|_F (the parity measure); 0/0 counts as 0."""
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = float(np.linalg.norm(ref))
    num = float(np.linalg.norm(a - ref))
    return 0.0 if num == 0.0 else (num / den if den > 0 else float("inf"))
