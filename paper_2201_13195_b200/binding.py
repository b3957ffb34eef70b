"""ctypes binding of librmm.so (include/rmm.h): argument marshalling only.

Every step of the layer runs in the CUDA kernels of the library; PyTorch is used here
for device memory and streams.  There is no fallback: if the library has not been
built, importing this module raises.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# RMM_LIBRARY names another build of the same library (e.g. the cycle-accounting build made by
# `python -m paper_2201_13195_b200.build --trace FILE`); by default the in-tree librmm.so is loaded.
LIB_PATH = os.environ.get("RMM_LIBRARY") or os.path.join(_HERE, "librmm.so")

RMM_OK, RMM_ERR_INVALID_ARG, RMM_ERR_UNSUPPORTED, RMM_ERR_WORKSPACE, RMM_ERR_CUDA, RMM_ERR_TIMEOUT = range(6)
RMM_DIST_GAUSSIAN, RMM_DIST_RADEMACHER, RMM_DIST_IDENTITY, RMM_DIST_SORS_HADAMARD, RMM_DIST_SORS_DCT = 0, 1, 2, 3, 4
RMM_DTYPE_BF16, RMM_DTYPE_F32 = 0, 1

EXPORTS = ("rmm_workspace_bytes", "rmm_workspace_bytes_for", "rmm_forward", "rmm_backward", "rmm_debug_generate_s",
           "rmm_last_device_status", "rmm_status_string", "rmm_host_staging_bytes",
           "rmm_forward_host", "rmm_backward_host", "rmm_profile_enable", "rmm_profile_read",
           "rmm_bias_grad_static", "rmm_debug_gauss_words", "rmm_debug_sketch_schedule",
           "rmm_variance_probe_workspace_bytes", "rmm_variance_probe", "rmm_debug_pass_schedule", "rmm_debug_hadamard_plan", "rmm_layer_launch_count", "rmm_set_pass_mode")
RMM_BIAS_GRAD_STATIC_MAX_D_OUT = 4096
STEP_NAMES = ("y", "sketch", "dx", "sdy", "dw", "db", "fwd", "bwd")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2201_13195_b200.build` "
                      "(there is no non-CUDA path)")
_lib = C.CDLL(LIB_PATH)

_i64, _vp, _u64, _int, _sz = C.c_int64, C.c_void_p, C.c_uint64, C.c_int, C.c_size_t
_lib.rmm_workspace_bytes.argtypes = [_i64, _i64, _i64, _i64, _int]
_lib.rmm_workspace_bytes.restype = _sz
_lib.rmm_workspace_bytes_for.argtypes = [_i64, _i64, _i64, _i64, _int, _int]
_lib.rmm_workspace_bytes_for.restype = _sz
_lib.rmm_forward.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _u64, _i64, _int, _int, _vp, _vp, _vp, _sz, _vp]
_lib.rmm_forward.restype = _int
_lib.rmm_backward.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _u64, _i64, _int, _int, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.rmm_backward.restype = _int
_lib.rmm_debug_generate_s.argtypes = [_u64, _i64, _i64, _int, _int, _vp, _vp]
_lib.rmm_debug_generate_s.restype = _int
_lib.rmm_last_device_status.argtypes = [_vp]
_lib.rmm_last_device_status.restype = _int
_lib.rmm_status_string.argtypes = [_int]
_lib.rmm_status_string.restype = C.c_char_p
_lib.rmm_host_staging_bytes.argtypes = [_i64, _i64, _i64, _i64, _int, _int, _int]
_lib.rmm_host_staging_bytes.restype = _sz
_lib.rmm_forward_host.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _u64, _i64, _int, _int, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.rmm_forward_host.restype = _int
_lib.rmm_backward_host.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _u64, _i64, _int, _int, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.rmm_backward_host.restype = _int
_lib.rmm_bias_grad_static.argtypes = [_vp, _i64, _i64, _int, _vp, _vp]
_lib.rmm_bias_grad_static.restype = _int
_lib.rmm_debug_gauss_words.argtypes = [_vp, _i64, _vp, _vp]
_lib.rmm_debug_gauss_words.restype = _int
_lib.rmm_debug_sketch_schedule.argtypes = [_i64, _i64, _i64, _int, _int, _vp, _i64, _vp]
_lib.rmm_debug_sketch_schedule.restype = _i64
_lib.rmm_debug_pass_schedule.argtypes = [_i64, _i64, _i64, _i64, _i64, _i64, _int, _vp, _i64]
_lib.rmm_debug_pass_schedule.restype = _i64
_lib.rmm_debug_hadamard_plan.argtypes = [_i64, _i64, _i64, _sz, C.POINTER(C.c_int64)]
_lib.rmm_debug_hadamard_plan.restype = _int
_lib.rmm_variance_probe_workspace_bytes.argtypes = [_i64, _i64, _i64]
_lib.rmm_variance_probe_workspace_bytes.restype = _sz
_lib.rmm_variance_probe.argtypes = [_vp, _vp, _i64, _i64, _i64, _i64, _int, _int, _vp, _vp, _vp, _sz, _vp]
_lib.rmm_variance_probe.restype = _int
_lib.rmm_set_pass_mode.argtypes = [_int]
_lib.rmm_set_pass_mode.restype = _int
_lib.rmm_layer_launch_count.argtypes = []
_lib.rmm_layer_launch_count.restype = _i64
_lib.rmm_profile_enable.argtypes = [_int]
_lib.rmm_profile_enable.restype = _int
_lib.rmm_profile_read.argtypes = [C.POINTER(C.c_int), C.POINTER(C.c_float), _int]
_lib.rmm_profile_read.restype = _int


class RmmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {rmm_status_string(code)}")


def rmm_status_string(code: int) -> str:
    return _lib.rmm_status_string(int(code)).decode()


def _check(code, where):
    if code != RMM_OK:
        raise RmmError(code, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return RMM_DTYPE_BF16
    if t.dtype == torch.float32:
        return RMM_DTYPE_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream_ptr(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def rmm_workspace_bytes(N, D_in, D_out, B_proj, dt) -> int:
    return int(_lib.rmm_workspace_bytes(N, D_in, D_out, B_proj, dt))


def rmm_workspace_bytes_for(N, D_in, D_out, B_proj, dt, dist) -> int:
    return int(_lib.rmm_workspace_bytes_for(N, D_in, D_out, B_proj, dt, dist))


def alloc_workspace(N, D_in, D_out, B_proj, dt, device="cuda", dist=None):
    """A workspace of the smallest valid size, or (with `dist`) of the size that suits that sketch best."""
    nbytes = rmm_workspace_bytes(N, D_in, D_out, B_proj, dt) if dist is None else \
        rmm_workspace_bytes_for(N, D_in, D_out, B_proj, dt, dist)
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def rmm_forward(X, W, b, seed, B_proj, dist, Y=None, X_proj=None, workspace=None, stream=None, want_y=True):
    """(Y, X_proj) = (X W^T + 1 b^T, S^T X); device tensors, contiguous."""
    N, D_in = X.shape
    D_out = W.shape[0]
    dt = _dtype_code(X)
    assert X.is_cuda and X.is_contiguous() and W.is_contiguous() and W.shape[1] == D_in and W.dtype == X.dtype
    if want_y and Y is None:
        Y = torch.empty((N, D_out), dtype=X.dtype, device=X.device)
    if X_proj is None:
        X_proj = torch.empty((B_proj, D_in), dtype=X.dtype, device=X.device)
    if workspace is None:
        workspace = alloc_workspace(N, D_in, D_out, B_proj, dt, X.device)
    _check(_lib.rmm_forward(_ptr(X), _ptr(W), _ptr(b), N, D_in, D_out, seed, B_proj, dist, dt,
                            _ptr(Y) if want_y else None, _ptr(X_proj), _ptr(workspace), workspace.numel(),
                            _stream_ptr(stream)), "rmm_forward")
    return Y, X_proj


def rmm_backward(dY, W, X_proj, seed, dist, dX=None, dW=None, db=None, workspace=None, stream=None,
                 want_dx=True, want_db=True):
    """(dX, dW, db) = (dY W, (S^T dY)^T X_proj, sum_rows dY)."""
    N, D_out = dY.shape
    D_in = W.shape[1]
    B_proj = X_proj.shape[0]
    dt = _dtype_code(dY)
    assert dY.is_cuda and dY.is_contiguous() and W.is_contiguous() and X_proj.is_contiguous()
    if want_dx and dX is None:
        dX = torch.empty((N, D_in), dtype=dY.dtype, device=dY.device)
    if dW is None:
        dW = torch.empty((D_out, D_in), dtype=dY.dtype, device=dY.device)
    if want_db and db is None:
        db = torch.empty((D_out,), dtype=dY.dtype, device=dY.device)
    if workspace is None:
        workspace = alloc_workspace(N, D_in, D_out, B_proj, dt, dY.device)
    _check(_lib.rmm_backward(_ptr(dY), _ptr(W), _ptr(X_proj), N, D_in, D_out, seed, B_proj, dist, dt,
                             _ptr(dX) if want_dx else None, _ptr(dW), _ptr(db) if want_db else None,
                             _ptr(workspace), workspace.numel(), _stream_ptr(stream)), "rmm_backward")
    return dX, dW, db


def rmm_debug_generate_s(seed, N, B_proj, dist, dtype=torch.bfloat16, device="cuda", stream=None):
    """Unscaled sketch entries P [N, B_proj] as the kernels generate them."""
    out = torch.empty((N, B_proj), dtype=dtype, device=device)
    _check(_lib.rmm_debug_generate_s(seed, N, B_proj, dist, _dtype_code(out), _ptr(out), _stream_ptr(stream)),
           "rmm_debug_generate_s")
    return out


def rmm_last_device_status(workspace) -> int:
    return int(_lib.rmm_last_device_status(_ptr(workspace)))


def rmm_host_staging_bytes(N, D_in, D_out, B_proj, dt, backward, outputs) -> int:
    return int(_lib.rmm_host_staging_bytes(N, D_in, D_out, B_proj, dt, int(backward), int(outputs)))


def rmm_forward_host(X, W, b, seed, B_proj, dist, Y, X_proj, dev_in, dev_out, workspace, stream=None):
    """Host tensors in and out (pinned recommended); copies are part of the call."""
    N, D_in = X.shape
    D_out = W.shape[0]
    dt = _dtype_code(X)
    assert not X.is_cuda and not Y.is_cuda and dev_in.is_cuda and dev_out.is_cuda
    _check(_lib.rmm_forward_host(_ptr(X), _ptr(W), _ptr(b), N, D_in, D_out, seed, B_proj, dist, dt, _ptr(Y),
                                 _ptr(X_proj), _ptr(dev_in), _ptr(dev_out), _ptr(workspace), workspace.numel(),
                                 _stream_ptr(stream)), "rmm_forward_host")
    return Y, X_proj


def rmm_backward_host(dY, W, X_proj, seed, dist, dX, dW, db, dev_in, dev_out, workspace, stream=None):
    N, D_out = dY.shape
    D_in = W.shape[1]
    B_proj = X_proj.shape[0]
    dt = _dtype_code(dY)
    _check(_lib.rmm_backward_host(_ptr(dY), _ptr(W), _ptr(X_proj), N, D_in, D_out, seed, B_proj, dist, dt,
                                  _ptr(dX), _ptr(dW), _ptr(db), _ptr(dev_in), _ptr(dev_out), _ptr(workspace),
                                  workspace.numel(), _stream_ptr(stream)), "rmm_backward_host")
    return dX, dW, db


VARIANCE_FIELDS = ("x_frob2", "dy_frob2", "rownorm_products", "xtdy_frob2", "d2_sgd", "d2_rmm", "d2_rmm_printed", "alpha")


def rmm_variance_probe_workspace_bytes(N, D_in, D_out) -> int:
    return int(_lib.rmm_variance_probe_workspace_bytes(N, D_in, D_out))


def rmm_variance_probe(X, dY, B_proj, dist, out=None, dW_exact=None, workspace=None, stream=None):
    """Device tensor of 8 doubles (VARIANCE_FIELDS) for one layer's X [N, D_in] and dY [N, D_out] (bf16)."""
    N, D_in = X.shape
    D_out = dY.shape[1]
    assert X.is_cuda and dY.is_cuda and X.is_contiguous() and dY.is_contiguous() and dY.shape[0] == N
    if out is None:
        out = torch.empty(8, dtype=torch.float64, device=X.device)
    if workspace is None:
        workspace = torch.empty(rmm_variance_probe_workspace_bytes(N, D_in, D_out), dtype=torch.uint8,
                                device=X.device)
    _check(_lib.rmm_variance_probe(_ptr(X), _ptr(dY), N, D_in, D_out, B_proj, dist, _dtype_code(X), _ptr(out),
                                   _ptr(dW_exact), _ptr(workspace), workspace.numel(), _stream_ptr(stream)),
           "rmm_variance_probe")
    return out


def rmm_profile_enable(capacity: int) -> None:
    """Bracket each kernel launch of the next calls with CUDA events (capacity launches); 0 switches it off."""
    _check(_lib.rmm_profile_enable(int(capacity)), "rmm_profile_enable")


def rmm_profile_read(max_records: int):
    """[(step name, milliseconds)] of the launches recorded since the last read."""
    ids = (C.c_int * max_records)()
    ms = (C.c_float * max_records)()
    n = _lib.rmm_profile_read(ids, ms, max_records)
    return [(STEP_NAMES[ids[i]], float(ms[i])) for i in range(n)]


def rmm_bias_grad_static(dY, db=None, stream=None):
    """db = column sums of dY through the entry point that allocates nothing in the library
    (its scratch is a fixed array inside librmm.so).  Pass `db` to avoid the one output
    allocation this wrapper would otherwise make; D_out is limited to
    RMM_BIAS_GRAD_STATIC_MAX_D_OUT."""
    N, D_out = dY.shape
    assert dY.is_cuda and dY.is_contiguous()
    if db is None:
        db = torch.empty((D_out,), dtype=dY.dtype, device=dY.device)
    _check(_lib.rmm_bias_grad_static(_ptr(dY), N, D_out, _dtype_code(dY), _ptr(db), _stream_ptr(stream)),
           "rmm_bias_grad_static")
    return db


def rmm_debug_gauss_words(words, stream=None):
    """fp32 [n, 2]: the (even, odd) normals the Gaussian transform makes of each uint32 word
    (words: device tensor of n bit patterns stored as int32)."""
    assert words.is_cuda and words.dtype == torch.int32 and words.is_contiguous()
    out = torch.empty((words.numel(), 2), dtype=torch.float32, device=words.device)
    _check(_lib.rmm_debug_gauss_words(_ptr(words), words.numel(), _ptr(out), _stream_ptr(stream)),
           "rmm_debug_gauss_words")
    return out


def rmm_set_pass_mode(mode: int) -> None:
    """0: the two kernels of a pass side by side (default); 1: one launch per pass."""
    _check(_lib.rmm_set_pass_mode(int(mode)), "rmm_set_pass_mode")


TRACE_SLOTS = ("kernel", "producer_wait", "producer_loop", "mma_wait_s", "mma_wait_data", "mma_wait_accumulator",
               "mma_sketch_loop", "mma_dense_loop", "generator_arithmetic", "generator_wait_stage", "generator_loop",
               "drain_wait", "drain", "epilogue_loop", "reduction_wait", "reduction", "generator_store", "generator_fence",
               "generator_handover", "mma_fence", "mma_issue", "mma_commit")


def rmm_debug_pass_trace():
    """Cycle counters of the last sketch or one-launch pass kernel, per CTA: {slot name: [148 values]}.  Only the
    cycle-accounting build of the library (RMM_LIBRARY) exports them; returns None otherwise."""
    if not hasattr(_lib, "rmm_debug_pass_trace"):
        return None
    buf = (C.c_longlong * (148 * 32))()
    _lib.rmm_debug_pass_trace.argtypes = [_vp]
    _lib.rmm_debug_pass_trace.restype = _int
    if _lib.rmm_debug_pass_trace(C.addressof(buf)) != 0:
        return None
    return {name: [int(buf[cta * 32 + i]) for cta in range(148)] for i, name in enumerate(TRACE_SLOTS)}


def rmm_layer_launch_count() -> int:
    return int(_lib.rmm_layer_launch_count())


def rmm_debug_hadamard_plan(rows, cols, tokens, scratch_bytes):
    """How the fast Hadamard transform would take a sketch (host only): dict, or None outside the fast path."""
    info = (C.c_int64 * 4)()
    r = _lib.rmm_debug_hadamard_plan(rows, cols, tokens, scratch_bytes, info)
    if r < 0:
        raise ValueError("invalid arguments")
    if r == 0:
        return None
    return {"order": int(info[0]), "blocks": int(info[1]), "columns_per_round": int(info[2]), "rounds": int(info[3])}


def rmm_debug_pass_schedule(gemm, sketch, max_pairs=74):
    """The static schedule of one pass launch (host only).  gemm = (M, N, K) or None, sketch = (rows, cols, tokens) or None."""
    gm, gn, gk = gemm if gemm else (0, 0, 0)
    rows, cols, tokens = sketch if sketch else (0, 0, 0)
    n = _lib.rmm_debug_pass_schedule(gm, gn, gk, rows, cols, tokens, max_pairs, None, 0)
    if n < 0:
        raise ValueError("invalid arguments")
    buf = (C.c_int64 * n)()
    _lib.rmm_debug_pass_schedule(gm, gn, gk, rows, cols, tokens, max_pairs, C.addressof(buf), n)
    names = ("num_pairs", "gemm_tiles", "tiles_n", "num_kb", "tiles_m", "groups", "nat", "ksteps", "nb", "blen")
    d = {k: int(buf[i]) for i, k in enumerate(names)}
    d["gemm_begin"] = [int(buf[10 + i]) for i in range(d["num_pairs"] + 1)]
    return d


def rmm_debug_sketch_schedule(rows, cols, tokens, max_ctas=148, mode=0):
    """(records, info): the sketch kernels' static schedule as lists of 5-tuples (host only)."""
    info = (C.c_int64 * 8)()
    n = _lib.rmm_debug_sketch_schedule(rows, cols, tokens, max_ctas, mode, None, 0, C.addressof(info))
    buf = (C.c_int64 * (5 * max(n, 1)))()
    _lib.rmm_debug_sketch_schedule(rows, cols, tokens, max_ctas, mode, C.addressof(buf), n, C.addressof(info))
    recs = [tuple(buf[5 * i + j] for j in range(5)) for i in range(n)]
    return recs, {"tiles": info[0], "ksteps": info[1], "num_ctas": info[2], "num_slots": info[3], "cluster": info[4],
                  "rounds": info[5], "full_blocks": info[6], "w_last": info[7]}
