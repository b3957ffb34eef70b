"""Seeded synthetic inputs for the RMM linear layer: shapes and value distributions only.

This module serves both the CUDA tests/benchmark and the CPU oracle.  It holds none
of the method's arithmetic: no sketch matrix, no contraction.  Every tensor is drawn
with numpy's PCG64 generator from a seed derived from (config name, tensor name),
rounded once to the storage type, and the identical values go to both sides.

The shapes stand in for the linear layers of RoBERTa-base / RoBERTa-large fine-tuning
(token rows = batch x sequence length); the value distributions are Gaussian with the
variances listed per workload.
"""
import zlib
from dataclasses import dataclass

import numpy as np

DIST_GAUSSIAN, DIST_RADEMACHER, DIST_IDENTITY, DIST_SORS, DIST_DCT = 0, 1, 2, 3, 4
DTYPE_BF16, DTYPE_F32 = 0, 1


def bproj_from_rho(n_tokens: int, rho: float) -> int:
    """B_proj = rho * B rounded to the nearest integer, at least 1 (Section 2.4.2)."""
    return max(1, int(np.floor(rho * n_tokens + 0.5)))


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: int          # DTYPE_BF16 or DTYPE_F32
    n_tokens: int
    d_in: int
    d_out: int
    rho: float
    dist: int
    seed: int
    x_std: float = 1.0
    w_std: float = 0.02
    dy_std: float = 0.01
    b_std: float = 0.0
    k_fixed: int = 0    # when > 0: B_proj given directly instead of through rho (labelled variants)

    @property
    def b_proj(self) -> int:
        return self.k_fixed if self.k_fixed > 0 else bproj_from_rho(self.n_tokens, self.rho)

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == DTYPE_BF16 else 4

    def flops(self) -> dict:
        """Arithmetic of one forward+backward (Section 2.4.2, Table 1), in FLOPs."""
        n, di, do, k = self.n_tokens, self.d_in, self.d_out, self.b_proj
        f = {"y": 2 * n * di * do, "sketch": 2 * n * k * di, "dx": 2 * n * di * do,
             "sdy": 2 * n * k * do, "dw": 2 * k * di * do}
        f["total"] = sum(f.values())
        f["exact_layer"] = 6 * n * di * do
        return f

    def saved_bytes(self) -> dict:
        """Activation bytes kept between the passes: X_proj + seed vs the whole X."""
        return {"rmm": self.b_proj * self.d_in * self.elem_bytes + 8,
                "standard": self.n_tokens * self.d_in * self.elem_bytes}


def _w(name, dtype, n, di, do, rho, dist, seed, **kw):
    return Workload(name, dtype, n, di, do, rho, dist, seed, **kw)


WORKLOADS = {w.name: w for w in [
    # single fp32 layer, rho = 0.5, seed 0
    _w("fp32_768x768_rho0.5", DTYPE_F32, 512, 768, 768, 0.5, DIST_GAUSSIAN, 0,
       w_std=float(np.sqrt(1.0 / 768.0)), dy_std=1.0),
    # RoBERTa-base FFN-up
    _w("base_ffn_up_rho0.1", DTYPE_BF16, 4096, 768, 3072, 0.1, DIST_GAUSSIAN, 1),
    _w("base_ffn_up_rho0.2", DTYPE_BF16, 4096, 768, 3072, 0.2, DIST_GAUSSIAN, 2),
    _w("base_ffn_up_rho0.5", DTYPE_BF16, 4096, 768, 3072, 0.5, DIST_GAUSSIAN, 3),
    _w("base_ffn_up_rho0.9", DTYPE_BF16, 4096, 768, 3072, 0.9, DIST_GAUSSIAN, 4),
    # RoBERTa-base FFN-down and fused QKV, Rademacher
    _w("base_ffn_down_rad_rho0.2", DTYPE_BF16, 4096, 3072, 768, 0.2, DIST_RADEMACHER, 5),
    _w("base_qkv_rad_rho0.2", DTYPE_BF16, 4096, 768, 2304, 0.2, DIST_RADEMACHER, 6),
    # RoBERTa-large
    _w("large_ffn_up_rho0.1", DTYPE_BF16, 16384, 1024, 4096, 0.1, DIST_GAUSSIAN, 7),
    _w("large_ffn_down_rho0.1", DTYPE_BF16, 16384, 4096, 1024, 0.1, DIST_GAUSSIAN, 8),
    # tile-aligned variant of the RoBERTa-large shape: B_proj raised to the next value for which B_proj + 1 (the
    # sketch rows plus the row of ones that carries db) fills whole 128-row tiles: 13 * 128 - 1.  Same tile count
    # and cost as B_proj = 1638, 1.5 % more sketch rows (lower variance); reported in addition, never instead.
    _w("large_ffn_up_k1663_aligned", DTYPE_BF16, 16384, 1024, 4096, 1663 / 16384, DIST_GAUSSIAN, 10, k_fixed=1663),
    # the RoBERTa-large shape with the subsampled-Hadamard sketch (in bf16 mode applied by the two-level Walsh-Hadamard
    # transform; the dense contraction with the same S only outside Hadamard orders 128 .. 16384)
    _w("large_ffn_up_sors_rho0.1", DTYPE_BF16, 16384, 1024, 4096, 0.1, DIST_SORS, 11),
    # the RoBERTa-large shape with the subsampled-DCT sketch (dense contraction with generated cosines)
    _w("large_ffn_up_dct_rho0.1", DTYPE_BF16, 16384, 1024, 4096, 0.1, DIST_DCT, 12),
    # diagnostic: the RoBERTa-large shape with the cheap sketch distribution (isolates the cost of the normals)
    _w("large_ffn_up_rad_rho0.1", DTYPE_BF16, 16384, 1024, 4096, 0.1, DIST_RADEMACHER, 9),
]}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of fp32 values to bfloat16, returned as fp32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of fp32 values that are already bf16-representable."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    assert not np.any(u & np.uint32(0xFFFF)), "values are not bf16-representable"
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(workload_name: str, tensor: str) -> np.random.Generator:
    return np.random.default_rng([zlib.crc32(workload_name.encode()), zlib.crc32(tensor.encode())])


def normal_tensor(workload_name, tensor, shape, std, dtype):
    """fp32 array of N(0, std^2) draws, rounded once to the storage dtype."""
    a = _rng(workload_name, tensor).standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(std)
    return round_to_bf16(a) if dtype == DTYPE_BF16 else a


def make_inputs(w: Workload, n_tokens=None, with_bias=None):
    """X [N,D_in], W [D_out,D_in], b [D_out], dY [N,D_out] as fp32 arrays holding
    values representable in the workload's storage type.  ``n_tokens`` overrides the
    row count (a bounded sample of the same workload)."""
    n = w.n_tokens if n_tokens is None else n_tokens
    b_std = w.b_std if with_bias is None else with_bias
    X = normal_tensor(w.name, "X", (n, w.d_in), w.x_std, w.dtype)
    W = normal_tensor(w.name, "W", (w.d_out, w.d_in), w.w_std, w.dtype)
    dY = normal_tensor(w.name, "dY", (n, w.d_out), w.dy_std, w.dtype)
    b = normal_tensor(w.name, "b", (w.d_out,), b_std, w.dtype) if b_std else np.zeros(w.d_out, np.float32)
    return X, W, b, dY


def small_case(name, dtype, n, d_in, d_out, k, dist, seed, bias=True):
    """A small ragged parity case with the same value distributions."""
    w = Workload(name, dtype, n, d_in, d_out, k / n, dist, seed, b_std=0.5 if bias else 0.0)
    assert w.b_proj == k, (w.b_proj, k)
    return w
