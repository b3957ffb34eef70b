"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs.  S bit-exact; Y, X_proj, dX, dW, db within a relative Frobenius error
of 1e-2 (bf16 mode) or 1e-5 (fp32 mode)."""
import numpy as np
import pytest
import torch

import rmm_inputs as R
from oracle import oracle as O

pytestmark = pytest.mark.gpu

from tests.gpu_util import (STORE, TOL, TORCH_DTYPE, assert_parity, oracle_layer, run_layer, to_dev, to_np)  # noqa: E402


def _P():
    import paper_2201_13195_b200 as P
    return P


# ------------------------------------------------------------------ S bit-exact
@pytest.mark.parametrize("dtype", [R.DTYPE_BF16, R.DTYPE_F32])
@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER, R.DIST_SORS])
@pytest.mark.parametrize("N,k,seed", [(37, 5, 0), (300, 130, 0xDEADBEEF12345678), (1024, 64, 3)])
def test_sketch_dump_bit_exact(dtype, dist, N, k, seed):
    P = _P()
    got = P.rmm_debug_generate_s(seed, N, k, dist, dtype=TORCH_DTYPE[dtype])
    want = O.generate_p(seed, N, k, dist, STORE[dtype])
    assert np.array_equal(got.to(torch.float32).cpu().numpy(), want)


def test_gaussian_transform_bit_exact_on_all_radius_and_angle_inputs():
    """Every one of the 2^16 radius inputs (with three angle patterns) and of the 2^16 angle
    inputs (with three radius patterns) of the uniform -> normal map, bit for bit."""
    P = _P()
    hi = np.arange(65536, dtype=np.uint64)
    words = np.concatenate([(hi << 16) | lo for lo in (16383, 0x8001, 0x5A5A)] +
                           [(np.uint64(h) << 16) | hi for h in (0, 20000, 65535)]).astype(np.uint32)
    got = P.rmm_debug_gauss_words(torch.from_numpy(words.view(np.int32)).cuda()).cpu().numpy()
    want = np.array([O.gauss_pair(int(w)) for w in words], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("dtype", [R.DTYPE_BF16, R.DTYPE_F32])
@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER, R.DIST_SORS])
def test_production_kernel_sketch_bit_exact(dtype, dist):
    """X = I makes X_proj = c * P^T: the sketch kernel's own S, entry by entry."""
    P = _P()
    N, k, seed = 328, 141, 77
    X = torch.eye(N, dtype=TORCH_DTYPE[dtype], device="cuda")
    W = torch.zeros((8, N), dtype=TORCH_DTYPE[dtype], device="cuda")
    _, Xp = P.rmm_forward(X, W, None, seed, k, dist, want_y=False)
    torch.cuda.synchronize()
    Pm = O.generate_p(seed, N, k, dist, STORE[dtype])                 # [N, k] fp32
    want = (Pm.T * np.float32(O.scale(k, dist))).astype(np.float32)   # one fp32 multiply per entry
    if dtype == R.DTYPE_BF16:
        want = R.round_to_bf16(want)
    assert np.array_equal(Xp.to(torch.float32).cpu().numpy(), want)


# ------------------------------------------------------------------ whole layer, small and ragged
CASES = [
    # name, dtype, N, D_in, D_out, k, dist
    ("tiny_ragged_f32", R.DTYPE_F32, 37, 24, 40, 5, R.DIST_GAUSSIAN),
    ("tiny_ragged_bf16", R.DTYPE_BF16, 37, 24, 40, 5, R.DIST_GAUSSIAN),
    ("one_row", R.DTYPE_BF16, 1, 8, 8, 1, R.DIST_GAUSSIAN),
    ("one_row_f32", R.DTYPE_F32, 1, 3, 5, 1, R.DIST_RADEMACHER),
    ("multi_tile_ragged_bf16", R.DTYPE_BF16, 300, 264, 520, 130, R.DIST_GAUSSIAN),
    ("multi_tile_ragged_rad", R.DTYPE_BF16, 389, 520, 264, 77, R.DIST_RADEMACHER),
    ("multi_tile_ragged_f32", R.DTYPE_F32, 150, 70, 130, 66, R.DIST_RADEMACHER),
    ("rho_one_gauss", R.DTYPE_BF16, 200, 72, 136, 200, R.DIST_GAUSSIAN),
    ("k_multiple_of_tile", R.DTYPE_BF16, 512, 128, 256, 256, R.DIST_GAUSSIAN),
    ("sors_ragged_bf16", R.DTYPE_BF16, 389, 264, 520, 77, R.DIST_SORS),
    ("sors_ragged_f32", R.DTYPE_F32, 150, 70, 130, 66, R.DIST_SORS),
    ("sors_below_fast_path", R.DTYPE_BF16, 37, 24, 40, 5, R.DIST_SORS),          # Hadamard order 64: dense kernel
    ("sors_one_block", R.DTYPE_BF16, 128, 64, 72, 128, R.DIST_SORS),             # order 128: one block, no second level
    ("sors_many_blocks", R.DTYPE_BF16, 2100, 136, 200, 300, R.DIST_SORS),        # order 4096: 32 blocks, last ones empty
    # dX has 38 x 2 = 76 tiles of 256 x 256: more than the 74 CTA pairs, so two pairs take a second tile
    # (both accumulator buffers in use), with ragged last rows: 9700 = 37 * 256 + 228
    ("dx_second_wave", R.DTYPE_BF16, 9700, 512, 64, 16, R.DIST_RADEMACHER),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_layer_parity_small(case):
    name, dtype, N, Di, Do, k, dist = case
    w = R.small_case(name, dtype, N, Di, Do, k, dist, seed=len(name) * 1000003)
    got = run_layer(w)
    ref = oracle_layer(w, got["inputs"], gpu_xproj=got["X_proj"])
    assert_parity(got, ref, dtype)
    # end to end (oracle's own fp64 X_proj in backward)
    ref2 = oracle_layer(w, got["inputs"])
    assert_parity(got, ref2, dtype, names=("dW",))


def test_identity_sketch_is_exact_layer():
    """rho = 1 with S = I: X_proj == X bit for bit and dW is the exact dY^T X."""
    w = R.small_case("identity", R.DTYPE_BF16, 192, 136, 264, 192, R.DIST_IDENTITY, seed=5)
    got = run_layer(w)
    X, W, b, dY = got["inputs"]
    assert np.array_equal(got["X_proj"], X.astype(np.float64))
    assert O.rel_frobenius(got["dW"], O.exact_dw(dY.astype(np.float64), X.astype(np.float64))) <= TOL[R.DTYPE_BF16]


def test_fp32_config_parity():
    w = R.WORKLOADS["fp32_768x768_rho0.5"]
    got = run_layer(w)
    ref = oracle_layer(w, got["inputs"], gpu_xproj=got["X_proj"])
    errs = assert_parity(got, ref, w.dtype)
    print("fp32 config errors", errs)


def test_determinism_and_seed_dependence():
    w = R.small_case("determinism", R.DTYPE_BF16, 260, 136, 264, 70, R.DIST_GAUSSIAN, seed=9)
    a, b_ = run_layer(w), run_layer(w)
    for n in ("Y", "X_proj", "dX", "dW", "db"):
        assert np.array_equal(a[n], b_[n]), n
    w2 = R.Workload(w.name, w.dtype, w.n_tokens, w.d_in, w.d_out, w.rho, w.dist, w.seed + 1, b_std=w.b_std)
    c = run_layer(w2)
    assert np.array_equal(a["Y"], c["Y"]) and np.array_equal(a["dX"], c["dX"])
    assert not np.array_equal(a["X_proj"], c["X_proj"])


def test_optional_outputs_and_no_bias():
    P = _P()
    w = R.small_case("optional", R.DTYPE_BF16, 130, 72, 136, 40, R.DIST_RADEMACHER, seed=4, bias=False)
    X, W, b, dY = R.make_inputs(w)
    Xd, Wd, dYd = to_dev(X, w.dtype), to_dev(W, w.dtype), to_dev(dY, w.dtype)
    _, Xp = P.rmm_forward(Xd, Wd, None, w.seed, w.b_proj, w.dist, want_y=False)
    dX, dW, db = P.rmm_backward(dYd, Wd, Xp, w.seed, w.dist, want_dx=False, want_db=False)
    torch.cuda.synchronize()
    assert dX is None and db is None
    ref = oracle_layer(w, (X, W, None, dY), gpu_xproj=to_np(Xp))
    assert O.rel_frobenius(to_np(dW), ref["dW"]) <= TOL[w.dtype]
    assert O.rel_frobenius(to_np(Xp), ref["X_proj"]) <= TOL[w.dtype]


def test_host_buffer_entry_points():
    P = _P()
    w = R.small_case("host", R.DTYPE_BF16, 200, 72, 136, 60, R.DIST_GAUSSIAN, seed=8)
    X, W, b, dY = R.make_inputs(w)
    td = TORCH_DTYPE[w.dtype]
    hX, hW, hb, hdY = [torch.from_numpy(a).to(td).pin_memory() for a in (X, W, b, dY)]
    N, k = w.n_tokens, w.b_proj
    hY = torch.empty((N, w.d_out), dtype=td).pin_memory()
    hXp = torch.empty((k, w.d_in), dtype=td).pin_memory()
    hdX = torch.empty((N, w.d_in), dtype=td).pin_memory()
    hdW = torch.empty((w.d_out, w.d_in), dtype=td).pin_memory()
    hdb = torch.empty((w.d_out,), dtype=td).pin_memory()
    nb = max(P.rmm_host_staging_bytes(N, w.d_in, w.d_out, k, w.dtype, bwd, out) for bwd in (0, 1) for out in (0, 1))
    dev_in = torch.empty(nb, dtype=torch.uint8, device="cuda")
    dev_out = torch.empty(nb, dtype=torch.uint8, device="cuda")
    ws = P.alloc_workspace(N, w.d_in, w.d_out, k, w.dtype)
    P.rmm_forward_host(hX, hW, hb, w.seed, k, w.dist, hY, hXp, dev_in, dev_out, ws)
    P.rmm_backward_host(hdY, hW, hXp, w.seed, w.dist, hdX, hdW, hdb, dev_in, dev_out, ws)
    got = {"Y": hY.float().numpy(), "X_proj": hXp.float().numpy(), "dX": hdX.float().numpy(),
           "dW": hdW.float().numpy(), "db": hdb.float().numpy()}
    ref = oracle_layer(w, (X, W, b, dY), gpu_xproj=got["X_proj"].astype(np.float64))
    assert_parity(got, ref, w.dtype)


# ------------------------------------------------------------------ full-size workloads, sampled outputs
def _sampled_full_size(name, n_samples=48):
    P = _P()
    w = R.WORKLOADS[name]
    X, W, b, dY = R.make_inputs(w)
    N, k, Di, Do = w.n_tokens, w.b_proj, w.d_in, w.d_out
    Xd, Wd, dYd = to_dev(X, w.dtype), to_dev(W, w.dtype), to_dev(dY, w.dtype)
    ws = P.alloc_workspace(N, Di, Do, k, w.dtype)
    Y, Xp = P.rmm_forward(Xd, Wd, None, w.seed, k, w.dist, workspace=ws)
    dX, dW, db = P.rmm_backward(dYd, Wd, Xp, w.seed, w.dist, workspace=ws)
    torch.cuda.synchronize()
    assert P.rmm_last_device_status(ws) == P.RMM_OK
    rng = np.random.default_rng(1)
    X64, W64, dY64 = X.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    c = float(np.float32(O.scale(k, w.dist)))
    tol = TOL[w.dtype]

    def close(got, want, what):
        got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
        err = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert err <= tol, (what, err)

    # Y and dX: sampled rows (full rows, so the Frobenius measure is over thousands of entries)
    rows = rng.choice(N, size=8, replace=False)
    close(to_np(Y[rows]), X64[rows] @ W64.T, "Y")
    close(to_np(dX[rows]), dY64[rows] @ W64, "dX")
    # db: all of it
    close(to_np(db), dY64.sum(axis=0), "db")
    # X_proj: sampled sketch columns j (rows of X_proj), each needs the whole column of S
    js = sorted(set([0, k - 1] + [int(j) for j in rng.choice(k, size=6, replace=False)]))
    for j in js:
        pj = O.generate_p(w.seed, N, k, w.dist, STORE[w.dtype], j, j + 1)[:, 0].astype(np.float64) * c
        close(to_np(Xp[j]), pj @ X64, f"X_proj[{j}]")
    # dW: sampled output rows o need G[:, o] = S^T dY[:, o], i.e. all of S once
    Pm = O.generate_p(w.seed, N, k, w.dist, STORE[w.dtype])          # [N, k] fp32
    os_ = rng.choice(Do, size=4, replace=False)
    G = (Pm.astype(np.float64).T @ dY64[:, os_]) * c                   # [k, 4]
    Xp64 = to_np(Xp)
    for t, o in enumerate(os_):
        close(to_np(dW[o]), G[:, t] @ Xp64, f"dW[{o}]")
    # properties that hold at any size: unbiasedness scale -- |dW| is of the order of |dY^T X|
    return True


@pytest.mark.parametrize("name", ["base_ffn_up_rho0.2", "base_ffn_down_rad_rho0.2", "base_qkv_rad_rho0.2",
                                  "large_ffn_up_rho0.1", "large_ffn_down_rho0.1", "large_ffn_up_k1663_aligned",
                                  "large_ffn_up_sors_rho0.1"])
def test_full_size_sampled(name):
    assert _sampled_full_size(name)


@pytest.mark.parametrize("name", ["base_ffn_up_rho0.1", "base_ffn_up_rho0.5", "base_ffn_up_rho0.9"])
def test_full_size_sampled_other_rho(name):
    assert _sampled_full_size(name)
