"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs.  S bit-exact; Y, X_proj, dX, dW, db within a relative Frobenius error
of 1e-2 (bf16 mode) or 1e-5 (fp32 mode)."""
import numpy as np
import pytest
import torch

import rmm_inputs as R
from oracle import oracle as O

pytestmark = pytest.mark.gpu

from tests.gpu_util import (SORS_FAST_PATH_EXTRA, STORE, TOL, TORCH_DTYPE, assert_parity, contraction_lengths, dw_operand_term,  # noqa: E402
                            elementwise_excess, oracle_layer, run_layer, to_dev, to_np)


def _P():
    import paper_2201_13195_b200 as P
    return P


# ------------------------------------------------------------------ S bit-exact
@pytest.mark.parametrize("dtype", [R.DTYPE_BF16, R.DTYPE_F32])
@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER, R.DIST_SORS, R.DIST_DCT])
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
@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER, R.DIST_SORS, R.DIST_DCT])
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


def _selector(N, tokens, dtype):
    """X [N, len(tokens)] with X[tokens[i]][i] = 1 and zeros elsewhere: X_proj[j][i] = c * P[tokens[i]][j] exactly
    (one non-zero product per sum), so the production sketch kernel's own S can be compared bit for bit at the
    chosen tokens without an N x N identity."""
    X = torch.zeros((N, len(tokens)), dtype=TORCH_DTYPE[dtype], device="cuda")
    X[torch.as_tensor(tokens, device="cuda"), torch.arange(len(tokens), device="cuda")] = 1.0
    return X


WIDE_S_CASES = [
    # name, N, number of selected tokens (= D_in), k, seed
    ("two_blocks_identity", 1024, 1024, 141, 78),        # X = I with two 512-column blocks: S stages shared by a CTA pair
    ("four_blocks_many_steps", 4096, 2048, 300, 79),     # several column groups, 64 token steps, three row tiles
    ("odd_blocks", 2000, 1536, 260, 80),                 # three 512-column blocks, ragged last token step
    ("above_hadamard_fast_path", 16500, 1024, 141, 81),  # Hadamard order 32768: the dense kernel also for SORS
]


@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER, R.DIST_SORS, R.DIST_DCT])
@pytest.mark.parametrize("case", WIDE_S_CASES, ids=[c[0] for c in WIDE_S_CASES])
def test_production_kernel_sketch_bit_exact_wide(case, dist):
    """S entry by entry on the launch shapes of the RoBERTa layers: results wider than one 512-column block
    (stages of S^T exchanged inside a CTA pair or cluster), many token steps per tile, several row tiles."""
    P = _P()
    _, N, D, k, seed = case
    rng = np.random.default_rng(seed)
    if D == N:
        tokens = np.arange(N)
    else:   # first and last tokens, the edges of the 64-token steps, and random ones
        edges = np.concatenate([np.arange(0, N, 64), np.arange(63, N, 64), [N - 1]])
        rest = np.setdiff1d(np.arange(N), edges)
        tokens = np.sort(np.concatenate([edges[:D // 2], rng.choice(rest, size=D - len(edges[:D // 2]), replace=False)]))
    X = _selector(N, tokens, R.DTYPE_BF16)
    W = torch.zeros((8, D), dtype=torch.bfloat16, device="cuda")
    _, Xp = P.rmm_forward(X, W, None, seed, k, dist, want_y=False)
    torch.cuda.synchronize()
    Pm = O.generate_p(seed, N, k, dist, O.STORE_BF16)[tokens]          # [D, k] fp32
    want = R.round_to_bf16((Pm.T * np.float32(O.scale(k, dist))).astype(np.float32))
    got = Xp.to(torch.float32).cpu().numpy()
    assert got.shape == want.shape
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{len(bad)} entries differ, first at sketch row {bad[0][0]}, token {tokens[bad[0][1]]}"


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
    ("dct_ragged_bf16", R.DTYPE_BF16, 389, 264, 520, 77, R.DIST_DCT),
    ("dct_ragged_f32", R.DTYPE_F32, 150, 70, 130, 66, R.DIST_DCT),
    ("dct_widths_768_2304", R.DTYPE_BF16, 320, 768, 2304, 140, R.DIST_DCT),
    ("sors_below_fast_path", R.DTYPE_BF16, 37, 24, 40, 5, R.DIST_SORS),          # Hadamard order 64: dense kernel
    ("sors_one_block", R.DTYPE_BF16, 128, 64, 72, 128, R.DIST_SORS),             # order 128: one block, no second level
    ("sors_many_blocks", R.DTYPE_BF16, 2100, 136, 200, 300, R.DIST_SORS),        # order 4096: 32 blocks, last ones empty
    ("sors_wide", R.DTYPE_BF16, 300, 2200, 2312, 40, R.DIST_SORS),                # 35 and 37 column slabs of 64, the last one ragged
    # dX has 38 x 2 = 76 tiles of 256 x 256: more than the 74 CTA pairs, so two pairs take a second tile
    # (both accumulator buffers in use), with ragged last rows: 9700 = 37 * 256 + 228
    ("dx_second_wave", R.DTYPE_BF16, 9700, 512, 64, 16, R.DIST_RADEMACHER),
    # the RoBERTa-base widths: 768 = one and a half 512-column blocks (the cluster's fourth 256-column half is empty),
    # 2304 = four and a half (odd block count: the last cluster's second CTA only generates its half of S^T)
    ("widths_768_2304", R.DTYPE_BF16, 320, 768, 2304, 140, R.DIST_GAUSSIAN),
    # a ragged last 256-column half: 1160 = 4 * 256 + 136
    ("ragged_column_half", R.DTYPE_BF16, 200, 1160, 648, 90, R.DIST_RADEMACHER),
]


def _check_layer(w, N, Di, Do, k, dist, dtype, got):
    K = contraction_lengths(N, Di, Do, k)
    ref = oracle_layer(w, got["inputs"], gpu_xproj=got["X_proj"])
    assert_parity(got, ref, dtype, K=K, dist=dist)
    # end to end (oracle's own fp64 X_proj in backward)
    ref2 = oracle_layer(w, got["inputs"])
    assert_parity(got, ref2, dtype, names=("dW",), K=K, end_to_end=True, dist=dist)


@pytest.fixture
def pass_mode():
    """Sets how the library runs a bf16 pass for one test and puts the default back afterwards."""
    P = _P()
    yield P.rmm_set_pass_mode
    P.rmm_set_pass_mode(0)


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_layer_parity_small(case):
    name, dtype, N, Di, Do, k, dist = case
    w = R.small_case(name, dtype, N, Di, Do, k, dist, seed=len(name) * 1000003)
    _check_layer(w, N, Di, Do, k, dist, dtype, run_layer(w))


# Shapes chosen for the launch paths they reach, small enough for a full-tensor fp64 comparison.
PATH_CASES = [
    # dX is 75 x 4 = 300 tiles of 256 x 256 with a single K block: four and more tiles per CTA pair, both
    # accumulator buffers reused twice; Y has 75 tiles
    ("gemm_many_tiles_per_pair", 19200, 1024, 64, 16, R.DIST_RADEMACHER),
    # forward sketch: 22 row tiles x 4 column groups = 88 tile groups on 74 clusters: a round of whole tiles, then
    # the remaining tiles cut into token blocks
    ("sketch_whole_tile_round_and_remainder", 2900, 4096, 64, 2816, R.DIST_GAUSSIAN),
    # backward sketch: 10 row tiles (1153 rows with the row of ones) x 4 column groups = 40 tile groups on 74
    # clusters: one full block per tile and a last, narrower block shared tile after tile by the other clusters
    ("sketch_last_block_line", 4096, 64, 4096, 1152, R.DIST_RADEMACHER),
]


@pytest.mark.parametrize("case", PATH_CASES, ids=[c[0] for c in PATH_CASES])
def test_layer_parity_launch_paths(case, pass_mode):
    """Every element of every output against the oracle on shapes that reach the remaining branches of the static
    schedules, with the two kernels of a pass side by side (default) and one after the other on the whole device
    (the grid the schedule branches below are stated for)."""
    P = _P()
    name, N, Di, Do, k, dist = case
    w = R.small_case(name, R.DTYPE_BF16, N, Di, Do, k, dist, seed=len(name) * 7919)
    if name == "sketch_whole_tile_round_and_remainder":
        _, info = P.rmm_debug_sketch_schedule(k, Di, N, 148)
        assert info["rounds"] >= 1 and info["tiles"] % info["num_ctas"] != 0
    if name == "sketch_last_block_line":
        _, info = P.rmm_debug_sketch_schedule(k + 1, Do, N, 148)
        assert info["rounds"] == 0 and info["w_last"] > 0
    if name == "gemm_many_tiles_per_pair":
        assert -(-N // 256) * -(-Di // 256) >= 4 * 74
    inputs = R.make_inputs(w)
    X, W, b, dY = [None if a is None else a.astype(np.float64) for a in inputs]
    S = O.generate_s(w.seed, N, k, dist, O.STORE_BF16)
    Y, Xp = O.forward(X, W, b, S)
    K = contraction_lengths(N, Di, Do, k)
    for mode in (0, 2):
        pass_mode(mode)
        got = run_layer(w, inputs=inputs)
        dX, dW, db, G = O.backward(dY, W, got["X_proj"], S)      # stage-wise: the GPU's own X_proj
        ref = {"Y": Y, "X_proj": Xp, "dX": dX, "dW": dW, "db": db, "G": G, "X_proj_used": got["X_proj"]}
        assert_parity(got, ref, R.DTYPE_BF16, K=K, dist=dist)


ONE_LAUNCH_CASES = [c for c in CASES if c[1] == R.DTYPE_BF16 and c[0] in (
    "tiny_ragged_bf16", "one_row", "multi_tile_ragged_bf16", "multi_tile_ragged_rad", "rho_one_gauss",
    "k_multiple_of_tile", "sors_below_fast_path", "dx_second_wave", "dct_ragged_bf16")]


@pytest.mark.parametrize("case", ONE_LAUNCH_CASES, ids=[c[0] for c in ONE_LAUNCH_CASES])
def test_layer_parity_one_launch_per_pass(case, pass_mode):
    """The alternative execution of a pass as a single launch (sketch units and dense tiles of one static schedule,
    in-kernel reduction of the partial tiles): same gates as the default path."""
    name, dtype, N, Di, Do, k, dist = case
    pass_mode(1)
    w = R.small_case(name, dtype, N, Di, Do, k, dist, seed=len(name) * 1000003)
    _check_layer(w, N, Di, Do, k, dist, dtype, run_layer(w))


@pytest.mark.parametrize("dist", [R.DIST_GAUSSIAN, R.DIST_RADEMACHER, R.DIST_SORS, R.DIST_DCT])
def test_one_launch_pass_sketch_bit_exact(dist, pass_mode):
    """S entry by entry through the one-launch pass kernel (X = selector matrix), several token blocks per tile."""
    P = _P()
    pass_mode(1)
    N, D, k, seed = 16500, 1024, 141, 91
    rng = np.random.default_rng(seed)
    tokens = np.sort(rng.choice(N, size=D, replace=False))
    X = _selector(N, tokens, R.DTYPE_BF16)
    W = torch.zeros((8, D), dtype=torch.bfloat16, device="cuda")
    _, Xp = P.rmm_forward(X, W, None, seed, k, dist, want_y=False)
    torch.cuda.synchronize()
    Pm = O.generate_p(seed, N, k, dist, O.STORE_BF16)[tokens]
    want = R.round_to_bf16((Pm.T * np.float32(O.scale(k, dist))).astype(np.float32))
    assert np.array_equal(Xp.to(torch.float32).cpu().numpy(), want)


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
    errs = assert_parity(got, ref, w.dtype, K=contraction_lengths(w.n_tokens, w.d_in, w.d_out, w.b_proj))
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
    assert_parity(got, ref, w.dtype, K=contraction_lengths(N, w.d_in, w.d_out, k))


# ------------------------------------------------------------------ full-size workloads, sampled outputs
def _sampled_full_size(name, roomy=False):
    """The launch configuration the benchmark times, checked on outputs the oracle computes one by one: one row
    of Y and of dX in every 128-row block (every row block of every output tile), one row of X_proj in every
    128-row sketch tile plus the first and last, one row of dW in every 128-row block, all of db; all columns of
    each sampled row, so every column block of every tile is covered.  Expected values come from oracle.forward /
    oracle.backward on the row subsets; each sampled row passes the Frobenius gate and every sampled element the
    element-wise one."""
    P = _P()
    w = R.WORKLOADS[name]
    X, W, b, dY = R.make_inputs(w)
    N, k, Di, Do = w.n_tokens, w.b_proj, w.d_in, w.d_out
    Xd, Wd, dYd = to_dev(X, w.dtype), to_dev(W, w.dtype), to_dev(dY, w.dtype)
    # roomy: the workspace size the library suggests for this sketch (what the benchmark allocates) instead of the smallest
    ws = P.alloc_workspace(N, Di, Do, k, w.dtype, dist=w.dist if roomy else None)
    Y, Xp = P.rmm_forward(Xd, Wd, None, w.seed, k, w.dist, workspace=ws)
    dX, dW, db = P.rmm_backward(dYd, Wd, Xp, w.seed, w.dist, workspace=ws)
    torch.cuda.synchronize()
    assert P.rmm_last_device_status(ws) == P.RMM_OK
    rng = np.random.default_rng(1)
    X64, W64, dY64 = X.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    K = contraction_lengths(N, Di, Do, k)
    tol = TOL[w.dtype]

    def close(got, want, what, Klen, term=None):
        got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
        err = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert err <= tol, (what, err)
        for r in range(got.shape[0]):                      # every sampled row on its own as well
            e = np.linalg.norm(got[r] - want[r]) / np.linalg.norm(want[r])
            assert e <= tol, (what, r, e)
        extra = SORS_FAST_PATH_EXTRA if (w.dist == R.DIST_SORS and what in ("X_proj", "dW")) else 0.0
        ex, where = elementwise_excess(got, want, w.dtype, Klen, term, extra)
        assert ex <= 1.0, (what, where, ex)

    def one_per_block(total, block):
        starts = np.arange(0, total, block)
        return np.minimum(starts + rng.integers(0, block, size=len(starts)), total - 1)

    # Y and dX: one row in every 128-row block
    rows = one_per_block(N, 128)
    nothing = np.zeros((len(rows), 1))
    Yref, _ = O.forward(X64[rows], W64, None, nothing, want_xproj=False)
    close(to_np(Y[rows]), Yref, "Y", K["Y"])
    dXref, _, _, _ = O.backward(dY64[rows], W64, np.zeros((1, Di)), nothing, want_dw=False, want_db=False)
    close(to_np(dX[rows]), dXref, "dX", K["dX"])
    # db: all of it
    _, _, dbref, _ = O.backward(dY64, W64[:, :1], np.zeros((1, 1)), np.zeros((N, 1)), want_dx=False, want_dw=False)
    close(to_np(db)[None, :], dbref[None, :], "db", K["db"])
    # S once (fp64, scaled): X_proj rows need columns of it, dW rows need all of it
    S = O.generate_s(w.seed, N, k, w.dist, STORE[w.dtype])
    js = np.unique(np.concatenate([[0, k - 1], one_per_block(k, 128)]))
    _, Xpref = O.forward(X64, W64[:1], None, np.ascontiguousarray(S[:, js]), want_y=False)
    close(to_np(Xp[js]), Xpref, "X_proj", K["X_proj"])
    # dW: one row in every 128-row block of D_out; stage-wise (the GPU's own X_proj, as rmm_backward receives it)
    os_ = one_per_block(Do, 128)
    Xp64 = to_np(Xp)
    _, dWref, _, G = O.backward(np.ascontiguousarray(dY64[:, os_]), W64[os_], Xp64, S, want_dx=False, want_db=False)
    close(to_np(dW[os_]), dWref, "dW", K["dW"], dw_operand_term(G, Xp64, w.dtype))
    return True


@pytest.mark.parametrize("name", ["base_ffn_up_rho0.2", "base_ffn_down_rad_rho0.2", "base_qkv_rad_rho0.2",
                                  "large_ffn_up_rho0.1", "large_ffn_down_rho0.1", "large_ffn_up_k1663_aligned",
                                  "large_ffn_up_sors_rho0.1", "large_ffn_up_dct_rho0.1"])
def test_full_size_sampled(name):
    assert _sampled_full_size(name)


def test_full_size_sampled_suggested_workspace():
    """The subsampled-Hadamard fast path with the workspace of rmm_workspace_bytes_for: all of dY's columns in one round
    (with the smallest workspace, above, it takes them in two)."""
    P = _P()
    w = R.WORKLOADS["large_ffn_up_sors_rho0.1"]
    small = P.rmm_workspace_bytes(w.n_tokens, w.d_in, w.d_out, w.b_proj, w.dtype)
    roomy = P.rmm_workspace_bytes_for(w.n_tokens, w.d_in, w.d_out, w.b_proj, w.dtype, w.dist)
    assert roomy > small
    assert P.rmm_workspace_bytes_for(w.n_tokens, w.d_in, w.d_out, w.b_proj, w.dtype, R.DIST_GAUSSIAN) == small
    assert _sampled_full_size("large_ffn_up_sors_rho0.1", roomy=True)


@pytest.mark.parametrize("name", ["base_ffn_up_rho0.1", "base_ffn_up_rho0.5", "base_ffn_up_rho0.9"])
def test_full_size_sampled_other_rho(name):
    assert _sampled_full_size(name)


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("name", ["base_qkv_rad_rho0.2", "large_ffn_up_rho0.1"])
def test_full_size_sampled_other_pass_modes(name, mode, pass_mode):
    pass_mode(mode)
    assert _sampled_full_size(name)
