"""Host-side checks that need no GPU: the library loads, exports every symbol that
include/rmm.h declares, sizes its workspace sensibly and rejects bad arguments with the
documented codes before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LIB = os.path.join(ROOT, "paper_2201_13195_b200", "librmm.so")


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(LIB):
        import paper_2201_13195_b200.build as B
        B.build()
    return C.CDLL(LIB)


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rmm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rmm_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert {"rmm_forward", "rmm_backward", "rmm_workspace_bytes", "rmm_debug_generate_s",
            "rmm_last_device_status", "rmm_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_exports_match_header():
    import paper_2201_13195_b200 as P
    assert sorted(P.EXPORTS) == _declared_symbols()
    for n in P.EXPORTS:
        assert callable(getattr(P, n))


def test_status_strings(lib):
    lib.rmm_status_string.restype = C.c_char_p
    names = [lib.rmm_status_string(i).decode() for i in range(6)]
    assert names == ["RMM_OK", "RMM_ERR_INVALID_ARG", "RMM_ERR_UNSUPPORTED", "RMM_ERR_WORKSPACE", "RMM_ERR_CUDA",
                     "RMM_ERR_TIMEOUT"]


def test_workspace_bytes(lib):
    f = lib.rmm_workspace_bytes
    f.restype = C.c_size_t
    f.argtypes = [C.c_int64] * 4 + [C.c_int]
    big = f(16384, 1024, 4096, 1638, 0)
    assert big >= 1638 * 4096 * 2 and big % 256 == 0          # holds G = S^T dY in bf16
    assert f(16384, 1024, 4096, 1638, 1) >= 1638 * 4096 * 4
    assert f(0, 8, 8, 1, 0) == 0 and f(8, 8, 8, 9, 0) == 0 and f(8, 8, 8, 1, 7) == 0


def test_workspace_bytes_for_a_sketch(lib):
    """The suggested size is the smallest valid one except for the subsampled-Hadamard sketch in bf16 mode inside the fast
    path's range (Hadamard order 128 .. 16384), where it adds room for the transform's intermediate: L x D bf16 values."""
    base = lib.rmm_workspace_bytes
    base.restype = C.c_size_t
    base.argtypes = [C.c_int64] * 4 + [C.c_int]
    f = lib.rmm_workspace_bytes_for
    f.restype = C.c_size_t
    f.argtypes = [C.c_int64] * 4 + [C.c_int, C.c_int]
    shape = (16384, 1024, 4096, 1638)
    small = base(*shape, 0)
    for dist in (0, 1, 2, 4):
        assert f(*shape, 0, dist) == small
    roomy = f(*shape, 0, 3)
    assert roomy % 256 == 0 and roomy >= small and roomy >= 16384 * 4096 * 2       # T for all of dY's columns
    assert roomy < small + 16384 * 4096 * 2 + (16 << 20)
    assert f(*shape, 1, 3) == base(*shape, 1)                                      # fp32 mode: no fast path
    assert f(16500, 1024, 4096, 1638, 0, 3) == base(16500, 1024, 4096, 1638, 0)    # Hadamard order 32768: dense kernel
    assert f(100, 64, 64, 10, 0, 3) == base(100, 64, 64, 10, 0)                    # the smallest size already has room
    assert f(0, 8, 8, 1, 0, 3) == 0 and f(8, 8, 8, 9, 0, 3) == 0


def test_hadamard_fast_path_plan(lib):
    """Rounds of the fast transform: the intermediate T (L x columns, bf16) has to fit the scratch it is given."""
    f = lib.rmm_debug_hadamard_plan
    f.restype = C.c_int
    f.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_size_t, C.POINTER(C.c_int64)]
    info = (C.c_int64 * 4)()
    mib = 1 << 20
    assert f(1639, 4096, 16384, 160 * mib, info) == 1
    assert list(info) == [16384, 128, 4096, 1]                      # all of dY's columns at once
    assert f(1639, 4096, 16384, 70 * mib, info) == 1
    assert info[3] == 2 and info[2] == 2048 and info[2] % 64 == 0   # two equal rounds rather than a full and a narrow one
    assert f(1639, 4096, 16384, 40 * mib, info) == 1 and info[3] == 4 and info[2] == 1024
    assert f(77, 520, 389, 8 * mib, info) == 1 and list(info) == [512, 4, 576, 1]     # ragged width: whole 64-column slabs
    assert f(128, 72, 128, 8 * mib, info) == 1 and info[0] == 128 and info[1] == 1
    assert f(5, 40, 37, 8 * mib, info) == 0                         # Hadamard order 64: dense kernel
    assert f(141, 1024, 16500, 512 * mib, info) == 0                # order 32768: dense kernel
    assert f(1639, 4096, 16384, 1 * mib, info) == 0                 # not even one slab of T fits
    assert f(0, 8, 8, mib, info) == -1 and f(8, 8, 8, mib, None) == -1


def test_argument_errors_are_reported_before_any_launch(lib):
    i64, vp = C.c_int64, C.c_void_p
    fwd = lib.rmm_forward
    fwd.argtypes = [vp, vp, vp, i64, i64, i64, C.c_uint64, i64, C.c_int, C.c_int, vp, vp, vp, C.c_size_t, vp]
    bwd = lib.rmm_backward
    bwd.argtypes = [vp, vp, vp, i64, i64, i64, C.c_uint64, i64, C.c_int, C.c_int, vp, vp, vp, vp, C.c_size_t, vp]
    p = 4096  # a non-null, 16-byte aligned fake pointer: must never be dereferenced on the host
    INVALID, UNSUPPORTED, WORKSPACE = 1, 2, 3
    assert fwd(None, p, None, 8, 8, 8, 0, 4, 0, 0, p, p, p, 1 << 20, None) == INVALID       # null X
    assert fwd(p, p, None, 8, 8, 8, 0, 9, 0, 0, p, p, p, 1 << 20, None) == INVALID          # B_proj > N
    assert fwd(p, p, None, 8, 8, 8, 0, 0, 0, 0, p, p, p, 1 << 20, None) == INVALID          # B_proj < 1
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 5, 0, p, p, p, 1 << 20, None) == INVALID          # bad dist
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 3, 0, p, p, None, 0, None) == WORKSPACE           # dist 3 is valid: next check
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 0, 3, p, p, p, 1 << 20, None) == INVALID          # bad dtype
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 2, 0, p, p, p, 1 << 20, None) == INVALID          # identity needs k == N
    assert fwd(p + 4, p, None, 8, 8, 8, 0, 4, 0, 0, p, p, p, 1 << 20, None) == INVALID      # misaligned X
    assert fwd(p, p, None, 8, 12, 8, 0, 4, 0, 0, p, p, p, 1 << 20, None) == UNSUPPORTED     # D_in % 8 in bf16
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 0, 0, p, p, None, 0, None) == WORKSPACE           # no workspace
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 0, 0, p, p, p, 16, None) == WORKSPACE             # too small
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 0, 0, p, p, p + 16, 1 << 20, None) == WORKSPACE   # misaligned workspace
    assert bwd(p, p, p, 8, 8, 8, 0, 4, 0, 0, p, None, p, p, 1 << 20, None) == INVALID       # dW is required
    assert bwd(p, p, p, 8, 8, 8, 0, 4, 0, 0, p, p, p, None, 0, None) == WORKSPACE
    gen = lib.rmm_debug_generate_s
    gen.argtypes = [C.c_uint64, i64, i64, C.c_int, C.c_int, vp, vp]
    assert gen(0, 8, 9, 0, 0, p, None) == INVALID
    assert gen(0, 8, 4, 0, 0, None, None) == INVALID


def test_no_device_is_an_error_not_a_fallback(lib):
    """Without a usable sm_100a device a well-formed call must fail with RMM_ERR_CUDA."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    i64, vp = C.c_int64, C.c_void_p
    fwd = lib.rmm_forward
    fwd.argtypes = [vp, vp, vp, i64, i64, i64, C.c_uint64, i64, C.c_int, C.c_int, vp, vp, vp, C.c_size_t, vp]
    p = 4096
    assert fwd(p, p, None, 8, 8, 8, 0, 4, 0, 0, p, p, p, 1 << 40, None) == 4


@pytest.mark.parametrize("rows,cols,tokens,ctas", [
    (1639, 4096, 16384, 148), (1638, 1024, 16384, 148), (820, 3072, 4096, 148), (819, 768, 4096, 148),
    (3687, 3072, 4096, 148), (5, 24, 37, 148), (131, 520, 300, 148), (1, 8, 1, 148), (2049, 768, 4096, 148),
    (1153, 4096, 4096, 74), (1639, 4096, 16384, 7), (300, 1500, 1000, 3), (129, 513, 65, 74),
    (7000, 3072, 4096, 74), (40000, 3072, 4096, 148),
])
def test_sketch_schedule_covers_every_unit_once(rows, cols, tokens, ctas):
    """Host logic of the sketch kernels' stream-K schedule: every (tile, token step) unit belongs to
    exactly one segment, no two segments share a partial-tile slot, and the reduction's slot list
    per tile is exactly the set of slots that the kernel writes for that tile."""
    import collections

    import paper_2201_13195_b200 as P
    segs, info = P.rmm_debug_sketch_schedule(rows, cols, tokens, ctas, mode=0)
    red, info2 = P.rmm_debug_sketch_schedule(rows, cols, tokens, ctas, mode=1)
    assert info == info2
    tiles, ksteps = info["tiles"], info["ksteps"]
    blocks = -(-cols // 512)
    c = 2 if blocks >= 2 else 1               # an odd block count leaves the last cluster's second CTA without columns
    assert info["cluster"] == c
    assert tiles == -(-rows // 128) * -(-blocks // c) and ksteps == -(-tokens // 64)
    ctas = max(1, ctas // c)
    assert info["num_ctas"] <= ctas
    cover = collections.Counter()
    slots = set()
    by_tile = collections.defaultdict(list)
    per_cta = collections.Counter()
    for cta, tile, ks0, ks1, slot in segs:
        assert 0 <= cta < info["num_ctas"] and 0 <= tile < tiles and 0 <= ks0 < ks1 <= ksteps
        assert 0 <= slot < info["num_slots"] and slot not in slots
        slots.add(slot)
        by_tile[tile].append(slot)
        per_cta[cta] += ks1 - ks0
        for ks in range(ks0, ks1):
            cover[(tile, ks)] += 1
    assert len(cover) == tiles * ksteps and set(cover.values()) == {1}
    red_by_tile = collections.defaultdict(list)
    for tile, slot, *_ in red:
        red_by_tile[tile].append(slot)
    assert {t: sorted(v) for t, v in by_tile.items()} == {t: sorted(v) for t, v in red_by_tile.items()}
    # balance: no CTA carries much more than the mean
    mean = tiles * ksteps / info["num_ctas"]
    assert max(per_cta.values()) <= 1.5 * mean + (ksteps if tiles >= ctas else 8) + 1
    # no CTA is left with a long tail of tiny segments
    nseg = collections.Counter(c for c, _, ks0, ks1, _ in segs if ks1 - ks0 < ksteps)
    assert not nseg or max(nseg.values()) <= 6


def test_rmm_linear_bproj_rule_matches_harness_rule():
    """The module's B_proj = round(rho * tokens) is the rule the workloads use."""
    import rmm_inputs as R
    from paper_2201_13195_b200.rmm_linear import bproj_from_rho
    for n, rho in ((4096, 0.1), (4096, 0.2), (4096, 0.5), (4096, 0.9), (16384, 0.1), (512, 0.5), (7, 0.01), (3, 1.0)):
        assert bproj_from_rho(n, rho) == R.bproj_from_rho(n, rho) >= 1


def test_variance_probe_argument_errors(lib):
    i64, vp = C.c_int64, C.c_void_p
    probe = lib.rmm_variance_probe
    probe.argtypes = [vp, vp, i64, i64, i64, i64, C.c_int, C.c_int, vp, vp, vp, C.c_size_t, vp]
    size = lib.rmm_variance_probe_workspace_bytes
    size.argtypes = [i64, i64, i64]
    size.restype = C.c_size_t
    assert size(1, 8, 8) == 0 and size(16, 0, 8) == 0
    need = size(4096, 768, 3072)
    assert need >= 3072 * 768 * 2          # room for the exact gradient when the caller does not want it
    p = 4096
    INVALID, UNSUPPORTED, WORKSPACE, CUDA = 1, 2, 3, 4
    assert probe(p, p, 1, 8, 8, 1, 0, 0, p, None, p, 1 << 30, None) == INVALID         # N < 2: Eq. 9 divides by N - 1
    assert probe(None, p, 16, 8, 8, 4, 0, 0, p, None, p, 1 << 30, None) == INVALID     # null X
    assert probe(p, p, 16, 8, 8, 4, 0, 0, None, None, p, 1 << 30, None) == INVALID     # null out
    assert probe(p, p, 16, 8, 8, 17, 0, 0, p, None, p, 1 << 30, None) == INVALID       # B_proj > N
    assert probe(p, p, 16, 8, 8, 4, 0, 1, p, None, p, 1 << 30, None) == UNSUPPORTED    # fp32 tensors
    assert probe(p, p, 16, 8, 8, 4, 3, 0, p, None, p, 1 << 30, None) == UNSUPPORTED    # no closed form for the Hadamard sketch
    assert probe(p, p, 16, 12, 8, 4, 0, 0, p, None, p, 1 << 30, None) == UNSUPPORTED   # D_in % 8
    assert probe(p, p, 16, 8, 8, 4, 0, 0, p, None, p, 64, None) == WORKSPACE           # too small
    assert probe(p, p, 16, 8, 8, 4, 0, 0, p, None, None, 0, None) == WORKSPACE
    import torch
    if not torch.cuda.is_available():
        assert probe(p, p, 16, 8, 8, 4, 0, 0, p, None, p, 1 << 30, None) == CUDA        # no device: an error, no fallback


@pytest.mark.parametrize("N,d_in,d_out,k,pairs", [
    (16384, 1024, 4096, 1638, 74), (16384, 4096, 1024, 1638, 74), (4096, 768, 3072, 819, 74), (4096, 768, 3072, 3686, 74),
    (4096, 3072, 768, 819, 74), (4096, 768, 2304, 819, 74), (4096, 768, 768, 819, 74), (37, 24, 40, 5, 74),
    (1, 8, 8, 1, 74), (300, 264, 520, 130, 74), (9700, 512, 64, 16, 74), (19200, 1024, 64, 16, 74),
    (2900, 4096, 64, 2816, 74), (16384, 1024, 4096, 1638, 5), (4096, 768, 3072, 819, 1), (100000, 64, 64, 16, 74),
])
def test_pass_schedule_covers_all_work_and_fits_the_workspace(N, d_in, d_out, k, pairs):
    """Host logic of the one-launch passes: every dense tile belongs to exactly one pair, the token blocks of a
    sketch tile cover its steps exactly once, no pair index is out of range, and the partial tiles fit the
    scratch part of the workspace that rmm_workspace_bytes asks for."""
    import paper_2201_13195_b200 as P
    ws = P.rmm_workspace_bytes(N, d_in, d_out, k, P.RMM_DTYPE_BF16)
    for gemm, sketch in (((N, d_out, d_in), (k, d_in, N)), ((N, d_in, d_out), (k + 1, d_out, N)),
                         (None, (k, d_in, N)), ((N, d_out, d_in), None)):
        s = P.rmm_debug_pass_schedule(gemm, sketch, pairs)
        assert 1 <= s["num_pairs"] <= pairs
        gb = s["gemm_begin"]
        assert gb[0] == 0 and gb[-1] == s["gemm_tiles"] and all(a <= b for a, b in zip(gb, gb[1:]))
        if gemm:
            assert s["gemm_tiles"] == -(-gemm[0] // 256) * -(-gemm[1] // 256) and s["num_kb"] == -(-gemm[2] // 64)
        else:
            assert s["gemm_tiles"] == 0
        if sketch:
            rows, cols, tokens = sketch
            assert s["tiles_m"] == -(-rows // 128) and s["ksteps"] == -(-tokens // 64)
            assert 1 <= s["nat"] <= 4 and s["groups"] * s["nat"] * 256 >= cols > (s["groups"] - 1) * s["nat"] * 256
            assert (s["nb"] - 1) * s["blen"] < s["ksteps"] <= s["nb"] * s["blen"]      # blocks: non-empty, cover all steps
            units = s["tiles_m"] * s["groups"] * s["nb"]
            assert units * 128 * s["nat"] * 256 * 4 <= ws                             # partial tiles fit the workspace
            assert s["num_pairs"] == min(pairs, units + s["gemm_tiles"])
        else:
            assert s["tiles_m"] == 0
