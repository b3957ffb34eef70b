"""Run forward+backward of one RMM layer of a given shape a few times on cuda:0.

    python -m paper_2201_13195_b200.run_case --n 4096 --d-in 1024 --d-out 4096 --k 1152 --dist gaussian --reps 3

A small driver for profilers and quick timing: random bf16 (or fp32) inputs, one workspace,
`reps` forward+backward pairs on the current stream, prints the mean time per pair.
"""
import argparse

import torch

from . import binding as P


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--d-in", type=int, default=1024)
    ap.add_argument("--d-out", type=int, default=4096)
    ap.add_argument("--k", type=int, default=410)
    ap.add_argument("--dist", default="gaussian", choices=["gaussian", "rademacher", "sors"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--forward-only", action="store_true")
    ap.add_argument("--variance-probe", action="store_true", help="run rmm_variance_probe instead of the layer")
    a = ap.parse_args()
    td = torch.bfloat16 if a.dtype == "bf16" else torch.float32
    dist = {"gaussian": P.RMM_DIST_GAUSSIAN, "rademacher": P.RMM_DIST_RADEMACHER, "sors": P.RMM_DIST_SORS_HADAMARD}[a.dist]
    g = torch.Generator(device="cuda").manual_seed(0)
    X = torch.randn(a.n, a.d_in, device="cuda", generator=g).to(td)
    W = (0.02 * torch.randn(a.d_out, a.d_in, device="cuda", generator=g)).to(td)
    dY = (0.01 * torch.randn(a.n, a.d_out, device="cuda", generator=g)).to(td)
    ws = P.alloc_workspace(a.n, a.d_in, a.d_out, a.k, P.RMM_DTYPE_BF16 if a.dtype == "bf16" else P.RMM_DTYPE_F32)
    Y = torch.empty(a.n, a.d_out, device="cuda", dtype=td)
    Xp = torch.empty(a.k, a.d_in, device="cuda", dtype=td)
    dX = torch.empty(a.n, a.d_in, device="cuda", dtype=td)
    dW = torch.empty(a.d_out, a.d_in, device="cuda", dtype=td)
    db = torch.empty(a.d_out, device="cuda", dtype=td)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if a.variance_probe:
        pws = torch.empty(P.rmm_variance_probe_workspace_bytes(a.n, a.d_in, a.d_out), dtype=torch.uint8, device="cuda")
        out = torch.empty(8, dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        e0.record()
        for i in range(a.reps):
            P.rmm_variance_probe(X, dY, a.k, dist, out=out, workspace=pws)
        e1.record()
        torch.cuda.synchronize()
        assert P.rmm_last_device_status(pws) == P.RMM_OK
        print(f"{e0.elapsed_time(e1) / a.reps:.4f} ms per probe;", dict(zip(P.VARIANCE_FIELDS, out.cpu().tolist())))
        return
    torch.cuda.synchronize()
    e0.record()
    for i in range(a.reps):
        P.rmm_forward(X, W, None, i, a.k, dist, Y=Y, X_proj=Xp, workspace=ws)
        if not a.forward_only:
            P.rmm_backward(dY, W, Xp, i, dist, dX=dX, dW=dW, db=db, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    assert P.rmm_last_device_status(ws) == P.RMM_OK
    print(f"{e0.elapsed_time(e1) / a.reps:.4f} ms per {'forward' if a.forward_only else 'forward+backward'}")


if __name__ == "__main__":
    main()
