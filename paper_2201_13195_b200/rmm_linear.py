"""torch.autograd wrapper of the RMM linear layer (Algorithm 1) over the C-ABI binding.

Forward computes Y = X W^T + b and X_proj = S^T X with one `rmm_forward` call and keeps only
X_proj, the weight and the 64-bit seed for the backward pass (B_proj * D_in elements instead
of N * D_in, Section 2.4.1); backward is one `rmm_backward` call that regenerates S from the
seed.  Nothing is computed here: the module reshapes, picks B_proj and the seed, and hands
device pointers to the library.  There is no fallback: CPU tensors raise.
"""
import math

import torch

from . import binding as P

_DIST = {"gaussian": P.RMM_DIST_GAUSSIAN, "rademacher": P.RMM_DIST_RADEMACHER, "identity": P.RMM_DIST_IDENTITY,
         "sors": P.RMM_DIST_SORS_HADAMARD, "dct": P.RMM_DIST_SORS_DCT}


def bproj_from_rho(n_tokens: int, rho: float) -> int:
    """B_proj = rho * B (Section 2.4) rounded to the nearest integer, at least 1, at most the token count."""
    return min(n_tokens, max(1, int(math.floor(rho * n_tokens + 0.5))))


class Workspace:
    """One growing device buffer shared by all layers that run on the same stream (the library's
    workspace holds only transients of a single call: G = S^T dY and partial tiles)."""

    def __init__(self):
        self.buf = None

    def get(self, N, D_in, D_out, B_proj, dt, device, dist=None):
        need = P.rmm_workspace_bytes(N, D_in, D_out, B_proj, dt) if dist is None else \
            P.rmm_workspace_bytes_for(N, D_in, D_out, B_proj, dt, dist)
        if self.buf is None or self.buf.numel() < need or self.buf.device != device:
            self.buf = torch.empty(need, dtype=torch.uint8, device=device)
        return self.buf


class RMMLinearFunction(torch.autograd.Function):
    """y = rmm_linear(x, weight, bias); saves (X_proj, weight, seed), not x."""

    @staticmethod
    def forward(ctx, x, weight, bias, seed, b_proj, dist, workspace, trace):
        if not x.is_cuda:
            raise RuntimeError("RMMLinear runs only on a CUDA device (there is no CPU path)")
        d_in = weight.shape[1]
        x2 = x.reshape(-1, d_in)
        if not x2.is_contiguous():
            x2 = x2.contiguous()
        n = x2.shape[0]
        dt = P.RMM_DTYPE_BF16 if x.dtype == torch.bfloat16 else P.RMM_DTYPE_F32
        ws = workspace.get(n, d_in, weight.shape[0], b_proj, dt, x.device, dist)
        y, x_proj = P.rmm_forward(x2, weight, bias, seed, b_proj, dist, workspace=ws)
        ctx.save_for_backward(weight, x_proj)
        ctx.rmm = (seed, dist, x.shape, bias is not None, workspace, trace)
        if trace is not None:
            trace.append({"X": x2.detach().clone(), "W": weight.detach().clone(),
                          "b": None if bias is None else bias.detach().clone(), "seed": seed, "b_proj": b_proj,
                          "dist": dist, "Y": y.detach().clone(), "X_proj": x_proj.detach().clone()})
            ctx.rmm_trace_index = len(trace) - 1
        return y.view(*x.shape[:-1], weight.shape[0])

    @staticmethod
    def backward(ctx, dy):
        weight, x_proj = ctx.saved_tensors
        seed, dist, x_shape, has_bias, workspace, trace = ctx.rmm
        d_out, d_in = weight.shape
        dy2 = dy.reshape(-1, d_out)
        if not dy2.is_contiguous():
            dy2 = dy2.contiguous()
        n = dy2.shape[0]
        dt = P.RMM_DTYPE_BF16 if dy.dtype == torch.bfloat16 else P.RMM_DTYPE_F32
        ws = workspace.get(n, d_in, d_out, x_proj.shape[0], dt, dy.device, dist)
        want_dx = ctx.needs_input_grad[0]
        dx, dw, db = P.rmm_backward(dy2, weight, x_proj, seed, dist, workspace=ws, want_dx=want_dx, want_db=has_bias)
        if trace is not None:
            trace[ctx.rmm_trace_index].update({"dY": dy2.detach().clone(), "dX": None if dx is None else dx.clone(),
                                               "dW": dw.clone(), "db": None if db is None else db.clone()})
        return (dx.view(x_shape) if want_dx else None, dw, db if has_bias else None, None, None, None, None, None)


class RMMLinear(torch.nn.Module):
    """Drop-in replacement of torch.nn.Linear whose backward uses the randomized weight gradient
    of Algorithm 1.  rho is the compression rate B_proj / B of Section 2.4; every call draws a
    fresh seed (layer seed in the high word, call counter in the low word), so S is independent
    of the gradients it multiplies."""

    def __init__(self, d_in, d_out, rho=0.2, dist="gaussian", bias=True, layer_seed=0, workspace=None,
                 dtype=torch.bfloat16, device="cuda"):
        super().__init__()
        self.d_in, self.d_out, self.rho = d_in, d_out, float(rho)
        self.dist = _DIST[dist]
        self.weight = torch.nn.Parameter(torch.empty(d_out, d_in, dtype=dtype, device=device))
        self.bias = torch.nn.Parameter(torch.zeros(d_out, dtype=dtype, device=device)) if bias else None
        torch.nn.init.normal_(self.weight, std=0.02)
        self.layer_seed = int(layer_seed) & 0xFFFFFFFF
        self.calls = 0
        self.workspace = workspace if workspace is not None else Workspace()
        self.trace = None          # set to a list to record the tensors of every call (tests)

    def forward(self, x):
        n = x.numel() // self.d_in
        b_proj = n if self.dist == P.RMM_DIST_IDENTITY else bproj_from_rho(n, self.rho)
        seed = (self.layer_seed << 32) | (self.calls & 0xFFFFFFFF)
        self.calls += 1
        return RMMLinearFunction.apply(x, self.weight, self.bias, seed, b_proj, self.dist, self.workspace, self.trace)

    def saved_activation_bytes(self, n_tokens: int) -> int:
        """Bytes this layer keeps between forward and backward for n_tokens rows: X_proj and the seed."""
        b_proj = n_tokens if self.dist == P.RMM_DIST_IDENTITY else bproj_from_rho(n_tokens, self.rho)
        return b_proj * self.d_in * self.weight.element_size() + 8
