"""One training step of a random-init RoBERTa-base-shaped encoder whose six linear layers per
block are RMM layers (the paper's experimental model, Section 3: all linear layers of the
Transformer blocks are replaced).

The harness around the layer is stock PyTorch (embeddings, scaled-dot-product attention,
LayerNorm, GELU, classifier head, cross-entropy, AdamW): it is not the subject, it supplies
the layer with the activations and gradients of a real training step.  `linear="rmm"` builds
the blocks from `RMMLinear` (C-ABI library), `linear="exact"` from torch.nn.Linear with the
same initial weights, for step-time and saved-activation comparisons.

Inputs are synthetic: token ids uniform over the vocabulary, labels uniform over two classes.
"""
import contextlib

import torch
import torch.nn.functional as F


class Config:
    def __init__(self, hidden=768, heads=12, ffn=3072, layers=12, vocab=50265, max_pos=514, classes=2, dropout=0.1,
                 rho=0.2, dist="gaussian", fused_qkv=False):
        self.hidden, self.heads, self.ffn, self.layers = hidden, heads, ffn, layers
        self.vocab, self.max_pos, self.classes, self.dropout = vocab, max_pos, classes, dropout
        self.rho, self.dist = rho, dist
        # fused_qkv: one hidden -> 3 hidden layer for Q, K and V.  As an RMM layer it draws one S and
        # keeps one X_proj for the three projections, which all read the same input.
        self.fused_qkv = fused_qkv


ROBERTA_BASE = dict(hidden=768, heads=12, ffn=3072, layers=12)


def _make_linear(kind, d_in, d_out, cfg, layer_seed, workspace):
    if kind == "rmm":
        from paper_2201_13195_b200.rmm_linear import RMMLinear
        return RMMLinear(d_in, d_out, rho=cfg.rho, dist=cfg.dist, bias=True, layer_seed=layer_seed, workspace=workspace)
    lin = torch.nn.Linear(d_in, d_out, bias=True, device="cuda", dtype=torch.bfloat16)
    torch.nn.init.normal_(lin.weight, std=0.02)
    torch.nn.init.zeros_(lin.bias)
    return lin


class Block(torch.nn.Module):
    """Post-LayerNorm Transformer block: self-attention (q, k, v, o) and feed-forward (up, down)."""

    NAMES = ("q", "k", "v", "o", "up", "down")
    NAMES_FUSED = ("qkv", "o", "up", "down")

    def __init__(self, cfg, kind, index, workspace):
        super().__init__()
        h, f = cfg.hidden, cfg.ffn
        shapes = {"q": (h, h), "k": (h, h), "v": (h, h), "qkv": (h, 3 * h), "o": (h, h), "up": (h, f), "down": (f, h)}
        self.names = self.NAMES_FUSED if cfg.fused_qkv else self.NAMES
        for i, name in enumerate(self.names):
            setattr(self, name, _make_linear(kind, *shapes[name], cfg, 6 * index + i + 1, workspace))
        self.ln1 = torch.nn.LayerNorm(h, device="cuda", dtype=torch.bfloat16)
        self.ln2 = torch.nn.LayerNorm(h, device="cuda", dtype=torch.bfloat16)
        self.heads, self.p = cfg.heads, cfg.dropout

    def forward(self, x):
        b, s, h = x.shape
        split = lambda t: t.view(b, s, self.heads, h // self.heads).transpose(1, 2)
        if len(self.names) == 4:
            q, k, v = self.qkv(x).split(h, dim=-1)
        else:
            q, k, v = self.q(x), self.k(x), self.v(x)
        a = F.scaled_dot_product_attention(split(q), split(k), split(v), dropout_p=self.p if self.training else 0.0)
        a = self.o(a.transpose(1, 2).reshape(b, s, h))
        x = self.ln1(x + F.dropout(a, self.p, self.training))
        y = self.down(F.gelu(self.up(x)))
        return self.ln2(x + F.dropout(y, self.p, self.training))


class Encoder(torch.nn.Module):
    def __init__(self, cfg: Config, linear="rmm"):
        super().__init__()
        self.cfg, self.kind = cfg, linear
        workspace = None
        if linear == "rmm":
            from paper_2201_13195_b200.rmm_linear import Workspace
            workspace = Workspace()
        kw = dict(device="cuda", dtype=torch.bfloat16)
        self.tok = torch.nn.Embedding(cfg.vocab, cfg.hidden, **kw)
        self.pos = torch.nn.Embedding(cfg.max_pos, cfg.hidden, **kw)
        self.ln = torch.nn.LayerNorm(cfg.hidden, **kw)
        self.blocks = torch.nn.ModuleList([Block(cfg, linear, i, workspace) for i in range(cfg.layers)])
        self.head_dense = torch.nn.Linear(cfg.hidden, cfg.hidden, **kw)
        self.head_out = torch.nn.Linear(cfg.hidden, cfg.classes, **kw)
        for emb in (self.tok, self.pos):
            torch.nn.init.normal_(emb.weight, std=0.02)

    def forward(self, ids):
        pos = torch.arange(ids.shape[1], device=ids.device) + 2      # RoBERTa's position offset
        x = self.ln(self.tok(ids) + self.pos(pos)[None])
        x = F.dropout(x, self.cfg.dropout, self.training)
        for blk in self.blocks:
            x = blk(x)
        return self.head_out(torch.tanh(self.head_dense(x[:, 0]))).float()

    def block_linears(self):
        """[(name, module)] of the linear layers inside the blocks (6 per block, 4 with fused QKV), in forward order."""
        return [(f"block{i}.{n}", getattr(b, n)) for i, b in enumerate(self.blocks) for n in b.names]


def copy_weights(dst: Encoder, src: Encoder):
    """Same initial parameters in both models (their parameter names coincide)."""
    dst.load_state_dict(src.state_dict())


def make_batch(seed, batch=32, seq=128, vocab=50265, classes=2):
    g = torch.Generator(device="cuda").manual_seed(seed)
    ids = torch.randint(0, vocab, (batch, seq), device="cuda", generator=g)
    labels = torch.randint(0, classes, (batch,), device="cuda", generator=g)
    return ids, labels


def make_optimizer(model):
    return torch.optim.AdamW(model.parameters(), lr=1e-5, weight_decay=0.1, fused=True)


def train_step(model, opt, ids, labels):
    """Forward, 2-class cross-entropy, backward, AdamW update; returns the loss tensor."""
    loss = F.cross_entropy(model(ids), labels)
    loss.backward()
    if opt is not None:
        opt.step()
        opt.zero_grad(set_to_none=True)
    return loss.detach()


@contextlib.contextmanager
def count_saved_bytes(model, out):
    """Counts the bytes autograd keeps for backward while the block is active (distinct storages,
    parameters excluded): out["bytes"] = activations saved between forward and backward."""
    params = {p.untyped_storage().data_ptr() for p in model.parameters()}
    seen = {}

    def pack(t):
        if isinstance(t, torch.Tensor) and t.is_cuda:
            st = t.untyped_storage()
            if st.data_ptr() not in params:
                seen[st.data_ptr()] = st.nbytes()
        return t

    with torch.autograd.graph.saved_tensors_hooks(pack, lambda t: t):
        yield
    out["bytes"] = sum(seen.values())
    out["tensors"] = len(seen)


def measure(linear, cfg: Config, batch=32, seq=128, steps=10, warmup=3, seed=0):
    """Step time (CUDA events), saved-activation bytes and peak allocated memory of one model."""
    torch.manual_seed(seed)
    model = Encoder(cfg, linear).train()
    opt = make_optimizer(model)
    ids, labels = make_batch(seed, batch, seq, cfg.vocab, cfg.classes)
    for _ in range(warmup):
        train_step(model, opt, ids, labels)
    torch.cuda.synchronize()
    saved = {}
    base = torch.cuda.memory_allocated()
    torch.cuda.reset_peak_memory_stats()
    with count_saved_bytes(model, saved):
        loss = F.cross_entropy(model(ids), labels)
    after_forward = torch.cuda.memory_allocated()
    loss.backward()
    opt.step()
    opt.zero_grad(set_to_none=True)
    torch.cuda.synchronize()
    peak = torch.cuda.max_memory_allocated()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        loss = train_step(model, opt, ids, labels)
    e1.record()
    torch.cuda.synchronize()
    n_tokens = batch * seq
    lin_saved = None
    if linear == "rmm":
        lin_saved = sum(m.saved_activation_bytes(n_tokens) for _, m in model.block_linears())
    else:
        lin_saved = sum(n_tokens * m.in_features * 2 for _, m in model.block_linears())
    return {"linear": linear, "ms_per_step": e0.elapsed_time(e1) / steps, "loss": float(loss),
            "saved_bytes_all": saved["bytes"], "saved_bytes_block_linear_inputs": lin_saved,
            "held_after_forward_bytes": after_forward - base, "peak_allocated_bytes": peak,
            "tokens": n_tokens}


def main():
    """python encoder_step.py [--steps K] [--warmup W] [--rho R]: one JSON line with the step time, the
    saved-activation bytes and the peak allocated memory of the RoBERTa-base-shaped encoder built
    from RMM linears and from exact linears (batch 32, sequence 128, one GPU)."""
    import argparse
    import json
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--rho", type=float, default=0.2)
    ap.add_argument("--dist", default="gaussian", choices=["gaussian", "rademacher", "sors", "dct"])
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--seq", type=int, default=128)
    ap.add_argument("--fused-qkv", action="store_true", help="one 768 -> 2304 layer (one S, one X_proj) for Q, K, V")
    # Default 2: in this eager-PyTorch harness the step is bound by the host's enqueue rate (about a thousand small
    # launches per step), and the side-by-side mode enqueues four more stream operations per pass; the per-layer
    # benchmark (bench.py), where the GPU is the bound, uses the library's default 0.
    ap.add_argument("--pass-mode", type=int, default=2, choices=[0, 1, 2],
                    help="how the library runs a pass: 0 two kernels side by side, 1 one launch, 2 two kernels in turn")
    a = ap.parse_args()
    import paper_2201_13195_b200 as P
    P.rmm_set_pass_mode(a.pass_mode)
    cfg = Config(**ROBERTA_BASE, rho=a.rho, dist=a.dist, fused_qkv=a.fused_qkv)
    res = {}
    for kind in ("rmm", "exact"):
        res[kind] = measure(kind, cfg, a.batch, a.seq, a.steps, max(a.warmup, 3))
        torch.cuda.empty_cache()
    n = a.batch * a.seq
    shared_qkv_exact = cfg.layers * n * (cfg.hidden * 3 + cfg.ffn) * 2      # q, k, v read one saved input
    line = {"metric": "RoBERTa-base encoder training step, all 6 linears per block as RMM", "unit": "ms",
            "value": res["rmm"]["ms_per_step"], "higher_is_better": False, "n_gpus": 1, "steps": a.steps,
            "warmup": max(a.warmup, 3), "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "roberta_base_encoder", "layers": cfg.layers, "hidden": cfg.hidden, "ffn": cfg.ffn,
                       "batch": a.batch, "seq": a.seq, "rho": a.rho, "sketch": a.dist, "optimizer": "AdamW (fused)",
                       "fused_qkv": a.fused_qkv, "pass_mode": a.pass_mode},
            "exact_linear_ms": res["exact"]["ms_per_step"],
            "saved_activation_bytes": {
                "block_linear_inputs_rmm": res["rmm"]["saved_bytes_block_linear_inputs"],
                "block_linear_inputs_exact_per_linear": res["exact"]["saved_bytes_block_linear_inputs"],
                "block_linear_inputs_exact_shared_qkv": shared_qkv_exact,
                "all_saved_tensors_rmm": res["rmm"]["saved_bytes_all"],
                "all_saved_tensors_exact": res["exact"]["saved_bytes_all"]},
            "held_after_forward_bytes": {"rmm": res["rmm"]["held_after_forward_bytes"],
                                         "exact": res["exact"]["held_after_forward_bytes"]},
            "peak_allocated_bytes": {"rmm": res["rmm"]["peak_allocated_bytes"],
                                     "exact": res["exact"]["peak_allocated_bytes"]},
            "loss": {"rmm": res["rmm"]["loss"], "exact": res["exact"]["loss"]}}
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
