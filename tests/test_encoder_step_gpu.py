"""One training step of an encoder built from RMM linear layers (the paper's experimental model,
Section 3): every block linear, with the activations and gradients the step actually produces,
is checked against the CPU oracle; the autograd wiring is checked against stock linears."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

TOL = 1e-2   # relative Frobenius error, bf16 mode


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _check_trace_against_oracle(rec, name):
    """Frobenius gate per tensor and the element-wise gate of tests/gpu_util.py on every element."""
    from oracle import oracle as O
    import rmm_inputs as R
    from tests.gpu_util import contraction_lengths, dw_operand_term, elementwise_excess
    X, W, dY = _np(rec["X"]), _np(rec["W"]), _np(rec["dY"])
    b = None if rec["b"] is None else _np(rec["b"])
    S = O.generate_s(rec["seed"], X.shape[0], rec["b_proj"], rec["dist"], O.STORE_BF16)
    Y, Xp = O.forward(X, W, b, S)
    got_xp = _np(rec["X_proj"])
    dX, dW, db, G = O.backward(dY, W, got_xp, S)     # stage-wise: backward gets the saved X_proj, as the library does
    got = {"Y": _np(rec["Y"]), "X_proj": got_xp, "dX": _np(rec["dX"]), "dW": _np(rec["dW"]), "db": _np(rec["db"])}
    ref = {"Y": Y, "X_proj": Xp, "dX": dX, "dW": dW, "db": db}
    errs = {k: O.rel_frobenius(got[k], ref[k]) for k in ref}
    bad = {k: v for k, v in errs.items() if not v <= TOL}
    assert not bad, f"{name}: {bad} (all {errs})"
    K = contraction_lengths(X.shape[0], X.shape[1], W.shape[0], rec["b_proj"])
    for k in ref:
        term = dw_operand_term(G, got_xp, R.DTYPE_BF16) if k == "dW" else None
        ex, where = elementwise_excess(got[k], ref[k], R.DTYPE_BF16, K[k], term)
        assert ex <= 1.0, f"{name}: {k}{list(where)} is {ex:.2f} x its element-wise bound"
    return errs


def test_small_encoder_every_layer_matches_oracle():
    import encoder_step as E
    cfg = E.Config(hidden=128, heads=2, ffn=512, layers=2, vocab=1000, dropout=0.1, rho=0.5)
    torch.manual_seed(1)
    model = E.Encoder(cfg, "rmm").train()
    for _, m in model.block_linears():
        m.trace = []
    ids, labels = E.make_batch(3, batch=4, seq=72, vocab=cfg.vocab)      # 288 tokens: ragged against every tile size
    loss = E.train_step(model, None, ids, labels)
    torch.cuda.synchronize()
    assert torch.isfinite(loss)
    for name, m in model.block_linears():
        assert len(m.trace) == 1 and "dY" in m.trace[0], name
        assert m.trace[0]["b_proj"] == 144
        _check_trace_against_oracle(m.trace[0], name)
        assert m.weight.grad is not None and torch.equal(m.weight.grad, m.trace[0]["dW"])
        assert torch.equal(m.bias.grad, m.trace[0]["db"])


def test_fused_qkv_layer_matches_oracle_and_saves_one_sketch():
    """Q, K and V as one 3x-wide RMM layer: one S and one X_proj for the three projections."""
    import encoder_step as E
    cfg = E.Config(hidden=64, heads=2, ffn=128, layers=1, vocab=300, dropout=0.0, rho=0.25, fused_qkv=True)
    torch.manual_seed(4)
    model = E.Encoder(cfg, "rmm").train()
    names = [n for n, _ in model.block_linears()]
    assert names == ["block0.qkv", "block0.o", "block0.up", "block0.down"]
    for _, m in model.block_linears():
        m.trace = []
    ids, labels = E.make_batch(7, batch=3, seq=40, vocab=cfg.vocab)
    E.train_step(model, None, ids, labels)
    torch.cuda.synchronize()
    qkv = dict(model.block_linears())["block0.qkv"]
    assert qkv.trace[0]["X_proj"].shape == (30, 64) and qkv.trace[0]["Y"].shape == (120, 192)
    for name, m in model.block_linears():
        _check_trace_against_oracle(m.trace[0], name)


def test_identity_sketch_reproduces_exact_linear_gradients():
    """With S = I (B_proj = N) the layer is the plain linear layer: every parameter gradient of the
    step must equal the one of the same model built from torch.nn.Linear."""
    import encoder_step as E
    cfg = E.Config(hidden=128, heads=4, ffn=256, layers=2, vocab=500, dropout=0.0, dist="identity")
    torch.manual_seed(2)
    rmm = E.Encoder(cfg, "rmm").train()
    exact = E.Encoder(cfg, "exact").train()
    E.copy_weights(exact, rmm)
    ids, labels = E.make_batch(5, batch=2, seq=64, vocab=cfg.vocab)
    l1 = E.train_step(rmm, None, ids, labels)
    l2 = E.train_step(exact, None, ids, labels)
    assert abs(float(l1) - float(l2)) < 2e-2
    ge = dict(exact.named_parameters())
    for name, p in rmm.named_parameters():
        a, b = p.grad.float(), ge[name].grad.float()
        rel = float((a - b).norm() / (b.norm() + 1e-30))
        assert rel < 3e-2, (name, rel)


def test_seed_changes_every_call_and_saved_tensors_are_the_sketch():
    import encoder_step as E
    from paper_2201_13195_b200.rmm_linear import RMMLinear
    lin = RMMLinear(64, 96, rho=0.25, layer_seed=9)
    lin.trace = []
    x = torch.randn(4, 40, 64, device="cuda", dtype=torch.bfloat16, requires_grad=True)
    saved = {}
    with E.count_saved_bytes(lin, saved):
        y = lin(x)
    assert saved["bytes"] == 40 * 64 * 2          # X_proj only: 160 tokens * 0.25 = 40 rows of 64 bf16
    y.sum().backward()
    lin(x).sum().backward()
    s0, s1 = lin.trace[0]["seed"], lin.trace[1]["seed"]
    assert s0 != s1 and s0 >> 32 == 9 and s1 >> 32 == 9
    assert not torch.equal(lin.trace[0]["X_proj"], lin.trace[1]["X_proj"])
    assert x.grad.shape == x.shape and lin.saved_activation_bytes(160) == 40 * 64 * 2 + 8


def test_cpu_tensor_is_rejected():
    from paper_2201_13195_b200.rmm_linear import RMMLinear
    lin = RMMLinear(16, 16)
    with pytest.raises(RuntimeError):
        lin(torch.zeros(8, 16, dtype=torch.bfloat16))


def test_roberta_base_step_sampled_layers_match_oracle():
    """The full configuration (12 blocks, hidden 768, batch 32 x sequence 128 = 4096 tokens, rho = 0.2):
    one layer of each shape, at three depths, against the oracle on the step's own tensors."""
    import encoder_step as E
    cfg = E.Config(**E.ROBERTA_BASE, rho=0.2)
    torch.manual_seed(0)
    model = E.Encoder(cfg, "rmm").train()
    sampled = {"block0.q", "block5.up", "block11.down"}
    mods = dict(model.block_linears())
    for name in sampled:
        mods[name].trace = []
    opt = E.make_optimizer(model)
    ids, labels = E.make_batch(0)
    loss = E.train_step(model, opt, ids, labels)
    torch.cuda.synchronize()
    assert torch.isfinite(loss) and abs(float(loss) - np.log(2.0)) < 0.5     # random init, two classes
    for name in sorted(sampled):
        rec = mods[name].trace[0]
        assert rec["X"].shape[0] == 4096 and rec["b_proj"] == 819
        _check_trace_against_oracle(rec, name)
