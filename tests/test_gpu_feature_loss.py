"""GPU parity of the hidden-state feature loss (MSE and cosine) against the fp64 oracle, through the C ABI.

Tolerances, from the arithmetic: row sums of H <= 20000 products are taken in fp32 (a tree over the
threads of a row, 8..80 serial terms per thread) and the sum over tokens in fp64, so per-token values
and the loss agree with fp64 to a few 1e-6 relative; the gradient is rounded once to bf16
(relative 2^-9 per element), so its relative Frobenius error stays below 4e-3.
"""
import numpy as np
import pytest
import torch

from oracle.feature_oracle import KIND_COSINE, KIND_MSE, feature_loss_oracle
from paper_2608_03796_b200 import binding as B
from paper_2608_03796_b200 import inputs as I

pytestmark = pytest.mark.gpu

LOSS_RTOL, TOK_TOL, GRAD_FRO = 2e-5, 2e-5, 4e-3


def _pair(T, H, seed):
    g = torch.Generator().manual_seed(seed)
    s = torch.randn(T, H, generator=g)
    r = 0.7 * s + 0.7 * torch.randn(T, H, generator=g) + 0.1
    return s.to(torch.bfloat16), r.to(torch.bfloat16)


def _run(s, r, kind, dev, mask=None, weight=1.0, grad_loss=1.0, denom=0.0, accumulate=0, dst=None, want_grad=True):
    T, H = s.shape
    ws = torch.empty(B.kdkl_feature_loss_workspace_bytes(T), dtype=torch.uint8, device=dev)
    loss = torch.full((1,), float("nan"), device=dev)
    tok = torch.full((T,), float("nan"), device=dev)
    if want_grad and dst is None:
        dst = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device=dev)
    B.kdkl_feature_loss(s.to(dev), r.to(dev), ws, loss, kind=kind, loss_mask=None if mask is None else mask.to(dev),
                        weight=weight, grad_loss=grad_loss, denom_override=denom, accumulate=accumulate,
                        loss_per_token=tok, dstudent=dst if want_grad else None)
    torch.cuda.synchronize()
    return loss.item(), tok.cpu().double().numpy(), None if not want_grad else dst.float().cpu().double().numpy()


def _fro(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


@pytest.mark.parametrize("kind", [KIND_MSE, KIND_COSINE])
@pytest.mark.parametrize("T,H", [
    (1, 8),            # one token, the narrowest legal row
    (37, 72),          # one warp per row, ragged last vector group
    (130, 1024),       # one warp per row, four vectors per lane
    (9, 1032),         # first width past one warp per row
    (40, 3072),        # 128 threads per row, three vectors each
    (257, 4096),       # the benchmark's hidden size
    (21, 8192),        # whole block per row, four vectors per thread
    (33, 16384),       # eight vectors per thread
    (19, 20000),       # wider than the register budget: the tail is re-read
])
def test_matches_oracle(kind, T, H):
    dev = torch.device("cuda:0")
    s, r = _pair(T, H, seed=T * 31 + H)
    mask = (torch.arange(T) % 5 != 3).to(torch.uint8) if T > 4 else None
    if mask is not None:                                   # ignored rows hold NaN: they must never be read
        s = s.clone(); r = r.clone()
        s[mask == 0] = float("nan"); r[mask == 0] = float("inf")
    loss, tok, dS = _run(s, r, kind, dev, mask=mask, weight=0.6, grad_loss=1.5)
    with np.errstate(all="ignore"):
        o = feature_loss_oracle(s.double().numpy(), r.double().numpy(), kind, mask=None if mask is None else mask.numpy(),
                                weight=0.6, grad_loss=1.5)
    assert abs(loss - o["loss"]) <= LOSS_RTOL * abs(o["loss"]) + 1e-9
    np.testing.assert_allclose(tok, o["loss_tok"], rtol=TOK_TOL, atol=TOK_TOL)
    assert np.isfinite(dS).all()
    assert _fro(dS, o["dS"]) <= GRAD_FRO
    # element by element: within one bf16 rounding of the exact value (plus fp32 noise on the coefficients)
    assert (np.abs(dS - o["dS"]) <= 2.0 ** -8 * np.abs(o["dS"]) + 1e-30 + 1e-5 * np.abs(o["dS"]).max()).all()
    if mask is not None:
        assert not dS[mask.numpy() == 0].any() and not tok[mask.numpy() == 0].any()


@pytest.mark.parametrize("kind", [KIND_MSE, KIND_COSINE])
def test_accumulate_loss_only_and_denominator(kind):
    dev = torch.device("cuda:0")
    T, H = 150, 2048
    s, r = _pair(T, H, seed=5)
    mask = (torch.arange(T) % 4 != 0).to(torch.uint8)
    o = feature_loss_oracle(s.double().numpy(), r.double().numpy(), kind, mask=mask.numpy(), denom=500.0)
    # accumulate adds to what the buffer holds and leaves ignored rows alone
    base = torch.randn(T, H, generator=torch.Generator().manual_seed(9)).mul(float(np.abs(o["dS"]).mean()))
    base = base.to(torch.bfloat16)                         # same magnitude as the gradient that is added
    dst = base.clone().to(dev)
    loss, tok, dS = _run(s, r, kind, dev, mask=mask, denom=500.0, accumulate=1, dst=dst)
    assert abs(loss - o["loss"]) <= LOSS_RTOL * abs(o["loss"])
    want = base.double().numpy() + o["dS"]
    assert _fro(dS, want) <= GRAD_FRO
    assert np.array_equal(dS[mask.numpy() == 0], base.double().numpy()[mask.numpy() == 0])
    # loss only: same loss bit for bit, no gradient buffer needed
    loss2, tok2, _ = _run(s, r, kind, dev, mask=mask, denom=500.0, want_grad=False)
    assert loss2 == loss and np.array_equal(tok, tok2)


def test_degenerate_rows_and_empty_mask():
    dev = torch.device("cuda:0")
    s, r = _pair(6, 64, seed=2)
    s[2] = 0                                   # zero student row: cosine undefined, f = 1 and no gradient
    r[4] = s[4]                                # equal rows: both losses 0, both gradients 0
    loss, tok, dS = _run(s, r, KIND_COSINE, dev)
    o = feature_loss_oracle(s.double().numpy(), r.double().numpy(), KIND_COSINE)
    assert tok[2] == 1.0 and not dS[2].any()
    assert abs(tok[4]) < 1e-6 and np.abs(dS[4]).max() < 1e-6
    assert abs(loss - o["loss"]) <= LOSS_RTOL * abs(o["loss"])
    lm, tm, dm = _run(s, r, KIND_MSE, dev)
    assert tm[4] == 0.0 and not dm[4].any()
    for kind in (KIND_MSE, KIND_COSINE):
        l0, t0, d0 = _run(s, r, kind, dev, mask=torch.zeros(6, dtype=torch.uint8))
        assert l0 == 0.0 and not t0.any() and not d0.any()


@pytest.mark.parametrize("kind", [KIND_MSE, KIND_COSINE])
def test_fullsize_sampled_rows_and_reproducibility(kind):
    """The long-context shape (T=32768, H=4096): sampled rows against the oracle with the full run's
    denominator, the mean against the per-token values, and two runs bit for bit."""
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c5"] if kind == KIND_COSINE else I.CONFIGS["c3"]
    s = I.hidden(cfg, device=dev)
    r = I.teacher_hidden(cfg, device=dev)
    mask = I.loss_mask(cfg, device=dev)
    n = cfg.T if mask is None else int(mask.sum().item())
    ws = torch.empty(B.kdkl_feature_loss_workspace_bytes(cfg.T), dtype=torch.uint8, device=dev)
    out = []
    for _ in range(2):
        loss = torch.zeros(1, device=dev); tok = torch.empty(cfg.T, device=dev)
        dS = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device=dev)
        B.kdkl_feature_loss(s, r, ws, loss, kind=kind, loss_mask=mask, loss_per_token=tok, dstudent=dS)
        torch.cuda.synchronize()
        out.append((loss.clone(), tok, dS))
    assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1]) and torch.equal(out[0][2], out[1][2])
    loss, tok, dS = out[0]
    assert abs(loss.item() - tok.double().sum().item() / n) <= 1e-6 * abs(loss.item())
    R = I.sample_rows(cfg, 256).to(dev)
    mR = None if mask is None else mask[R].cpu().numpy()
    o = feature_loss_oracle(s[R].cpu().double().numpy(), r[R].cpu().double().numpy(), kind, mask=mR, denom=n)
    np.testing.assert_allclose(tok[R].cpu().double().numpy(), o["loss_tok"], rtol=TOK_TOL, atol=TOK_TOL)
    assert _fro(dS[R].float().cpu().double().numpy(), o["dS"]) <= GRAD_FRO
    if mask is not None:
        assert not dS[mask == 0].float().abs().sum().item()
    # statistical sanity of the generator (correlation 0.8, unit variances): a gross-error alarm only
    expect = 0.2 if kind == KIND_COSINE else 0.4
    assert abs(loss.item() - expect) < 0.02


def test_adds_onto_the_kl_gradient():
    """Logit KL + feature loss on the same final hidden states: kdkl_backward writes dHidden, the feature
    loss accumulates onto it, and the sum matches the two oracles' sum."""
    from oracle.kdkl_oracle import kdkl_oracle
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    r = I.teacher_hidden(cfg, device=dev)
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev)
    op.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
    op.backward(d["hidden"], d["weight"])
    ws = torch.empty(B.kdkl_feature_loss_workspace_bytes(cfg.T), dtype=torch.uint8, device=dev)
    floss = torch.zeros(1, device=dev)
    B.kdkl_feature_loss(d["hidden"], r, ws, floss, kind=KIND_MSE, weight=0.5, accumulate=1, dstudent=op.dhidden)
    torch.cuda.synchronize()
    assert op.status()[0] == 0
    ok = kdkl_oracle(d["hidden"].cpu().double().numpy(), d["weight"].cpu().double().numpy(), d["topk_idx"].cpu().numpy(),
                     d["topk_val"].cpu().numpy(), tau=cfg.tau)
    of = feature_loss_oracle(d["hidden"].cpu().double().numpy(), r.cpu().double().numpy(), KIND_MSE, weight=0.5)
    total = op.loss.item() + floss.item()
    assert abs(total - (ok["loss"] + of["loss"])) <= 1e-3 * abs(ok["loss"] + of["loss"])
    assert _fro(op.dhidden.float().cpu().double().numpy(), ok["dH"] + of["dS"]) <= 1e-2


@pytest.mark.parametrize("kind", [KIND_MSE, KIND_COSINE])
@pytest.mark.parametrize("masked", [False, True])
def test_upstream_gradient_read_on_the_device_gives_the_same_bits(kind, masked):
    """kdkl_feature_loss_device_grad: the gradient factor comes from device memory instead of the argument list;
    loss, per-token values and gradient must be those of the by-value call, with and without a mask (without one the
    by-value call takes N on the host and the device-gradient call counts it on the device)."""
    dev = torch.device("cuda:0")
    T, H = 300, 264
    s, r = _pair(T, H, seed=5)
    mask = (torch.arange(T) % 5 != 0).to(torch.uint8) if masked else None
    for g in (1.0, -2.5):
        a = _run(s, r, kind, dev, mask=mask, weight=0.6, grad_loss=g)
        b = _run(s, r, kind, dev, mask=mask, weight=0.6, grad_loss=torch.full((1,), g, device=dev))
        assert a[0] == b[0] and np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])
