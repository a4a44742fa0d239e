"""kdkl_forward_backward (single pass, three projections) against the fp64 oracle and against the two-call path.

Same tolerances as the two-call path: the only arithmetic difference is one more bf16 rounding inside G
(the stored exponential, 2^-9 relative), so the gradient error stays well inside the 1e-2 Frobenius bound;
loss, per-token loss and log Z come from the same sweep and must be bitwise those of kdkl_forward.
"""
import numpy as np
import pytest
import torch

from gradcheck import check_grad_matrix, check_support_rows, dense_dweight
from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import binding as B
from paper_2608_03796_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _fro(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


def _case(T, H, V, K, seed, mask_mode=0, dup=False):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    idx = (torch.randint(0, V, (T, K), generator=g) if dup
           else torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)])).to(torch.int32)
    val = (torch.randn(T, K, generator=g) * 3 ** 0.5).float()
    mask = None
    if mask_mode:
        mask = (torch.rand(T, generator=g) >= 0.15).to(torch.uint8)
        if mask_mode == 2 and T > 600:
            mask[100:100 + 300] = 0                       # a dead run that covers a whole row tile
        idx[mask == 0] = -1
        val[mask == 0] = float("nan")
    return h, W, idx.contiguous(), val.contiguous(), mask


@pytest.mark.parametrize("T,H,V,K,chunk,tau,mask_mode,dup,opts", [
    (256, 256, 4096, 16, 64, 1.0, 0, False, {}),
    (261, 264, 4120, 9, 100, 1.3, 1, False, {"grad_loss": 0.7, "partial": True}),
    (700, 72, 1001, 7, 256, 0.5, 2, True, {"grad_loss": -2.0}),
    (1300, 128, 3000, 33, 0, 2.0, 2, False, {"dh32": 1, "accumulate": 1}),
    (5, 8, 9, 9, 1, 1.0, 0, False, {}),
    (20, 64, 1500, 1024, 0, 1.0, 0, False, {}),            # the largest supported K
    (40, 64, 255, 5, 0, 2.0, 1, False, {}),                # vocabulary smaller than one tile
    (257, 4104, 520, 3, 256, 1.0, 0, False, {}),           # ragged last k-block, rows one past a pair tile
    (130, 72, 8200, 17, 37, 1.0, 1, True, {}),             # vocabulary just past one conversion segment, odd chunk
])
def test_single_pass_matches_oracle_and_two_call_path(T, H, V, K, chunk, tau, mask_mode, dup, opts):
    dev = torch.device("cuda:0")
    h, W, idx, val, mask = _case(T, H, V, K, seed=T + V, mask_mode=mask_mode, dup=dup)
    gl = opts.get("grad_loss", 1.0)
    lse = None
    if opts.get("partial"):
        lse = torch.logsumexp(torch.nan_to_num(val).double() / tau, 1).float() + 0.3
    opt = B.make_options(dhidden_dtype=opts.get("dh32", 0), accumulate_dweight=opts.get("accumulate", 0))
    to = lambda x: None if x is None else x.to(dev)
    base = torch.randn(V, H, generator=torch.Generator().manual_seed(7)) * 1e-4
    # two-call path
    two = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=tau, opt=opt, device=dev, want_per_token=True)
    two.dweight.copy_(base)
    two.forward(to(h), to(W), to(idx), to(val), teacher_lse=to(lse), loss_mask=to(mask))
    two.backward(to(h), to(W), loss_mask=to(mask), grad_loss=gl)
    # single pass
    one = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=tau, opt=opt, device=dev, want_per_token=True)
    one.workspace.view(torch.int16).fill_(0x7fc0)           # a workspace full of bf16 NaN: stale bytes must not matter
    one.dhidden.fill_(float("nan"))
    one.dweight.copy_(base) if opts.get("accumulate") else one.dweight.fill_(float("nan"))
    one.forward_backward(to(h), to(W), to(idx), to(val), teacher_lse=to(lse), loss_mask=to(mask), grad_loss=gl)
    assert one.status()[0] == 0 and two.status()[0] == 0
    assert torch.equal(one.loss, two.loss) and torch.equal(one.loss_per_token, two.loss_per_token)
    assert torch.equal(one.saved_state()[0], two.saved_state()[0])
    mask_np = None if mask is None else mask.numpy()
    with np.errstate(all="ignore"):
        o = kdkl_oracle(h.double().numpy(), W.double().numpy(), idx.numpy(), val.numpy(), tau=tau, mask=mask_np,
                        teacher_lse=None if lse is None else lse.double().numpy(), grad_loss=gl)
    assert abs(one.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
    dH = one.dhidden.float().cpu().double().numpy()
    dW = one.dweight.cpu().double().numpy()
    want_dW = o["dW"] + (base.double().numpy() if opts.get("accumulate") else 0.0)
    assert np.isfinite(dH).all() and np.isfinite(dW).all()
    assert _fro(dH, o["dH"]) <= 1e-2 and _fro(dW, want_dW) <= 1e-2
    if mask is not None:
        assert not dH[mask_np == 0].any()
    # row by row and element by element; G carries two bf16 roundings here (the stored exponential, then G)
    b64 = base.double().numpy() if opts.get("accumulate") else 0.0
    check_grad_matrix(dH, o["dH"], "dH", out_bf16=one.dhidden.dtype == torch.bfloat16, roundings=2)
    dense = dense_dweight(o, h.double().numpy(), W.double().numpy(), idx.numpy(), tau)
    check_grad_matrix(dW - b64, o["dW"], "dW", roundings=2, extra_tol=2.0 ** -22 * np.abs(b64), dense_mag=dense)
    cnt = np.ones(T, bool) if mask is None else mask_np != 0
    check_support_rows(dW - b64, o["dW"], idx.numpy(), list(np.flatnonzero(cnt)[:3]), "dW", roundings=2,
                       dense_mag=dense)
    # and close to the two-call gradients (two independent roundings of G against one)
    assert _fro(dH, two.dhidden.float().cpu().double().numpy()) <= 6e-3
    assert _fro(dW, two.dweight.cpu().double().numpy()) <= 6e-3


def test_single_pass_fullsize_sampled():
    """The benchmark shape: per-token outputs bitwise equal to the two-call path, dH rows on sampled tokens
    against the oracle, column sums of dW vanish, two runs bit for bit."""
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c2"]
    d = I.make_inputs(cfg, device=dev)
    two = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev,
                           want_per_token=True)
    two.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
    tok2 = two.loss_per_token.clone()
    del two
    one = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev,
                           want_per_token=True)
    one.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
    assert one.status()[0] == 0
    assert torch.equal(one.loss_per_token, tok2)
    first = (one.dhidden.clone(), one.dweight.clone())
    one.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
    assert torch.equal(one.dhidden, first[0]) and torch.equal(one.dweight, first[1])
    R = I.sample_rows(cfg, 32).to(dev)
    o = kdkl_oracle(d["hidden"][R].cpu().double().numpy(), d["weight"].cpu().double().numpy(),
                    d["topk_idx"][R].cpu().numpy(), d["topk_val"][R].cpu().numpy(), tau=cfg.tau, denom=cfg.T)
    assert _fro(one.dhidden[R].float().cpu().double().numpy(), o["dH"]) <= 1e-2
    check_grad_matrix(one.dhidden[R].float().cpu().double().numpy(), o["dH"], "dH (sampled rows)", out_bf16=True,
                      roundings=2)
    colsum = one.dweight.double().sum(0).abs()
    colabs = one.dweight.double().abs().sum(0)
    assert (colsum / colabs).max().item() < 3e-3


def test_overflowing_exponential_is_reported_not_hidden():
    """Scaled logits far beyond the representable range of the stored exponential (about 190): the single-pass
    call reports KDKL_ERR_NONFINITE with the row; the two-call path, which normalises by the running maximum,
    handles the same input."""
    dev = torch.device("cuda:0")
    T, H, V, K = 40, 64, 512, 4
    h, W, idx, val, _ = _case(T, H, V, K, seed=3)
    h[7] = 4.0
    W[11] = 4.0                                        # z[7, 11] = 4 * 4 * 64 = 1024, scaled 1477
    one = B.FusedChunkedKL(T, H, V, K, device=dev)
    one.forward_backward(h.to(dev), W.to(dev), idx.to(dev), val.to(dev))
    code, detail = one.status()
    assert code == -11 and detail[0] == 7
    two = B.FusedChunkedKL(T, H, V, K, device=dev)
    two.forward(h.to(dev), W.to(dev), idx.to(dev), val.to(dev))
    two.backward(h.to(dev), W.to(dev))
    assert two.status()[0] == 0 and torch.isfinite(two.dweight).all() and torch.isfinite(two.dhidden.float()).all()
    o = kdkl_oracle(h.double().numpy(), W.double().numpy(), idx.numpy(), val.numpy())
    assert abs(two.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])


def test_single_pass_packed_config_sampled_rows_and_dweight():
    """c5 (16 chunks, packing mask with a dead padding tail, tau = 2, ragged vocabulary): sampled dH rows with the
    full run's denominator, and dW through a second run whose mask is the indicator of the sample."""
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c5"]
    d = I.make_inputs(cfg, device=dev)
    mask = d["mask"]
    n_counted = int(mask.sum().item())
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev,
                          want_per_token=True)
    op.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], loss_mask=mask)
    assert op.status()[0] == 0
    R = I.sample_rows(cfg, 48)
    Rd = R.to(dev)
    hR = d["hidden"][Rd].cpu().double().numpy()
    W64 = d["weight"].cpu().double().numpy()
    idxR, valR = d["topk_idx"][Rd].cpu().numpy(), d["topk_val"][Rd].cpu().numpy()
    mR = mask[Rd].cpu().numpy()
    with np.errstate(all="ignore"):
        o = kdkl_oracle(hR, W64, idxR, valR, tau=cfg.tau, mask=mR, denom=n_counted)
    np.testing.assert_allclose(op.loss_per_token[Rd].cpu().double().numpy(), o["loss_tok"], rtol=0, atol=2e-4)
    assert _fro(op.dhidden[Rd].float().cpu().double().numpy(), o["dH"]) <= 1e-2
    assert not op.dhidden[mask == 0].float().abs().sum().item()
    colsum = op.dweight.double().sum(0).abs()
    assert (colsum / op.dweight.double().abs().sum(0)).max().item() < 3e-3
    # dW: mask = indicator of the counted sampled rows
    mR_full = torch.zeros(cfg.T, dtype=torch.uint8, device=dev)
    mR_full[Rd] = 1
    mR_full &= mask
    nR = int(mR_full.sum().item())
    op.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], loss_mask=mR_full)
    assert op.status()[0] == 0
    with np.errstate(all="ignore"):
        oR = kdkl_oracle(hR, W64, idxR, valR, tau=cfg.tau, mask=mR, denom=nR)
    assert abs(op.loss.item() - oR["loss"]) <= 1e-3 * abs(oR["loss"])
    assert _fro(op.dweight.cpu().double().numpy(), oR["dW"]) <= 1e-2
    check_grad_matrix(op.dweight.cpu().numpy(), oR["dW"], "dW (tokens of the sample)", roundings=2)
    check_support_rows(op.dweight.cpu().numpy(), oR["dW"], idxR, list(np.flatnonzero(mR != 0)[:4]),
                       "dW (tokens of the sample)", roundings=2)


def test_two_calls_with_stored_exponentials_one_chunk():
    """Option stored_exponentials: forward leaves the exponentials, backward forms G from them (no second
    projection), valid when one chunk covers all tokens. Same checks as the single-pass call."""
    dev = torch.device("cuda:0")
    T, H, V, K, tau = 700, 136, 3001, 12, 1.3
    h, W, idx, val, mask = _case(T, H, V, K, seed=77, mask_mode=2)
    opt = B.make_options(stored_exponentials=1)
    op = B.FusedChunkedKL(T, H, V, K, chunk=0, temperature=tau, opt=opt, device=dev, want_per_token=True)
    op.workspace.view(torch.int16).fill_(0x7fc0)
    to = lambda x: None if x is None else x.to(dev)
    op.forward(to(h), to(W), to(idx), to(val), loss_mask=to(mask))
    op.backward(to(h), to(W), loss_mask=to(mask), grad_loss=0.5)
    assert op.status()[0] == 0
    with np.errstate(all="ignore"):
        o = kdkl_oracle(h.double().numpy(), W.double().numpy(), idx.numpy(), val.numpy(), tau=tau, mask=mask.numpy(),
                        grad_loss=0.5)
    assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
    assert _fro(op.dhidden.float().cpu().double().numpy(), o["dH"]) <= 1e-2
    assert _fro(op.dweight.cpu().double().numpy(), o["dW"]) <= 1e-2
    check_grad_matrix(op.dhidden.float().cpu().numpy(), o["dH"], "dH", out_bf16=True, roundings=2)
    check_grad_matrix(op.dweight.cpu().numpy(), o["dW"], "dW", roundings=2)
    # more than one chunk is refused on the host
    with pytest.raises(B.KdklError) as e:
        B.FusedChunkedKL(T, H, V, K, chunk=256, temperature=tau, opt=opt, device=dev).forward(
            to(h), to(W), to(idx), to(val), loss_mask=to(mask))
    assert e.value.code == -5
