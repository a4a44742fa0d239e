"""Seeded random configurations of the fused loss against the fp64 oracle: shapes, chunk sizes, temperature,
masks with dead runs, duplicate / empty / out-of-range slots, partial teacher mass, log-probability mode,
upstream gradient sign, fp32 dHidden and dW accumulation are all drawn together, so that combinations no
hand-written case lists are exercised. Same tolerances as tests/test_gpu_parity.py.
"""
import numpy as np
import pytest
import torch

from gradcheck import check_grad_matrix, check_support_rows, dense_dweight, term_norms
from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import binding as B

pytestmark = pytest.mark.gpu

LOSS_RTOL, GRAD_FRO, TOK_ATOL, ZG_ATOL = 1e-3, 1e-2, 2e-4, 1e-4


def _draw(seed, wide=False):
    """wide: hidden widths at which the two output GEMMs take their 512-column tiles (and a smaller vocabulary, to
    keep the dense oracle quick)."""
    r = np.random.default_rng(seed)
    T = int(r.choice([1, 7, 64, 130, 257, 400, 700, 1100]))
    H = int(r.choice([1000, 1016, 1024, 1512, 1536, 2048])) if wide else 8 * int(r.integers(1, 40))
    K = int(r.choice([1, 2, 5, 16, 33, 100]))
    V = int(r.integers(max(K, 9), 1200 if wide else 3000))
    chunk = int(r.choice([0, 1, 37, 128, 256, 300, 512])) if T > 1 else 0
    tau = float(r.choice([0.5, 1.0, 1.0, 2.0]))
    mode = int(r.random() < 0.2)                      # log-probability mode needs tau = 1
    if mode:
        tau = 1.0
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    if r.random() < 0.3:
        idx = torch.randint(0, V, (T, K), generator=g)                                   # duplicates allowed
    else:
        idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)])
    idx = idx.to(torch.int32)
    val = (torch.randn(T, K, generator=g) * 3 ** 0.5).float()
    if r.random() < 0.4:
        idx[torch.rand(T, K, generator=g) < 0.15] = -1                                   # empty slots
    if r.random() < 0.25:
        bad = torch.rand(T, K, generator=g) < 0.05
        idx[bad & (idx >= 0)] = V + int(r.integers(0, 5))                                # out-of-range slots
    mask = None
    if r.random() < 0.6:
        mask = (torch.rand(T, generator=g) >= 0.2).to(torch.uint8)
        if T >= 400:                                                                     # a dead run covering row tiles
            a = int(r.integers(0, T - 300))
            mask[a:a + int(r.integers(256, min(T - a, 600) + 1))] = 0
        if r.random() < 0.08:
            mask[:] = 0
    lse = None
    if mode:
        val = val - torch.logsumexp(val, 1, keepdim=True) - float(r.random())           # total mass < 1
    elif r.random() < 0.4:
        lse = torch.logsumexp(val / tau, 1) + torch.rand(T, generator=g) * 0.5           # partial teacher mass
    if mask is not None:                                                                 # ignored rows: never read
        idx[mask == 0] = -1
        val[mask == 0] = float("nan")
    n_bad = int((idx >= V).sum())                     # what the device must count (ignored rows are not read)
    return dict(T=T, H=H, V=V, K=K, chunk=chunk, tau=tau, mode=mode, h=h, W=W, idx=idx.contiguous(),
                val=val.contiguous(), mask=mask, lse=lse, n_bad=n_bad,
                grad_loss=float(r.choice([1.0, 1.0, -0.5, 3.0])), dh32=int(r.random() < 0.3),
                accumulate=int(r.random() < 0.3), denom=float(r.choice([0.0, 0.0, 777.0])))


def _fro(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


@pytest.mark.parametrize("single_pass", [False, True])
@pytest.mark.parametrize("seed", list(range(1000, 1100)) + list(range(3000, 3030)))
def test_random_configuration_matches_oracle(seed, single_pass):
    c = _draw(seed, wide=seed >= 3000)
    dev = torch.device("cuda:0")
    T, H, V, K = c["T"], c["H"], c["V"], c["K"]
    opt = B.make_options(teacher_mode=c["mode"], accumulate_dweight=c["accumulate"], dhidden_dtype=c["dh32"],
                         denom_override=c["denom"])
    op = B.FusedChunkedKL(T, H, V, K, chunk=c["chunk"], temperature=c["tau"], opt=opt, device=dev,
                          want_gathered=True, want_per_token=True)
    base = torch.randn(V, H, generator=torch.Generator().manual_seed(seed + 1)) * 1e-4
    op.workspace.view(torch.int16).fill_(0x7fc0)      # NaN in every float field: nothing may depend on stale workspace
    op.dhidden.fill_(float("nan"))
    op.dweight.copy_(base) if c["accumulate"] else op.dweight.fill_(float("nan"))
    to = lambda x: None if x is None else x.to(dev)
    if single_pass:
        op.forward_backward(to(c["h"]), to(c["W"]), to(c["idx"]), to(c["val"]), teacher_lse=to(c["lse"]),
                            loss_mask=to(c["mask"]), grad_loss=c["grad_loss"])
    else:
        op.forward(to(c["h"]), to(c["W"]), to(c["idx"]), to(c["val"]), teacher_lse=to(c["lse"]),
                   loss_mask=to(c["mask"]))
        op.backward(to(c["h"]), to(c["W"]), loss_mask=to(c["mask"]), grad_loss=c["grad_loss"])
    code, detail = op.status()
    assert code == (-10 if c["n_bad"] else 0), (code, detail)
    if c["n_bad"]:
        assert detail[2] == c["n_bad"]
    mask_np = None if c["mask"] is None else c["mask"].numpy()
    counted = np.ones(T, bool) if mask_np is None else mask_np != 0
    with np.errstate(all="ignore"):
        o = kdkl_oracle(c["h"].double().numpy(), c["W"].double().numpy(), c["idx"].numpy(), c["val"].numpy(),
                        tau=c["tau"], mask=mask_np, teacher_lse=None if c["lse"] is None else c["lse"].double().numpy(),
                        teacher_mode=c["mode"], grad_loss=c["grad_loss"], denom=c["denom"] if c["denom"] > 0 else None)
    assert abs(op.loss.item() - o["loss"]) <= LOSS_RTOL * abs(o["loss"]) + 1e-6
    np.testing.assert_allclose(op.loss_per_token.cpu().double().numpy(), o["loss_tok"], rtol=0, atol=TOK_ATOL)
    lz, M = op.saved_state()
    np.testing.assert_allclose(lz.cpu().double().numpy()[counted], o["logZ"][counted], rtol=0, atol=TOK_ATOL)
    np.testing.assert_allclose(M.cpu().double().numpy()[counted], o["M"][counted], rtol=0, atol=1e-5)
    idx = c["idx"].numpy()
    if not single_pass:                               # the single-pass call does not return the gathered logits
        usable = (idx >= 0) & (idx < V) & counted[:, None]
        gi = op.gathered_idx.cpu().numpy()
        assert np.array_equal(gi[usable], idx[usable]) and np.all(gi[~usable] == -1)
        gl = op.gathered_logits.cpu().double().numpy()
        np.testing.assert_allclose(gl[usable], o["gathered_logits"][usable], rtol=0, atol=ZG_ATOL)
    dH = op.dhidden.float().cpu().double().numpy()
    dW = op.dweight.cpu().double().numpy()
    want_dW = o["dW"] + (base.double().numpy() if c["accumulate"] else 0.0)
    assert np.isfinite(dH).all() and np.isfinite(dW).all()
    assert not dH[~counted].any()
    if counted.any():
        assert _fro(dH, o["dH"]) <= GRAD_FRO and _fro(dW, want_dW) <= GRAD_FRO
        # every row and every element (the single-pass step rounds its stored exponential as well: two roundings)
        nr = 2 if single_pass else 1
        b64 = base.double().numpy() if c["accumulate"] else 0.0
        nH, nW = term_norms(o, c["h"].double().numpy(), c["W"].double().numpy(), idx, c["tau"])
        check_grad_matrix(dH, o["dH"], "dH", out_bf16=not c["dh32"], roundings=nr, row_scale=nH)
        dense = dense_dweight(o, c["h"].double().numpy(), c["W"].double().numpy(), idx, c["tau"]) if single_pass else None
        check_grad_matrix(dW - b64, o["dW"], "dW", roundings=nr, extra_tol=2.0 ** -22 * np.abs(b64), dense_mag=dense,
                          row_scale=nW)
        check_support_rows(dW - b64, o["dW"], idx, list(np.flatnonzero(counted)[:3]), "dW", roundings=nr,
                           dense_mag=dense, row_scale=nW)
    else:
        assert not dH.any() and np.array_equal(dW, want_dW)
