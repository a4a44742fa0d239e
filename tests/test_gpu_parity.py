"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle, element by element.

Tolerances (for bf16 inputs, fp32 accumulation, G rounded once to bf16):
  gathered indices            bit-exact
  mean loss                   relative error <= 1e-3
  dHidden, dWeight            relative Frobenius error <= 1e-2 over the whole matrix AND over every row, and
                              every element within the bound tests/gradcheck.py derives from the one bf16
                              rounding of G; the dWeight rows at teacher indices are checked by name
  per-token loss, log Z       absolute error <= 2e-4 (fp32 evaluation of O(10) quantities)
  gathered logits             absolute error <= 1e-4 (fp32 accumulation of exact bf16 products)
"""
import numpy as np
import pytest
import torch

from gradcheck import check_grad_matrix, check_support_rows
from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import binding as B
from paper_2608_03796_b200 import inputs as I

pytestmark = pytest.mark.gpu

LOSS_RTOL, GRAD_FRO, TOK_ATOL, ZG_ATOL = 1e-3, 1e-2, 2e-4, 1e-4


def _dev():
    return torch.device("cuda:0")


def _run(d, T, H, V, K, chunk, tau, lse=None, opt=None, grad_loss=1.0, backward=True):
    dev = _dev()
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    lse_d = None if lse is None else lse.to(dev)
    op = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=tau, opt=opt, device=dev, want_gathered=True,
                          want_per_token=True)
    # poison the outputs: every element must be written by the kernels
    op.dhidden.fill_(float("nan")); op.dweight.fill_(float("nan"))
    op.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], teacher_lse=lse_d, loss_mask=g["mask"])
    if backward:
        op.backward(g["hidden"], g["weight"], loss_mask=g["mask"], grad_loss=grad_loss)
    return op


def _oracle(d, tau, lse=None, teacher_mode=0, grad_loss=1.0, denom=None, want_grads=True):
    return kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                       d["topk_val"].numpy(), tau=tau, mask=None if d["mask"] is None else d["mask"].numpy(),
                       teacher_lse=None if lse is None else lse.double().numpy(), teacher_mode=teacher_mode,
                       grad_loss=grad_loss, denom=denom, want_grads=want_grads)


def _fro(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


def _compare(op, o, d, check_grads=True, dw_base=None):
    code, detail = op.status()
    assert code == 0, (code, detail)
    counted = np.ones(op.T, bool) if d["mask"] is None else d["mask"].numpy() != 0
    loss = op.loss.item()
    assert abs(loss - o["loss"]) <= LOSS_RTOL * abs(o["loss"]) + 1e-7
    lt = op.loss_per_token.cpu().double().numpy()
    np.testing.assert_allclose(lt, o["loss_tok"], rtol=0, atol=TOK_ATOL)
    lz, M = op.saved_state()
    np.testing.assert_allclose(lz.cpu().double().numpy()[counted], o["logZ"][counted], rtol=0, atol=TOK_ATOL)
    assert not lz.cpu().numpy()[~counted].any()            # ignored tokens: log Z is reported as 0
    np.testing.assert_allclose(M.cpu().double().numpy()[counted], o["M"][counted], rtol=0, atol=1e-5)
    # gathered columns: bit-exact wherever the slot holds a usable index of a counted token
    idx = d["topk_idx"].numpy()
    usable = (idx >= 0) & (idx < op.V) & counted[:, None]
    gi = op.gathered_idx.cpu().numpy()
    assert np.array_equal(gi[usable], idx[usable])
    assert np.all(gi[~usable] == -1)
    gl = op.gathered_logits.cpu().double().numpy()
    np.testing.assert_allclose(gl[usable], o["gathered_logits"][usable], rtol=0, atol=ZG_ATOL)
    assert np.all(np.isnan(gl[~usable]))
    if check_grads:
        dH = op.dhidden.float().cpu().double().numpy()
        dW = op.dweight.cpu().double().numpy()
        assert np.isfinite(dH).all() and np.isfinite(dW).all()
        assert _fro(dH, o["dH"]) <= GRAD_FRO, _fro(dH, o["dH"])
        assert _fro(dW, o["dW"]) <= GRAD_FRO, _fro(dW, o["dW"])
        assert not dH[~counted].any()                      # ignored tokens: exact zeros
        # row by row and element by element (a wrong tail row or a missed support entry hides in the norm above)
        base = 0.0 if dw_base is None else dw_base
        check_grad_matrix(dH, o["dH"], "dH", out_bf16=op.dhidden.dtype == torch.bfloat16)
        check_grad_matrix(dW - base, o["dW"] - base, "dW", extra_tol=2.0 ** -22 * np.abs(base))
        some = [t for t in (0, op.T // 2, op.T - 1) if counted[t]] or list(np.flatnonzero(counted)[:3])
        check_support_rows(dW - base, o["dW"] - base, idx, some, "dW")


def _small_case(T, H, V, K, seed, mask_frac=0.0, dup=False, empty=False):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    if dup:
        idx = torch.randint(0, V, (T, K), generator=g, dtype=torch.int64)
    else:
        idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)])
    val = (torch.randn(T, K, generator=g) * 3 ** 0.5).float()
    idx = idx.to(torch.int32)
    if empty:
        idx[torch.rand(T, K, generator=g) < 0.2] = -1
    mask = None
    if mask_frac > 0:
        mask = (torch.rand(T, generator=g) >= mask_frac).to(torch.uint8)
    return {"hidden": h, "weight": W, "topk_idx": idx.contiguous(), "topk_val": val.contiguous(), "mask": mask}


# ------------------------------------------------------------------------------------------ GEMM
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (328, 520, 200), (1024, 1280, 520),
                                   (328, 1000, 200), (520, 1024, 328), (264, 2048, 136)])   # N >= 1000: 512-wide tiles
def test_bare_gemm_all_operand_layouts(M, N, K, a_mn, b_mn):
    g = torch.Generator().manual_seed(M + N + K)
    A = torch.randn(M, K, generator=g).to(torch.bfloat16)
    Bm = torch.randn(N, K, generator=g).to(torch.bfloat16)
    ref = (A.double() @ Bm.double().T).numpy()
    dev = _dev()
    Ad = (A.T.contiguous() if a_mn else A).to(dev)
    Bd = (Bm.T.contiguous() if b_mn else Bm).to(dev)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device=dev)
    st = torch.zeros(2, dtype=torch.int32, device=dev)
    B.kdkl_gemm_bf16(Ad, Bd, C, M, N, K, a_mn, b_mn, st)
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0]
    np.testing.assert_allclose(C.cpu().double().numpy(), ref, rtol=0, atol=1e-5 * K ** 0.5 * 8)


# ------------------------------------------------------------------------------------------ configs
def test_c1_full_parity():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    op = _run(d, cfg.T, cfg.H, cfg.V, cfg.K, cfg.chunk, cfg.tau)
    _compare(op, _oracle(d, cfg.tau), d)
    # column sums of dW vanish: sum_v dz_v = (g/tau)(M - M) = 0 (up to the bf16 rounding of G)
    colsum = op.dweight.double().sum(0).abs()
    colabs = op.dweight.double().abs().sum(0)
    assert (colsum / colabs).max().item() < 2e-3


def test_c1_partial_mass_and_fp32_dhidden():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    lse = I.partial_mass_lse(cfg, d["topk_val"])
    opt = B.make_options(dhidden_dtype=1)
    op = _run(d, cfg.T, cfg.H, cfg.V, cfg.K, cfg.chunk, cfg.tau, lse=lse, opt=opt, grad_loss=0.5)
    o = _oracle(d, cfg.tau, lse=lse, grad_loss=0.5)
    assert o["M"].max() < 1.0
    _compare(op, o, d)


@pytest.mark.parametrize("chunk", [100, 261, 0])
def test_ragged_shapes_mask_temperature(chunk):
    T, H, V, K, tau = 261, 264, 4120, 7, 1.3
    d = _small_case(T, H, V, K, seed=11, mask_frac=0.1)
    d["topk_idx"], d["topk_val"] = I.poison_masked(d["topk_idx"], d["topk_val"], d["mask"])
    op = _run(d, T, H, V, K, chunk, tau)
    _compare(op, _oracle(d, tau), d)


@pytest.mark.parametrize("T,H,V,K,chunk,masked", [
    (700, 1000, 1100, 9, 256, True),     # 512-wide output tiles (ragged last tile), three chunks = groups of 2 + 1
    (700, 1024, 1100, 9, 100, True),     # chunk not a multiple of the row tile: the grouped dW pass takes no flags
    (1300, 1024, 520, 5, 512, True),     # a dead chunk inside a group, a dead tail
    (600, 1536, 777, 4, 0, False),       # one chunk: no grouping, wide tiles, several k-splits of dH
])
def test_wide_output_tiles_and_grouped_dweight(T, H, V, K, chunk, masked):
    """The two output GEMMs at hidden widths that select 512-column tiles, with the dW pass contracting over
    groups of two chunks: ragged widths, short last chunks and groups, ignored runs that kill whole row tiles."""
    d = _small_case(T, H, V, K, seed=T + H)
    if masked:
        mask = torch.ones(T, dtype=torch.uint8)
        mask[::9] = 0
        mask[T // 2: T // 2 + 300] = 0
        mask[T - 40:] = 0
        d["mask"] = mask
        d["topk_idx"], d["topk_val"] = I.poison_masked(d["topk_idx"], d["topk_val"], mask)
    op = _run(d, T, H, V, K, chunk, 1.0)
    _compare(op, _oracle(d, 1.0), d)
    # fp32 dHidden and dW += onto existing contents through the same kernels
    dev = _dev()
    opt = B.make_options(accumulate_dweight=1, dhidden_dtype=1)
    op2 = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=1.0, opt=opt, device=dev, want_gathered=True,
                           want_per_token=True)
    base = torch.randn(V, H, generator=torch.Generator().manual_seed(2)) * 1e-4
    op2.dweight.copy_(base)
    op2.dhidden.fill_(float("nan"))
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    op2.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], loss_mask=g["mask"])
    op2.backward(g["hidden"], g["weight"], loss_mask=g["mask"])
    o = _oracle(d, 1.0)
    o["dW"] = o["dW"] + base.double().numpy()
    _compare(op2, o, d, dw_base=base.double().numpy())
    # and the single-pass call on the same shapes
    op2.dweight.copy_(base)
    op2.dhidden.fill_(float("nan"))
    op2.forward_backward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], loss_mask=g["mask"])
    assert op2.status()[0] == 0
    dW = op2.dweight.cpu().double().numpy() - base.double().numpy()
    dH = op2.dhidden.cpu().double().numpy()
    check_grad_matrix(dH, o["dH"], "dH (single pass)", roundings=2)
    check_grad_matrix(dW, o["dW"] - base.double().numpy(), "dW (single pass)", roundings=2,
                      extra_tol=2.0 ** -22 * np.abs(base.double().numpy()))


def test_duplicates_empty_slots_and_log_prob_mode():
    T, H, V, K = 70, 64, 300, 12
    d = _small_case(T, H, V, K, seed=12, dup=True, empty=True)
    d["topk_idx"][0, :] = 5                                  # a row that is one index K times
    op = _run(d, T, H, V, K, 32, 1.0)
    _compare(op, _oracle(d, 1.0), d)
    # log-probability mode: values are log p with total mass < 1
    d["topk_val"] = d["topk_val"] - torch.logsumexp(d["topk_val"], 1, keepdim=True) - 0.3
    op = _run(d, T, H, V, K, 32, 1.0, opt=B.make_options(teacher_mode=1))
    _compare(op, _oracle(d, 1.0, teacher_mode=1), d)


def test_k1_and_large_k():
    d = _small_case(40, 128, 1000, 1, seed=13)
    _compare(_run(d, 40, 128, 1000, 1, 0, 1.0), _oracle(d, 1.0), d)
    d = _small_case(33, 64, 2048, 600, seed=14)              # K above the usual 100, not a power of two
    _compare(_run(d, 33, 64, 2048, 600, 0, 0.9), _oracle(d, 0.9), d)


@pytest.mark.parametrize("chunk,accumulate", [(600, 0), (600, 1), (0, 0), (256, 0), (300, 0)])
def test_row_tiles_without_counted_tokens_are_skipped(chunk, accumulate):
    """Runs of ignored tokens that cover whole row tiles (a padding tail, a dead first tile, a whole dead
    chunk): those tiles are not computed at all, yet every output must be as if they had been - zero
    dHidden rows, untouched dWeight contributions, per-token loss 0 - and the rest must match the oracle."""
    T, H, V, K = 1300, 72, 1001, 7
    d = _small_case(T, H, V, K, seed=123)
    mask = torch.ones(T, dtype=torch.uint8)
    mask[0:260] = 0            # first 256-row tile of the first chunk dead (whatever the chunk size)
    mask[600:1200] = 0         # with chunk = 600: the whole second chunk; with one chunk: tiles 768..1023 dead
    mask[1290:] = 0            # a short ignored tail inside a live tile
    mask[5] = 1 if chunk == 300 else 0     # chunk 300: a single counted token keeps the first tile alive
    d["mask"] = mask
    d["topk_idx"][mask == 0] = -1
    d["topk_val"][mask == 0] = float("nan")
    dev = torch.device("cuda:0")
    opt = B.make_options(accumulate_dweight=accumulate)
    op = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=1.0, opt=opt, device=dev, want_gathered=True,
                          want_per_token=True)
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    base = torch.randn(V, H, generator=torch.Generator().manual_seed(1)) * 1e-3
    op.dhidden.fill_(float("nan"))
    if accumulate:
        op.dweight.copy_(base)
    else:
        op.dweight.fill_(float("nan"))
    op.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], loss_mask=g["mask"])
    op.backward(g["hidden"], g["weight"], loss_mask=g["mask"])
    o = _oracle(d, 1.0)
    if accumulate:
        o["dW"] = o["dW"] + base.double().numpy()
    _compare(op, o, d, dw_base=base.double().numpy() if accumulate else None)


def test_negative_upstream_gradient():
    T, H, V, K = 130, 64, 1500, 6
    d = _small_case(T, H, V, K, seed=21, mask_frac=0.1)
    op = _run(d, T, H, V, K, 64, 1.2, grad_loss=-2.0)
    _compare(op, _oracle(d, 1.2, grad_loss=-2.0), d)


def test_all_tokens_ignored_gives_zero():
    d = _small_case(50, 64, 512, 4, seed=15)
    d["mask"] = torch.zeros(50, dtype=torch.uint8)
    op = _run(d, 50, 64, 512, 4, 0, 1.0)
    assert op.status()[0] == 0
    assert op.loss.item() == 0.0
    assert not op.dhidden.float().abs().sum().item() and not op.dweight.abs().sum().item()


def test_chunk_invariance_and_determinism():
    T, H, V, K = 384, 128, 3000, 9
    d = _small_case(T, H, V, K, seed=16, mask_frac=0.05)
    a = _run(d, T, H, V, K, 128, 1.0)
    b = _run(d, T, H, V, K, 384, 1.0)
    c = _run(d, T, H, V, K, 128, 1.0)
    # rows do not interact: everything per-token is bitwise independent of the chunk size
    assert torch.equal(a.loss_per_token, b.loss_per_token)
    assert torch.equal(a.dhidden, b.dhidden)
    assert a.loss.item() == b.loss.item()
    # dW sums over chunks in a different order: fp32 reassociation only
    assert _fro(a.dweight.cpu().double().numpy(), b.dweight.cpu().double().numpy()) < 1e-5
    # same call twice: bitwise identical
    assert torch.equal(a.dweight, c.dweight) and torch.equal(a.dhidden, c.dhidden)
    assert torch.equal(a.loss_per_token, c.loss_per_token)


def test_accumulate_dweight_and_denominator_override():
    T, H, V, K = 96, 64, 700, 5
    d = _small_case(T, H, V, K, seed=17)
    base = _run(d, T, H, V, K, 0, 1.0)
    dev = _dev()
    opt = B.make_options(accumulate_dweight=1, denom_override=2.0 * T)
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    op = B.FusedChunkedKL(T, H, V, K, opt=opt, device=dev)
    op.dweight.fill_(1.0)
    op.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"])
    op.backward(g["hidden"], g["weight"])
    assert abs(op.loss.item() - 0.5 * base.loss.item()) < 1e-6
    np.testing.assert_allclose(op.dweight.cpu().numpy(), 1.0 + 0.5 * base.dweight.cpu().numpy(), rtol=0, atol=1e-6)


# ------------------------------------------------------------------------------------------ errors
def test_host_side_error_codes():
    dev = _dev()
    T, H, V, K = 16, 64, 256, 4
    d = _small_case(T, H, V, K, seed=18)
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    ws = torch.empty(B.kdkl_workspace_bytes(T, H, V, K), dtype=torch.uint8, device=dev)
    loss = torch.zeros(1, device=dev)
    def code(fn):
        with pytest.raises(B.KdklError) as e:
            fn()
        return e.value.code
    assert code(lambda: B.kdkl_forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], ws[:1024], loss)) == -4
    assert code(lambda: B.kdkl_forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], ws, loss,
                                       temperature=0.0)) == -5
    assert code(lambda: B.kdkl_forward(g["hidden"][:, :60].contiguous(), g["weight"][:, :60].contiguous(),
                                       g["topk_idx"], g["topk_val"], ws, loss)) == -2
    assert code(lambda: B.kdkl_forward(g["hidden"].view(-1)[1:1 + 15 * 64].view(15, 64), g["weight"],
                                       g["topk_idx"][:15], g["topk_val"][:15], ws, loss)) == -3
    assert code(lambda: B.kdkl_forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], ws, loss,
                                       opt=B.make_options(teacher_mode=1), temperature=2.0)) == -5


def test_device_side_status_codes():
    dev = _dev()
    T, H, V, K = 32, 64, 256, 4
    d = _small_case(T, H, V, K, seed=19)
    # backward on a workspace no forward filled: reported, outputs untouched
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    op = B.FusedChunkedKL(T, H, V, K, device=dev)
    op.workspace.zero_()
    op.dhidden.fill_(7.0); op.dweight.fill_(7.0)
    op.backward(g["hidden"], g["weight"])
    assert op.status()[0] == -9
    assert (op.dhidden.float() == 7.0).all() and (op.dweight == 7.0).all()
    # an index >= V: entry ignored, status says so, result equals the run with the slot emptied
    d2 = {k: (v.clone() if v is not None else None) for k, v in d.items()}
    d2["topk_idx"][3, 1] = V + 5
    op2 = _run(d2, T, H, V, K, 0, 1.0)
    code, detail = op2.status()
    assert code == -10 and detail[2] == 1
    d2["topk_idx"][3, 1] = -1
    op3 = _run(d2, T, H, V, K, 0, 1.0)
    assert op3.status()[0] == 0
    assert torch.equal(op2.loss_per_token, op3.loss_per_token) and torch.equal(op2.dweight, op3.dweight)


def test_invariances_offset_and_slot_permutation():
    """Two invariances the definition has, checked on the GPU path itself: (i) with no teacher_lse the teacher
    is a softmax over the K values, so a per-token constant added to them changes nothing; (ii) the order of
    the K slots of a row is irrelevant (the kernel sorts them): losses agree to fp32 rounding, and the
    gathered logits follow their slots."""
    T, H, V, K, tau = 150, 72, 1001, 13, 1.3
    d = _small_case(T, H, V, K, seed=31)
    base = _run(d, T, H, V, K, 64, tau)
    g = torch.Generator().manual_seed(2)
    shifted = dict(d)
    shifted["topk_val"] = d["topk_val"] + torch.randn(T, 1, generator=g) * 5.0
    a = _run(shifted, T, H, V, K, 64, tau)
    assert (a.loss_per_token - base.loss_per_token).abs().max().item() < 5e-5
    assert ((a.dweight - base.dweight).norm() / base.dweight.norm()).item() < 2e-3
    perm = torch.stack([torch.randperm(K, generator=g) for _ in range(T)])
    shuffled = dict(d)
    shuffled["topk_idx"] = torch.gather(d["topk_idx"], 1, perm).contiguous()
    shuffled["topk_val"] = torch.gather(d["topk_val"], 1, perm).contiguous()
    b = _run(shuffled, T, H, V, K, 64, tau)
    assert (b.loss_per_token - base.loss_per_token).abs().max().item() < 5e-6
    assert torch.equal(b.gathered_idx.cpu(), shuffled["topk_idx"])
    assert torch.equal(b.gathered_logits.cpu(), torch.gather(base.gathered_logits.cpu(), 1, perm))
    # the teacher's normaliser is summed in slot order, so p moves in its last bits and single bf16 roundings of G flip
    assert ((b.dweight - base.dweight).norm() / base.dweight.norm()).item() < 2e-3
    assert ((b.dhidden.float() - base.dhidden.float()).norm() / base.dhidden.float().norm()).item() < 2e-3


def test_one_dweight_pass_per_chunk_option():
    """kdkl_options.dw_chunks_per_pass = 1: one dW pass per chunk instead of per two chunks. One [chunk, V] buffer
    less in the workspace; per-token outputs and dH bitwise the same, dW up to fp32 reassociation; and it matches
    the oracle on its own."""
    T, H, V, K, chunk = 1300, 1024, 900, 6, 256
    d = _small_case(T, H, V, K, seed=44, mask_frac=0.1)
    two = _run(d, T, H, V, K, chunk, 1.0)
    opt = B.make_options(dw_chunks_per_pass=1)
    one = _run(d, T, H, V, K, chunk, 1.0, opt=opt)
    assert B.kdkl_workspace_bytes(T, H, V, K, chunk) - B.kdkl_workspace_bytes(T, H, V, K, chunk, opt) >= chunk * V * 2
    assert torch.equal(one.loss_per_token, two.loss_per_token) and torch.equal(one.dhidden, two.dhidden)
    assert _fro(one.dweight.cpu().double().numpy(), two.dweight.cpu().double().numpy()) < 1e-5
    _compare(one, _oracle(d, 1.0), d)
    with pytest.raises(B.KdklError) as e:
        _run(d, T, H, V, K, chunk, 1.0, opt=B.make_options(dw_chunks_per_pass=3))
    assert e.value.code == -5
