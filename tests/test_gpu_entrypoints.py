"""The host-buffer end-to-end entry point and the per-stage profiling entry point against the plain calls."""
import pytest
import torch

from paper_2608_03796_b200 import binding as B
from paper_2608_03796_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _device_run(cfg, d, dev, opt=None):
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev, opt=opt)
    op.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], loss_mask=g["mask"])
    op.backward(g["hidden"], g["weight"], loss_mask=g["mask"])
    assert op.status()[0] == 0
    return g, op


def test_host_buffer_call_equals_device_calls_bitwise():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    dev = torch.device("cuda:0")
    _, op = _device_run(cfg, d, dev)
    arena = torch.empty(B.kdkl_host_arena_bytes(cfg.T, cfg.H, cfg.V, cfg.K, cfg.chunk), dtype=torch.uint8, device=dev)
    loss_h = torch.zeros(1).pin_memory()
    dh_h = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16).pin_memory()
    dw_h = torch.empty(cfg.V, cfg.H, dtype=torch.float32).pin_memory()
    hh = {k: (v.pin_memory() if v is not None else None) for k, v in d.items()}
    B.kdkl_forward_backward_host(hh["hidden"], hh["weight"], hh["topk_idx"], hh["topk_val"], arena, loss_h, dh_h, dw_h,
                                 chunk=cfg.chunk, temperature=cfg.tau)
    assert loss_h.item() == op.loss.item()
    assert torch.equal(dh_h, op.dhidden.cpu()) and torch.equal(dw_h, op.dweight.cpu())
    assert B.kdkl_last_launch_count() == op.launches
    # too small an arena is refused before anything is copied
    with pytest.raises(B.KdklError) as e:
        B.kdkl_forward_backward_host(hh["hidden"], hh["weight"], hh["topk_idx"], hh["topk_val"], arena[:4096], loss_h,
                                     dh_h, dw_h, chunk=cfg.chunk, temperature=cfg.tau)
    assert e.value.code == -4


def test_step_with_the_teacher_record_on_the_host_equals_device_calls_bitwise():
    """Teacher record + mask from pinned host memory, everything else resident: same bits as the device calls."""
    import dataclasses
    dev = torch.device("cuda:0")
    cfg = dataclasses.replace(I.CONFIGS["c5"], T=1300, H=256, V=4104, chunk=512)       # with the packing mask
    d = I.make_inputs(cfg)
    lse = I.partial_mass_lse(cfg, torch.nan_to_num(d["topk_val"]))
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev)
    op.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], teacher_lse=lse.to(dev), loss_mask=g["mask"])
    op.backward(g["hidden"], g["weight"], loss_mask=g["mask"], grad_loss=0.5)
    assert op.status()[0] == 0
    want = (op.loss.item(), op.dhidden.clone(), op.dweight.clone())
    staging = torch.empty(B.kdkl_record_staging_bytes(cfg.T, cfg.K), dtype=torch.uint8, device=dev)
    ws = torch.empty_like(op.workspace)
    dh = torch.full_like(op.dhidden, float("nan"))
    dw = torch.full_like(op.dweight, float("nan"))
    loss_h = torch.zeros(1).pin_memory()
    B.kdkl_step_host_record(g["hidden"], g["weight"], d["topk_idx"].pin_memory(), d["topk_val"].pin_memory(), staging,
                            ws, loss_h, dh, dw, teacher_lse_host=lse.pin_memory(), loss_mask_host=d["mask"].pin_memory(),
                            chunk=cfg.chunk, temperature=cfg.tau, grad_loss=0.5)
    assert B.kdkl_status(ws)[0] == 0
    assert loss_h.item() == want[0] and torch.equal(dh, want[1]) and torch.equal(dw, want[2])
    assert B.kdkl_last_launch_count() == op.launches
    with pytest.raises(B.KdklError) as e:
        B.kdkl_step_host_record(g["hidden"], g["weight"], d["topk_idx"].pin_memory(), d["topk_val"].pin_memory(),
                                staging[:1024], ws, loss_h, dh, dw, chunk=cfg.chunk, temperature=cfg.tau)
    assert e.value.code == -4


def test_profile_stages_accounts_for_every_launch_and_changes_nothing():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    dev = torch.device("cuda:0")
    g, op = _device_run(cfg, d, dev)
    ref_loss, ref_dw = op.loss.clone(), op.dweight.clone()
    st = B.kdkl_profile_stages(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], op.workspace, op.loss, op.dhidden,
                               op.dweight, chunk=cfg.chunk, temperature=cfg.tau)
    chunks = cfg.T // cfg.chunk
    assert st["fwd_gemm_lse"][1] == chunks and st["bwd_gemm_dlogits"][1] == chunks
    assert st["dhidden_gemm"][1] == chunks and st["combine"][1] == chunks
    assert st["dweight_gemm"][1] == (chunks + 1) // 2          # one dW pass per group of two chunks
    assert st["prep"][1] == 1 and st["loss_reduce"][1] == 1 and st["bwd_coef"][1] == 1
    assert all(ms > 0 for ms, n in st.values())
    assert torch.equal(op.loss, ref_loss) and torch.equal(op.dweight, ref_dw)


def test_profile_single_pass_accounts_for_every_stage_and_changes_nothing():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    dev = torch.device("cuda:0")
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev)
    op.forward_backward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"])
    ref = (op.loss.clone(), op.dhidden.clone(), op.dweight.clone())
    st = B.kdkl_profile_single_pass(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"], op.workspace, op.loss,
                                    op.dhidden, op.dweight, chunk=cfg.chunk, temperature=cfg.tau)
    chunks = cfg.T // cfg.chunk
    assert st["fwd_gemm_lse_exp"][1] == chunks and st["combine"][1] == chunks
    assert st["scale_and_patch"][1] == chunks                # per chunk: row scales + scaled hidden rows, support patch
    assert st["dhidden_gemm"][1] == chunks and st["dweight_gemm"][1] == (chunks + 1) // 2
    assert st["prep"][1] == 1 and st["loss_reduce"][1] == 1 and "bwd_coef" not in st
    assert all(ms > 0 for ms, n in st.values())
    assert torch.equal(op.loss, ref[0]) and torch.equal(op.dhidden, ref[1]) and torch.equal(op.dweight, ref[2])


def _random_case(T, H, V, K, seed, dev):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16).to(dev)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16).to(dev)
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32).to(dev)
    val = torch.randn(T, K, generator=g).float().to(dev)
    return h, W, idx, val


def test_count_tokens_and_device_side_divisor():
    """kdkl_count_tokens counts on the device; a divisor handed over through kdkl_options.denom_device gives bit
    for bit what the same number gives through denom_override (the data-parallel wrapper relies on this)."""
    dev = torch.device("cuda:0")
    T, H, V, K = 700, 72, 1001, 7
    h, W, idx, val = _random_case(T, H, V, K, 3, dev)
    mask = (torch.rand(T, generator=torch.Generator().manual_seed(4)) >= 0.3).to(torch.uint8).to(dev)
    n = torch.full((1,), -1.0, dtype=torch.float64, device=dev)
    B.kdkl_count_tokens(mask, T, n)
    assert n.item() == float(mask.sum().item())
    B.kdkl_count_tokens(None, T, n)
    assert n.item() == float(T)
    n.fill_(1234.0)
    for single_pass in (False, True):
        a = B.FusedChunkedKL(T, H, V, K, chunk=256, device=dev, opt=B.make_options(denom_override=1234.0))
        b = B.FusedChunkedKL(T, H, V, K, chunk=256, device=dev, opt=B.make_options(denom_device=n))
        for op in (a, b):
            if single_pass:
                op.forward_backward(h, W, idx, val, loss_mask=mask)
            else:
                op.forward(h, W, idx, val, loss_mask=mask)
                op.backward(h, W, loss_mask=mask)
            assert op.status()[0] == 0
        assert torch.equal(a.loss, b.loss) and torch.equal(a.dhidden, b.dhidden) and torch.equal(a.dweight, b.dweight)


def test_backward_refuses_a_state_it_cannot_use():
    """Device-side state check of kdkl_backward: another temperature or chunk size than the forward call's, and a
    second backward on stored exponentials (the in-place conversion can run once). Reported as KDKL_ERR_STATE,
    outputs untouched."""
    dev = torch.device("cuda:0")
    T, H, V, K = 300, 72, 1001, 7
    h, W, idx, val = _random_case(T, H, V, K, 5, dev)
    op = B.FusedChunkedKL(T, H, V, K, chunk=128, temperature=1.0, device=dev)
    op.forward(h, W, idx, val)
    op.dhidden.fill_(7.0); op.dweight.fill_(7.0)
    B.kdkl_backward(h, W, K, op.workspace, op.dhidden, op.dweight, chunk=128, temperature=1.5)
    assert op.status()[0] == -9
    assert (op.dhidden.float() == 7.0).all() and (op.dweight == 7.0).all()
    op.forward(h, W, idx, val)
    B.kdkl_backward(h, W, K, op.workspace, op.dhidden, op.dweight, chunk=64, temperature=1.0)
    assert op.status()[0] == -9
    assert (op.dhidden.float() == 7.0).all() and (op.dweight == 7.0).all()
    op.forward(h, W, idx, val)
    op.backward(h, W)                                         # the matching call goes through
    assert op.status()[0] == 0 and torch.isfinite(op.dweight).all()

    st = B.FusedChunkedKL(T, H, V, K, chunk=0, device=dev, opt=B.make_options(stored_exponentials=1))
    st.forward(h, W, idx, val)
    st.backward(h, W)
    assert st.status()[0] == 0
    first = (st.dhidden.clone(), st.dweight.clone())
    assert torch.allclose(first[1], op.dweight, rtol=0, atol=2e-2 * op.dweight.abs().max().item())
    st.dhidden.fill_(7.0); st.dweight.fill_(7.0)
    st.backward(h, W)                                         # the exponentials are gone: refused
    assert st.status()[0] == -9
    assert (st.dhidden.float() == 7.0).all() and (st.dweight == 7.0).all()
    # a forward without the option followed by a backward with it is refused as well
    plain = B.FusedChunkedKL(T, H, V, K, chunk=0, device=dev)
    plain.forward(h, W, idx, val)
    plain.dweight.fill_(7.0)
    B.kdkl_backward(h, W, K, plain.workspace, plain.dhidden, plain.dweight, opt=B.make_options(stored_exponentials=1))
    assert plain.status()[0] == -9 and (plain.dweight == 7.0).all()


def test_stored_exponentials_report_rows_below_their_range():
    """Every logit of a row at -64: the fixed-bias bf16 exponentials of the single-pass step would flush to zero
    there. The single-pass call says so (KDKL_ERR_RANGE); the two-call path has no such limit."""
    dev = torch.device("cuda:0")
    T, H, V, K = 40, 64, 600, 4
    h = torch.ones(T, H, dtype=torch.bfloat16, device=dev)
    W = -torch.ones(V, H, dtype=torch.bfloat16, device=dev)
    idx = torch.arange(K, dtype=torch.int32, device=dev).repeat(T, 1).contiguous()
    val = torch.zeros(T, K, device=dev)
    op = B.FusedChunkedKL(T, H, V, K, device=dev)
    op.forward(h, W, idx, val)
    op.backward(h, W)
    assert op.status()[0] == 0 and torch.isfinite(op.dweight).all()
    op.forward_backward(h, W, idx, val)
    assert op.status()[0] == -13


def test_tensor_on_another_device_than_the_current_one_is_refused(monkeypatch):
    """The library launches on the current device: a tensor that lives elsewhere must be refused by the binding
    before its address reaches a kernel (shown with one GPU by making the current device look like another)."""
    t = torch.zeros(8, device="cuda:0")
    assert B._dptr(t).value == t.data_ptr()
    monkeypatch.setattr(torch.cuda, "current_device", lambda: 1)
    with pytest.raises(TypeError):
        B._dptr(t)
