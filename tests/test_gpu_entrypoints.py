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
    assert st["dhidden_gemm"][1] == chunks and st["dweight_gemm"][1] == chunks and st["combine"][1] == chunks
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
    assert st["fwd_gemm_lse_exp"][1] == chunks and st["exp_to_dlogits"][1] == chunks and st["combine"][1] == chunks
    assert st["dhidden_gemm"][1] == chunks and st["dweight_gemm"][1] == chunks
    assert st["prep"][1] == 1 and st["loss_reduce"][1] == 1 and "bwd_coef" not in st
    assert all(ms > 0 for ms, n in st.values())
    assert torch.equal(op.loss, ref[0]) and torch.equal(op.dhidden, ref[1]) and torch.equal(op.dweight, ref[2])
