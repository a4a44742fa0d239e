"""The torch.autograd entry: loss.backward() through the fused kernels against the oracle."""
import numpy as np
import pytest
import torch

from oracle.feature_oracle import KIND_COSINE, feature_loss_oracle
from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import inputs as I
from paper_2608_03796_b200.autograd import feature_loss, fused_chunked_kl

pytestmark = pytest.mark.gpu


def _fro(a, b):
    return np.linalg.norm(a - b) / np.linalg.norm(b)


def test_loss_backward_matches_oracle_and_combines_with_the_feature_loss():
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    r = I.teacher_hidden(cfg, device=dev)
    h = d["hidden"].clone().requires_grad_(True)
    W = d["weight"].clone().requires_grad_(True)
    kl = fused_chunked_kl(h, W, d["topk_idx"], d["topk_val"], chunk=cfg.chunk, temperature=cfg.tau)
    ft = feature_loss(h, r, kind=KIND_COSINE, weight=0.3)
    total = 2.0 * kl + ft                                 # upstream gradients 2 and 1
    total.backward()
    hn, Wn = d["hidden"].cpu().double().numpy(), d["weight"].cpu().double().numpy()
    ok = kdkl_oracle(hn, Wn, d["topk_idx"].cpu().numpy(), d["topk_val"].cpu().numpy(), tau=cfg.tau, grad_loss=2.0)
    of = feature_loss_oracle(hn, r.cpu().double().numpy(), KIND_COSINE, weight=0.3)
    want = 2.0 * ok["loss"] + of["loss"]
    assert abs(total.item() - want) <= 1e-3 * abs(want)
    assert h.grad.dtype == torch.bfloat16 and W.grad.dtype == torch.bfloat16
    assert _fro(h.grad.float().cpu().double().numpy(), ok["dH"] + of["dS"]) <= 1e-2
    assert _fro(W.grad.float().cpu().double().numpy(), ok["dW"]) <= 1e-2


def test_main_grad_accumulation_and_second_step_reuses_buffers():
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    main_grad = torch.zeros(cfg.V, cfg.H, dtype=torch.float32, device=dev)
    o = kdkl_oracle(d["hidden"].cpu().double().numpy(), d["weight"].cpu().double().numpy(),
                    d["topk_idx"].cpu().numpy(), d["topk_val"].cpu().numpy(), tau=cfg.tau)
    before = None
    for step in range(2):
        h = d["hidden"].clone().requires_grad_(True)
        W = d["weight"].clone().requires_grad_(True)
        loss = fused_chunked_kl(h, W, d["topk_idx"], d["topk_val"], chunk=cfg.chunk, temperature=cfg.tau,
                                dweight_out=main_grad)
        loss.backward()
        assert W.grad is None                               # dW went into main_grad instead
        assert abs(loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
        if step == 0:
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() <= before + 2 * d["hidden"].numel() * 2 + 4096   # no new workspace
    assert _fro(main_grad.cpu().double().numpy(), 2.0 * o["dW"]) <= 1e-2                  # two steps accumulated


def test_single_pass_autograd_matches_oracle():
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    o = kdkl_oracle(d["hidden"].cpu().double().numpy(), d["weight"].cpu().double().numpy(),
                    d["topk_idx"].cpu().numpy(), d["topk_val"].cpu().numpy(), tau=cfg.tau)
    for scale, expected in ((1.0, 1.0), (3.0, 1.0), (0.25, 0.25)):   # (3.0, 1.0) takes the recompute path in backward
        h = d["hidden"].clone().requires_grad_(True)
        W = d["weight"].clone().requires_grad_(True)
        loss = fused_chunked_kl(h, W, d["topk_idx"], d["topk_val"], chunk=cfg.chunk, temperature=cfg.tau,
                                single_pass=True, expected_grad=expected)
        (scale * loss).backward()
        assert abs(loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
        assert _fro(h.grad.float().cpu().double().numpy(), scale * o["dH"]) <= 1e-2
        assert _fro(W.grad.float().cpu().double().numpy(), scale * o["dW"]) <= 1e-2


def test_two_live_losses_of_one_shape_do_not_share_state():
    """loss1 + loss2 with the same shapes, one backward: each forward must own its saved state (prepared teacher,
    log Z, retained mass) until its backward has run. Compared with the oracle on each batch."""
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d1 = I.make_inputs(cfg, device=dev)
    d2 = I.make_inputs(I.Config("c1b", T=cfg.T, H=cfg.H, V=cfg.V, K=cfg.K, chunk=cfg.chunk, tok_offset=False,
                                seed=cfg.seed + 7), device=dev)
    W = d1["weight"].clone().requires_grad_(True)
    for single_pass in (False, True):
        W.grad = None
        h1 = d1["hidden"].clone().requires_grad_(True)
        h2 = d2["hidden"].clone().requires_grad_(True)
        l1 = fused_chunked_kl(h1, W, d1["topk_idx"], d1["topk_val"], chunk=cfg.chunk, single_pass=single_pass)
        l2 = fused_chunked_kl(h2, W, d2["topk_idx"], d2["topk_val"], chunk=cfg.chunk, single_pass=single_pass)
        (l1 + l2).backward()
        Wn = d1["weight"].cpu().double().numpy()
        o1 = kdkl_oracle(d1["hidden"].cpu().double().numpy(), Wn, d1["topk_idx"].cpu().numpy(),
                         d1["topk_val"].cpu().numpy(), tau=cfg.tau)
        o2 = kdkl_oracle(d2["hidden"].cpu().double().numpy(), Wn, d2["topk_idx"].cpu().numpy(),
                         d2["topk_val"].cpu().numpy(), tau=cfg.tau)
        assert abs(l1.item() - o1["loss"]) <= 1e-3 * abs(o1["loss"]) and abs(l2.item() - o2["loss"]) <= 1e-3 * abs(o2["loss"])
        assert _fro(h1.grad.float().cpu().double().numpy(), o1["dH"]) <= 1e-2
        assert _fro(h2.grad.float().cpu().double().numpy(), o2["dH"]) <= 1e-2
        assert _fro(W.grad.float().cpu().double().numpy(), o1["dW"] + o2["dW"]) <= 1e-2


def test_backward_keeps_the_upstream_gradient_on_the_device_and_does_not_wait():
    """The two-call path with a negative upstream gradient (-0.5 * loss): the value reaches the kernels through
    kdkl_options.grad_loss_device, its sign through the workspace header. With torch's synchronisation check set to
    raise, a whole step (forward, backward, the status probe) must not contain a blocking call."""
    from paper_2608_03796_b200 import autograd as A
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    o = kdkl_oracle(d["hidden"].cpu().double().numpy(), d["weight"].cpu().double().numpy(),
                    d["topk_idx"].cpu().numpy(), d["topk_val"].cpu().numpy(), tau=cfg.tau, grad_loss=-0.5)
    r = I.teacher_hidden(cfg, device=dev)
    of = feature_loss_oracle(d["hidden"].cpu().double().numpy(), r.cpu().double().numpy(), KIND_COSINE, weight=0.3)
    for step in range(2):                                   # the second step reuses pooled buffers and collects the probe
        h = d["hidden"].clone().requires_grad_(True)
        W = d["weight"].clone().requires_grad_(True)
        scale = torch.full((), -0.5, device=dev)
        torch.cuda.set_sync_debug_mode("error")
        try:
            loss = fused_chunked_kl(h, W, d["topk_idx"], d["topk_val"], chunk=cfg.chunk, temperature=cfg.tau)
            total = scale * loss + 2.0 * feature_loss(h, r, kind=KIND_COSINE, weight=0.3)   # the recommended pair
            total.backward()
        finally:
            torch.cuda.set_sync_debug_mode("default")
        assert _fro(h.grad.float().cpu().double().numpy(), o["dH"] + 2.0 * of["dS"]) <= 1e-2
        assert _fro(W.grad.float().cpu().double().numpy(), o["dW"]) <= 1e-2
    A.check_status()


def test_a_failed_step_is_reported_when_its_status_is_collected():
    """Deferred status: the header of the workspace is wiped between forward and backward, so backward finds no
    saved state (KDKL_ERR_STATE) and writes nothing. loss.backward() itself does not wait and does not raise;
    check_status() - or the next step on the same buffers - does. With sync_status=True backward raises at once."""
    from paper_2608_03796_b200 import autograd as A
    from paper_2608_03796_b200 import binding as B
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    A.clear_cache()
    for sync in (False, True):
        h = d["hidden"].clone().requires_grad_(True)
        W = d["weight"].clone().requires_grad_(True)
        loss = fused_chunked_kl(h, W, d["topk_idx"], d["topk_val"], chunk=cfg.chunk, temperature=cfg.tau,
                                sync_status=sync)
        loss.grad_fn.op.workspace[:64].zero_()
        if sync:
            with pytest.raises(B.KdklError) as e:
                loss.backward()
        else:
            loss.backward()
            with pytest.raises(B.KdklError) as e:
                A.check_status()
            A.check_status()                                # reported once
        assert e.value.code == -9
    A.clear_cache()


def test_device_side_upstream_gradient_equals_the_by_value_argument_bitwise():
    from paper_2608_03796_b200 import binding as B
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev,
                          opt=B.make_options(dhidden_dtype=1))
    for g in (1.0, -0.75, 3.0):
        op.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
        op.backward(d["hidden"], d["weight"], grad_loss=g)
        want = (op.dhidden.clone(), op.dweight.clone())
        op.dhidden.fill_(float("nan")); op.dweight.fill_(float("nan"))
        op.backward(d["hidden"], d["weight"], grad_loss=torch.full((1,), g, device=dev))
        assert op.status()[0] == 0
        assert torch.equal(op.dhidden, want[0]) and torch.equal(op.dweight, want[1])
        op.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], grad_loss=g)
        want = (op.dhidden.clone(), op.dweight.clone())
        op.dhidden.fill_(float("nan")); op.dweight.fill_(float("nan"))
        op.forward_backward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"],
                            grad_loss=torch.full((), g, device=dev))
        assert op.status()[0] == 0
        assert torch.equal(op.dhidden, want[0]) and torch.equal(op.dweight, want[1])
