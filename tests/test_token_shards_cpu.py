"""Host-side logic of the token-sharded (data-parallel) wrapper under real collectives: two gloo ranks on CPU.

The CUDA entry points are replaced inside each worker by torch float64 stand-ins with the same argument contract,
so the test exercises what the wrapper adds: the count of counted tokens (the library's count call) summed over
ranks before forward and handed to the kernels as a device-side divisor, the sum of the partial losses, and the
sum of dweight; for the two-call form and for the
single-pass form. Uneven token slices, a mask on one rank only. Compared with the dense oracle over all tokens.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _install_stand_ins(B, state):
    def ws_bytes(T, H, V, K, chunk=0, opt=None):
        return 64

    def _loss_and_G(hidden, weight, idx, val, mask, tau, denom):
        z = hidden.double() @ weight.double().T / tau
        lz = torch.logsumexp(z, 1)
        p = torch.softmax(val.double() / tau, 1)
        m = torch.ones(hidden.shape[0], dtype=torch.float64) if mask is None else (mask != 0).double()
        L = (p * torch.log(p)).sum(1) - (p * torch.gather(z, 1, idx.long())).sum(1) + lz
        G = torch.exp(z - lz[:, None])
        G.scatter_add_(1, idx.long(), -p)
        return (L * m).sum() / denom, G * (m / denom / tau)[:, None]

    def fwd(hidden, weight, idx, val, ws, loss_out, *, teacher_lse=None, loss_mask=None, chunk=0, temperature=1.0,
            opt=None, loss_per_token=None, gathered_logits=None, gathered_idx=None):
        loss, G = _loss_and_G(hidden, weight, idx, val, loss_mask, temperature, float(opt.denom_device.item()))
        loss_out[0] = loss.float()
        state["G"] = G

    def bwd(hidden, weight, K, ws, dh, dw, *, loss_mask=None, chunk=0, temperature=1.0, opt=None, grad_loss=1.0):
        G = state["G"] * grad_loss
        dh.copy_((G @ weight.double()).to(dh.dtype))
        dw.copy_((G.T @ hidden.double()).float())

    def fwd_bwd(hidden, weight, idx, val, ws, loss_out, dh, dw, *, teacher_lse=None, loss_mask=None, chunk=0,
                temperature=1.0, opt=None, grad_loss=1.0, loss_per_token=None):
        fwd(hidden, weight, idx, val, ws, loss_out, loss_mask=loss_mask, temperature=temperature, opt=opt)
        bwd(hidden, weight, idx.shape[1], ws, dh, dw, grad_loss=grad_loss)

    def count(mask, T, out):
        out[0] = float(T if mask is None else int((mask != 0).sum()))

    def options(**kw):                                      # the wrapper passes the divisor as a tensor to read later
        import types
        return types.SimpleNamespace(**kw)

    B.kdkl_workspace_bytes, B.kdkl_forward, B.kdkl_backward, B.kdkl_forward_backward = ws_bytes, fwd, bwd, fwd_bwd
    B.kdkl_count_tokens, B.make_options = count, options


def _worker(rank, world, port, out, single_pass):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_03796_b200 import binding as B
    state = {}
    _install_stand_ins(B, state)
    T, H, V, K = 14, 8, 30, 4
    g = torch.Generator().manual_seed(9)
    h = torch.randn(T, H, generator=g)
    W = torch.randn(V, H, generator=g) / H ** 0.5
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32)
    val = torch.randn(T, K, generator=g)
    mask = torch.ones(T, dtype=torch.uint8)
    mask[1] = 0; mask[4] = 0                               # ignored tokens on rank 0's slice only
    bounds = [0, 5, T]                                     # uneven slices
    a, b = bounds[rank], bounds[rank + 1]
    op = B.TokenShardedFusedKL(b - a, H, V, K, device="cpu",
                               all_reduce_sum=lambda t: dist.all_reduce(t, op=dist.ReduceOp.SUM))
    op.dhidden = torch.empty(b - a, H, dtype=torch.float32)   # the stand-ins write fp32
    sl_mask = mask[a:b].contiguous() if rank == 0 else None  # rank 1 passes no mask: all its tokens count
    if single_pass:
        loss, dh, dw = op.forward_backward(h[a:b], W, idx[a:b], val[a:b], loss_mask=sl_mask)
    else:
        loss = op.forward(h[a:b], W, idx[a:b], val[a:b], loss_mask=sl_mask)
        dh, dw = op.backward(h[a:b], W, loss_mask=sl_mask)
    out.put((rank, float(loss.item()), dh.numpy().copy(), dw.numpy().copy(), h.numpy(), W.numpy(), idx.numpy(),
             val.numpy(), mask.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def _run(single_pass):
    from oracle.kdkl_oracle import kdkl_oracle
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q, single_pass)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=90) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    _, loss0, dh0, dw0, h, W, idx, val, mask = res[0]
    _, loss1, dh1, dw1 = res[1][:4]
    o = kdkl_oracle(h, W, idx, val, mask=mask)
    assert o["N"] == 12                                        # 14 tokens, two ignored: the divisor both ranks must use
    assert loss0 == loss1 and abs(loss0 - o["loss"]) < 1e-5    # summed partial means = the global mean, on every rank
    np.testing.assert_allclose(dw0, dw1, rtol=0, atol=0)       # all-reduced dweight is identical on both ranks
    np.testing.assert_allclose(dw0, o["dW"], rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(np.concatenate([dh0, dh1], 0), o["dH"], rtol=1e-4, atol=1e-6)


def test_two_token_shards_over_gloo_two_call():
    _run(False)


def test_two_token_shards_over_gloo_single_pass():
    _run(True)
