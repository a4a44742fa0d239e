"""Host-side logic of the vocabulary-sharded wrapper under real collectives: two gloo ranks on CPU.

The CUDA entry points are replaced inside each worker by small torch float64 stand-ins with the same
argument contract (local statistics [2, T]; finish from the gathered [R, 2, T]; partial dhidden), so the
test exercises what the wrapper adds: shard bookkeeping, the all-gather between the two forward phases
and the sum of dhidden after backward. The result is compared with the dense oracle.
"""
import math
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

LOG2E = 1.0 / math.log(2.0)


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _install_stand_ins(B, state):
    def ws_bytes(T, H, V, K, chunk=0, opt=None):
        return 64

    def fwd_shard(hidden, w_local, idx, val, ws, stats, *, vocab_offset, V_total, teacher_lse=None, loss_mask=None,
                  chunk=0, temperature=1.0, opt=None, gathered_logits=None, gathered_idx=None):
        z = hidden.double() @ w_local.double().T / temperature
        stats[0] = (torch.logsumexp(z, 1) * LOG2E).float()
        p = torch.softmax(val.double() / temperature, 1)
        local = (idx >= vocab_offset) & (idx < vocab_offset + w_local.shape[0])
        zl = torch.gather(z, 1, (idx.long() - vocab_offset).clamp(0, w_local.shape[0] - 1))
        stats[1] = (p * zl * local).sum(1).float()
        state.update(p=p, idx=idx, z=z, v0=vocab_offset, tau=temperature,
                     Hent=(p * torch.log(p)).sum(1), M=p.sum(1))

    def fwd_finish(all_stats, R, T, H, V_local, K, ws, loss_out, *, loss_mask=None, chunk=0, temperature=1.0,
                   opt=None, loss_per_token=None):
        lz = torch.logsumexp(all_stats[:, 0].double() / LOG2E, 0)
        L = state["Hent"] - all_stats[:, 1].double().sum(0) + state["M"] * lz
        state["logZ"] = lz
        loss_out[0] = L.mean().float()
        if loss_per_token is not None:
            loss_per_token.copy_(L.float())

    def bwd(hidden, w_local, K, ws, dh, dw, *, loss_mask=None, chunk=0, temperature=1.0, opt=None, grad_loss=1.0):
        T = hidden.shape[0]
        q = torch.exp(state["z"] - state["logZ"][:, None])
        G = state["M"][:, None] * q
        local = (state["idx"] >= state["v0"]) & (state["idx"] < state["v0"] + w_local.shape[0])
        li = (state["idx"].long() - state["v0"]).clamp(0, w_local.shape[0] - 1)
        G.scatter_add_(1, li, -(state["p"] * local))
        G *= grad_loss / T / state["tau"]
        dh.copy_((G @ w_local.double()).float())
        dw.copy_((G.T @ hidden.double()).float())

    B.kdkl_workspace_bytes, B.kdkl_forward_shard, B.kdkl_forward_finish, B.kdkl_backward = ws_bytes, fwd_shard, fwd_finish, bwd


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_03796_b200 import binding as B
    state = {}
    _install_stand_ins(B, state)
    T, H, V, K = 12, 8, 30, 4
    g = torch.Generator().manual_seed(5)
    h = torch.randn(T, H, generator=g)
    W = torch.randn(V, H, generator=g) / H ** 0.5
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32)
    val = torch.randn(T, K, generator=g)
    bounds = [0, 13, V]
    v0, v1 = bounds[rank], bounds[rank + 1]
    op = B.ShardedFusedChunkedKL(T, H, v1 - v0, v0, V, K, world, device="cpu", want_per_token=True)
    loss = op.forward(h, W[v0:v1].contiguous(), idx, val)
    dh, dw = op.backward(h, W[v0:v1].contiguous())
    out.put((rank, float(loss.item()), dh.numpy().copy(), dw.numpy().copy(), h.numpy(), W.numpy(), idx.numpy(), val.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_vocab_shards_over_gloo_match_the_oracle():
    from oracle.kdkl_oracle import kdkl_oracle
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=90) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    _, loss0, dh0, dw0, h, W, idx, val = res[0]
    _, loss1, dh1, dw1 = res[1][:4]
    o = kdkl_oracle(h, W, idx, val)
    assert loss0 == loss1                                       # every rank ends with the same loss
    assert abs(loss0 - o["loss"]) < 1e-5
    np.testing.assert_allclose(dh0, dh1, rtol=0, atol=0)        # all-reduced dhidden is identical on both ranks
    np.testing.assert_allclose(dh0, o["dH"], rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(np.concatenate([dw0, dw1], 0), o["dW"], rtol=1e-4, atol=1e-6)
