"""bench.py's sharded modes (--parallel tokens / vocab) on two gloo ranks on CPU.

The CUDA entry points are replaced by the float64 stand-ins of the two wrapper tests, so what runs here is what
bench.py adds around the wrappers: how a rank picks its tokens (rows [r*T, (r+1)*T) of one global batch) or its
vocabulary rows, the order of calls and collectives inside a step, repeated steps on the same buffers, and the
job-level bookkeeping (tokens per step, scaling kind). Results after two steps are compared with the dense oracle
over the whole batch.
"""
import dataclasses
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2608_03796_b200 import inputs as I

CFG = I.Config("tiny", T=14, H=8, V=30, K=4, chunk=8, tok_offset=False)


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close()
    return p


def _worker(rank, world, port, out, mode):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_03796_b200 import binding as B
    import test_token_shards_cpu as tok
    import test_vocab_shards_cpu as voc
    state = {}
    (tok if mode == "tokens" else voc)._install_stand_ins(B, state)
    run = bench.MODES[mode](CFG, rank, world, "cpu", B, I)
    op = run["op"]
    op.dhidden = torch.empty(CFG.T, CFG.H, dtype=torch.float32)      # the stand-ins write fp32
    for _ in range(2):                                                # a second step on the same buffers
        run["step"]()
    run["drain"]()
    out.put((rank, run["loss"](), op.dhidden.numpy().copy(), op.dweight.numpy().copy(), run["tokens_per_step"],
             run["scaling"], run["collective"]["bytes_per_step"]))
    dist.barrier()
    dist.destroy_process_group()


def _launch(mode):
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q, mode)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return res


def _oracle(cfg):
    from oracle.kdkl_oracle import kdkl_oracle
    d = I.make_inputs(cfg)
    return kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                       d["topk_val"].numpy(), tau=cfg.tau)


def test_token_sharded_mode_two_ranks():
    res = _launch("tokens")
    o = _oracle(dataclasses.replace(CFG, T=2 * CFG.T))                # the global batch both ranks cut their rows from
    (_, loss0, dh0, dw0, tps, scaling, nbytes), (_, loss1, dh1, dw1, *_rest) = res
    assert tps == 2 * CFG.T and scaling == "weak" and nbytes == CFG.V * CFG.H * 4 + 12
    assert loss0 == loss1 and abs(loss0 - o["loss"]) < 1e-5
    np.testing.assert_allclose(dw0, dw1, rtol=0, atol=0)
    np.testing.assert_allclose(dw0, o["dW"], rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(np.concatenate([dh0, dh1], 0), o["dH"], rtol=1e-4, atol=1e-6)


def test_vocab_sharded_mode_two_ranks():
    res = _launch("vocab")
    o = _oracle(CFG)
    (_, loss0, dh0, dw0, tps, scaling, _n), (_, loss1, dh1, dw1, *_rest) = res
    assert tps == CFG.T and scaling == "strong"
    assert loss0 == loss1 and abs(loss0 - o["loss"]) < 1e-5
    np.testing.assert_allclose(dh0, dh1, rtol=0, atol=0)
    np.testing.assert_allclose(dh0, o["dH"], rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(np.concatenate([dw0, dw1], 0), o["dW"], rtol=1e-4, atol=1e-6)
    assert bench.shard_bounds(30, 2, 0) == (0, 15) and bench.shard_bounds(31, 2, 1) == (16, 31)
