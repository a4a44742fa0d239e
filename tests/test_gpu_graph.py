"""kdkl_forward + kdkl_backward are enqueue-only, so a step can be captured once into a CUDA graph and
replayed on new data written into the same buffers."""
import pytest
import torch

from paper_2608_03796_b200 import binding as B
from paper_2608_03796_b200 import inputs as I

pytestmark = pytest.mark.gpu


def test_step_replays_from_a_cuda_graph():
    cfg = I.CONFIGS["c1"]
    dev = torch.device("cuda:0")
    d = {k: (v.to(dev) if v is not None else None) for k, v in I.make_inputs(cfg).items()}
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev)

    def step():
        op.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
        op.backward(d["hidden"], d["weight"])

    step()                                   # warm-up outside capture (driver entry points, attributes)
    torch.cuda.synchronize()
    ref_loss, ref_dw, ref_dh = op.loss.clone(), op.dweight.clone(), op.dhidden.clone()

    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)

    op.dweight.zero_(); op.dhidden.zero_(); op.loss.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert op.status()[0] == 0
    assert torch.equal(op.loss, ref_loss) and torch.equal(op.dweight, ref_dw) and torch.equal(op.dhidden, ref_dh)

    # new data in the same buffers: the replay follows it
    d2 = I.make_inputs(I.dataclasses.replace(cfg, seed=cfg.seed + 1))
    for k in ("hidden", "topk_idx", "topk_val"):
        d[k].copy_(d2[k].to(dev))
    graph.replay()
    torch.cuda.synchronize()
    replay_loss, replay_dw = op.loss.clone(), op.dweight.clone()
    step()
    torch.cuda.synchronize()
    assert torch.equal(op.loss, replay_loss) and torch.equal(op.dweight, replay_dw)
    assert replay_loss.item() != ref_loss.item()

    # latency: a replayed step launches nothing from the host
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    e0.record()
    for _ in range(20):
        step()
    e1.record()
    for _ in range(20):
        graph.replay()
    e2.record()
    torch.cuda.synchronize()
    print(f"c1 step: eager {e0.elapsed_time(e1) / 20:.3f} ms, graph replay {e1.elapsed_time(e2) / 20:.3f} ms")


def test_runs_on_a_side_stream_with_identical_bits():
    """Everything is enqueued on the caller's stream: a step issued on a non-default stream, with unrelated
    work on the default stream at the same time, gives the bits of a step on the default stream."""
    from paper_2608_03796_b200 import inputs as I
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg, device=dev)
    op = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev,
                          want_per_token=True)
    op.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
    op.backward(d["hidden"], d["weight"])
    torch.cuda.synchronize()
    ref = (op.loss.clone(), op.loss_per_token.clone(), op.dhidden.clone(), op.dweight.clone())
    for t in (op.loss, op.loss_per_token, op.dhidden, op.dweight):
        t.zero_()
    side = torch.cuda.Stream()
    noise = torch.randn(4096, 4096, device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        op.forward(d["hidden"], d["weight"], d["topk_idx"], d["topk_val"])
        op.backward(d["hidden"], d["weight"])
    for _ in range(4):
        noise = noise @ noise.T * 1e-4                    # keeps the default stream busy meanwhile
    side.synchronize()
    torch.cuda.synchronize()
    assert op.status()[0] == 0
    assert torch.equal(op.loss, ref[0]) and torch.equal(op.loss_per_token, ref[1])
    assert torch.equal(op.dhidden, ref[2]) and torch.equal(op.dweight, ref[3])
