"""GPU edge cases: degenerate and extreme shapes against the oracle, and the bounded-wait expiry path."""
import numpy as np
import pytest
import torch

from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import binding as B

pytestmark = pytest.mark.gpu


def _case(T, H, V, K, seed):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32)
    val = (torch.randn(T, K, generator=g) * 3 ** 0.5).float()
    return h, W, idx.contiguous(), val.contiguous()


def _fro(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


@pytest.mark.parametrize("T,H,V,K,chunk,tau", [
    (1, 8, 9, 1, 0, 1.0),            # a single token, the smallest legal hidden size
    (3, 8, 9, 9, 1, 0.5),            # K = V, one token per chunk
    (130, 72, 1001, 17, 37, 1.0),    # odd vocabulary (not a multiple of 8), odd chunk
    (40, 64, 255, 5, 0, 2.0),        # vocabulary smaller than one tile
    (20, 64, 1500, 1024, 0, 1.0),    # the largest supported K
    (257, 4104, 520, 3, 256, 1.0),   # hidden size with a ragged last k-block, rows one past a pair tile
])
def test_extreme_shapes_match_oracle(T, H, V, K, chunk, tau):
    dev = torch.device("cuda:0")
    h, W, idx, val = _case(T, H, V, K, seed=T * 7 + V)
    op = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=tau, device=dev, want_gathered=True,
                          want_per_token=True)
    op.dhidden.fill_(float("nan")); op.dweight.fill_(float("nan"))
    op.forward(h.to(dev), W.to(dev), idx.to(dev), val.to(dev))
    op.backward(h.to(dev), W.to(dev))
    assert op.status()[0] == 0
    o = kdkl_oracle(h.double().numpy(), W.double().numpy(), idx.numpy(), val.numpy(), tau=tau)
    assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"]) + 1e-6
    np.testing.assert_allclose(op.loss_per_token.cpu().double().numpy(), o["loss_tok"], rtol=0, atol=3e-4)
    assert np.array_equal(op.gathered_idx.cpu().numpy(), idx.numpy())
    np.testing.assert_allclose(op.gathered_logits.cpu().double().numpy(), o["gathered_logits"], rtol=0, atol=2e-4)
    dH = op.dhidden.float().cpu().double().numpy()
    dW = op.dweight.cpu().double().numpy()
    assert np.isfinite(dH).all() and np.isfinite(dW).all()
    assert _fro(dH, o["dH"]) <= 1e-2 and _fro(dW, o["dW"]) <= 1e-2


def test_bounded_wait_expires_and_context_survives():
    """A wait that nothing satisfies gives up after its limit, reports KDKL_ERR_TIMEOUT and the site,
    the kernel returns, and the same context runs the loss correctly afterwards."""
    dev = torch.device("cuda:0")
    st = torch.zeros(2, dtype=torch.int32, device=dev)
    B.kdkl_wait_selftest(st, 50_000_000)          # 50 ms
    torch.cuda.synchronize()
    assert st.tolist() == [-8, 99]
    h, W, idx, val = _case(64, 64, 512, 4, seed=3)
    op = B.FusedChunkedKL(64, 64, 512, 4, device=dev)
    op.forward(h.to(dev), W.to(dev), idx.to(dev), val.to(dev))
    assert op.status()[0] == 0
    o = kdkl_oracle(h.double().numpy(), W.double().numpy(), idx.numpy(), val.numpy(), want_grads=False)
    assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])


def test_large_logits_and_small_temperature():
    """Logits of standard deviation ~12 after the temperature (softmax close to one-hot on many rows):
    the online max / sum-exp must neither overflow nor lose the loss to cancellation."""
    dev = torch.device("cuda:0")
    T, H, V, K, tau = 200, 128, 5000, 12, 0.5
    h, W, idx, val = _case(T, H, V, K, seed=77)
    h = (h.float() * 6).to(torch.bfloat16)
    val = val * 4
    op = B.FusedChunkedKL(T, H, V, K, chunk=64, temperature=tau, device=dev, want_per_token=True)
    op.forward(h.to(dev), W.to(dev), idx.to(dev), val.to(dev))
    op.backward(h.to(dev), W.to(dev))
    assert op.status()[0] == 0
    o = kdkl_oracle(h.double().numpy(), W.double().numpy(), idx.numpy(), val.numpy(), tau=tau)
    assert o["logZ"].max() > 30
    assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
    np.testing.assert_allclose(op.loss_per_token.cpu().double().numpy(), o["loss_tok"], rtol=1e-4, atol=1e-3)
    assert _fro(op.dhidden.float().cpu().double().numpy(), o["dH"]) <= 1e-2
    assert _fro(op.dweight.cpu().double().numpy(), o["dW"]) <= 1e-2
