"""The allocation-free entry point against the regular one (collected last on purpose).

kdkl_logz_noalloc is for callers that cannot allocate device memory at all (for instance a plugin
inside a server whose pool already owns the GPU): its scratch is a fixed array inside the library.
It must give the same log Z as kdkl_forward, which uses a caller-allocated workspace, on two calls
in a row that share that array - and both must agree with the fp64 oracle's log Z.
"""
import numpy as np
import pytest
import torch

from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import binding as B

pytestmark = pytest.mark.gpu


def _case(T, H, V, K, seed, dev):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16).to(dev)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16).to(dev)
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32).to(dev)
    val = torch.randn(T, K, generator=g).float().to(dev)
    return h, W, idx, val


def test_logz_noalloc_matches_forward_twice_in_a_row():
    dev = torch.device("cuda:0")
    # second case is larger than one internal pass and ragged in every dimension
    for (T, H, V, K, tau, seed) in [(300, 264, 4120, 5, 1.0, 1), (2500, 128, 3000, 3, 1.7, 2)]:
        h, W, idx, val = _case(T, H, V, K, seed, dev)
        op = B.FusedChunkedKL(T, H, V, K, temperature=tau, device=dev)
        op.forward(h, W, idx, val)
        assert op.status()[0] == 0
        ref, _ = op.saved_state()
        out = torch.full((T,), float("nan"), dtype=torch.float32, device=dev)
        before = torch.cuda.memory_allocated()
        B.kdkl_logz_noalloc(h, W, out, temperature=tau)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert torch.isfinite(out).all()
        assert (out - ref).abs().max().item() <= 2e-4
        o = kdkl_oracle(h.cpu().double().numpy(), W.cpu().double().numpy(), idx.cpu().numpy(), val.cpu().numpy(),
                        tau=tau, want_grads=False)
        np.testing.assert_allclose(out.cpu().double().numpy(), o["logZ"], rtol=0, atol=2e-4)


def test_logz_noalloc_rejects_oversized_vocabulary():
    dev = torch.device("cuda:0")
    h = torch.zeros(8, 64, dtype=torch.bfloat16, device=dev)
    W = torch.zeros(8, 64, dtype=torch.bfloat16, device=dev)
    out = torch.zeros(8, device=dev)
    # the size check comes before anything is read, so a small buffer is enough to ask for a large V
    rc = B.lib().kdkl_logz_noalloc(h.data_ptr(), W.data_ptr(), 8, 64, 262144 + 256, 1.0, out.data_ptr(), None)
    assert rc == -4
