"""The two comparison losses (dense KL; forward-chunked sparse KL) against the fp64 oracle.

bench.py reports the fused path's iteration rate and peak memory next to these two programs, as the paper's
loss-only benchmark does (section "Isolating Loss-Kernel Scaling"); this test makes them verified programs.
They compute in bf16 / fp32 with library GEMMs, so the tolerances are the ones stated for the fused path:
loss relative 1e-3, dHidden / dWeight relative Frobenius 1e-2.
"""
import numpy as np
import pytest
import torch

from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import comparators as C
from paper_2608_03796_b200 import inputs as I


def _case(T, H, V, K, seed, tau, device):
    """A small ragged shape with a loss mask (poisoned teacher rows), empty slots and partial teacher mass."""
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32)
    val = (torch.randn(T, K, generator=g) * 3 ** 0.5).float()
    idx[torch.rand(T, K, generator=g) < 0.1] = -1
    mask = (torch.rand(T, generator=g) >= 0.15).to(torch.uint8)
    lse = torch.logsumexp(torch.where(idx >= 0, val, torch.full_like(val, -1e30)).double() / tau, 1).float() + 0.25
    idx, val = I.poison_masked(idx, val, mask)
    d = {"hidden": h, "weight": W, "topk_idx": idx.contiguous(), "topk_val": val.contiguous(), "mask": mask}
    return d, lse


def _check(method, device, partial):
    T, H, V, K, tau, chunk = 261, 72, 1001, 7, 1.3, 100
    d, lse = _case(T, H, V, K, seed=5, tau=tau, device=device)
    lse = lse if partial else None
    with np.errstate(all="ignore"):
        o = kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                        d["topk_val"].numpy(), tau=tau, mask=d["mask"].numpy(),
                        teacher_lse=None if lse is None else lse.double().numpy())
    if partial:
        assert o["M"][d["mask"].numpy() != 0].max() < 1.0
    g = {k: v.to(device) for k, v in d.items()}
    loss, dH, dW = C.run(method, g, tau, chunk, teacher_lse=None if lse is None else lse.to(device))
    fro = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    assert abs(loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
    dH, dW = dH.float().cpu().double().numpy(), dW.float().cpu().double().numpy()
    assert fro(dH, o["dH"]) <= 1e-2 and fro(dW, o["dW"]) <= 1e-2
    assert not dH[d["mask"].numpy() == 0].any()


@pytest.mark.parametrize("partial", [False, True])
@pytest.mark.parametrize("method", ["dense", "fwdchunk"])
def test_comparator_matches_oracle_cpu(method, partial):
    _check(method, torch.device("cpu"), partial)


@pytest.mark.gpu
@pytest.mark.parametrize("partial", [False, True])
@pytest.mark.parametrize("method", ["dense", "fwdchunk"])
def test_comparator_matches_oracle_gpu(method, partial):
    _check(method, torch.device("cuda:0"), partial)
