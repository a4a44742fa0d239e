"""The vocabulary-sharded variant (the paper's tensor-parallel configuration) on one GPU.

The ranks' kernels do not wait on one another, so the shards run one after the other on the same
device and the two collectives of Algorithm 1 (gather of the shard statistics, sum of dhidden) are
done with plain copies here. Everything is compared with the dense fp64 oracle over the FULL vocabulary.
"""
import numpy as np
import pytest
import torch

from oracle.kdkl_oracle import kdkl_oracle
from paper_2608_03796_b200 import binding as B
from paper_2608_03796_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _fro(a, b):
    return np.linalg.norm(a - b) / np.linalg.norm(b)


def _run_sharded(d, T, H, V, K, bounds, chunk, tau, lse=None, grad_loss=1.0, opt=None):
    dev = torch.device("cuda:0")
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    lse_d = None if lse is None else lse.to(dev)
    R = len(bounds) - 1
    ranks = []
    for r in range(R):
        v0, v1 = bounds[r], bounds[r + 1]
        ranks.append(B.ShardedFusedChunkedKL(T, H, v1 - v0, v0, V, K, R, chunk=chunk, temperature=tau, device=dev,
                                             want_per_token=True, opt=opt))
    W = [g["weight"][bounds[r]:bounds[r + 1]].contiguous() for r in range(R)]
    for r, op in enumerate(ranks):
        op.forward_local(g["hidden"], W[r], g["topk_idx"], g["topk_val"], teacher_lse=lse_d, loss_mask=g["mask"])
    stats = torch.stack([op.stats_local for op in ranks])            # what an all-gather delivers
    for op in ranks:
        op.stats_all.copy_(stats)
        op.forward_finish(loss_mask=g["mask"])
    for r, op in enumerate(ranks):
        op.backward_local(g["hidden"], W[r], loss_mask=g["mask"], grad_loss=grad_loss)
        assert op.status()[0] == 0
    dH = sum(op.dhidden for op in ranks)                              # what an all-reduce delivers
    dW = torch.cat([op.dweight for op in ranks], 0)
    return ranks, dH, dW


@pytest.mark.parametrize("bounds", [[0, 2048, 4120], [0, 1000, 2500, 4120]])
def test_sharded_matches_oracle_ragged(bounds):
    T, H, V, K, tau = 261, 264, 4120, 9, 1.3
    g = torch.Generator().manual_seed(31)
    d = {"hidden": torch.randn(T, H, generator=g).to(torch.bfloat16),
         "weight": (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16),
         "topk_idx": torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32),
         "topk_val": (torch.randn(T, K, generator=g) * 3 ** 0.5).float(),
         "mask": (torch.rand(T, generator=g) >= 0.1).to(torch.uint8)}
    d["topk_idx"][5, 2] = -1
    d["topk_idx"][7, :3] = 2047                          # duplicates right at a shard boundary
    lse = torch.logsumexp(d["topk_val"].double() / tau, 1).float() + 0.25      # retained mass < 1
    ranks, dH, dW = _run_sharded(d, T, H, V, K, bounds, 100, tau, lse=lse, grad_loss=0.7)
    o = kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                    d["topk_val"].numpy(), tau=tau, mask=d["mask"].numpy(), teacher_lse=lse.double().numpy(),
                    grad_loss=0.7)
    for op in ranks:                                      # every rank holds the same, complete loss
        assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
        np.testing.assert_allclose(op.loss_per_token.cpu().double().numpy(), o["loss_tok"], rtol=0, atol=2e-4)
    assert torch.equal(ranks[0].loss_per_token, ranks[-1].loss_per_token)
    assert _fro(dH.cpu().double().numpy(), o["dH"]) <= 1e-2
    assert _fro(dW.cpu().double().numpy(), o["dW"]) <= 1e-2
    assert not dH[d["mask"] == 0].abs().sum().item()


def test_sharded_c1_two_halves_equals_unsharded_loss():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    ranks, dH, dW = _run_sharded(d, cfg.T, cfg.H, cfg.V, cfg.K, [0, cfg.V // 2, cfg.V], cfg.chunk, cfg.tau)
    dev = torch.device("cuda:0")
    g = {k: (v.to(dev) if v is not None else None) for k, v in d.items()}
    full = B.FusedChunkedKL(cfg.T, cfg.H, cfg.V, cfg.K, chunk=cfg.chunk, temperature=cfg.tau, device=dev,
                            opt=B.make_options(dhidden_dtype=1), want_per_token=True)
    full.forward(g["hidden"], g["weight"], g["topk_idx"], g["topk_val"])
    full.backward(g["hidden"], g["weight"])
    assert abs(ranks[0].loss.item() - full.loss.item()) <= 1e-6 * abs(full.loss.item())
    assert (ranks[0].loss_per_token - full.loss_per_token).abs().max().item() < 2e-5
    # dW slices are computed from the same G values: only the rounding of log Z can differ
    assert _fro(dW.cpu().double().numpy(), full.dweight.cpu().double().numpy()) < 2e-3
    assert _fro(dH.cpu().double().numpy(), full.dhidden.cpu().double().numpy()) < 2e-3


@pytest.mark.parametrize("single_pass", [False, True])
def test_token_shards_match_oracle(single_pass):
    """Data-parallel form: uneven token slices, the global denominator on every rank, dW and loss summed."""
    T, H, V, K, tau = 300, 136, 2100, 7, 1.0
    g = torch.Generator().manual_seed(51)
    d = {"hidden": torch.randn(T, H, generator=g).to(torch.bfloat16),
         "weight": (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16),
         "topk_idx": torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32),
         "topk_val": (torch.randn(T, K, generator=g) * 3 ** 0.5).float(),
         "mask": (torch.rand(T, generator=g) >= 0.2).to(torch.uint8)}
    dev = torch.device("cuda:0")
    gd = {k: v.to(dev) for k, v in d.items()}
    bounds = [0, 77, 200, T]
    # the ranks run one after the other here, so the "all-reduce" of the count is a running sum over a first
    # pass of the library's count kernel; each rank then reads the global divisor from the device
    ops, counts = [], []
    for r in range(3):
        a, b = bounds[r], bounds[r + 1]
        op = B.TokenShardedFusedKL(b - a, H, V, K, chunk=64, temperature=tau, device=dev, all_reduce_sum=lambda t: t)
        counts.append(op.count_tokens(gd["mask"][a:b].contiguous()).clone())
        ops.append(op)
    n_global = torch.stack(counts).sum(0)
    assert n_global.item() == float(d["mask"].sum().item())
    ranks = []
    for r in range(3):
        a, b = bounds[r], bounds[r + 1]
        op = ops[r]
        op.n_global.copy_(n_global)
        sl = {k: (v[a:b].contiguous() if k != "weight" else v) for k, v in gd.items()}
        if single_pass:
            op.forward_backward_local(sl["hidden"], sl["weight"], sl["topk_idx"], sl["topk_val"], loss_mask=sl["mask"])
        else:
            op.forward_local(sl["hidden"], sl["weight"], sl["topk_idx"], sl["topk_val"], loss_mask=sl["mask"])
            op.backward_local(sl["hidden"], sl["weight"], loss_mask=sl["mask"])
        assert op.status()[0] == 0
        ranks.append(op)
    loss = sum(op.loss.item() for op in ranks)                       # what the all-reduces deliver
    dW = sum(op.dweight for op in ranks)
    dH = torch.cat([op.dhidden for op in ranks], 0)
    o = kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                    d["topk_val"].numpy(), tau=tau, mask=d["mask"].numpy())
    assert abs(loss - o["loss"]) <= 1e-3 * abs(o["loss"])
    assert _fro(dW.cpu().double().numpy(), o["dW"]) <= 1e-2
    assert _fro(dH.float().cpu().double().numpy(), o["dH"]) <= 1e-2


@pytest.mark.parametrize("seed", list(range(2000, 2016)))
def test_random_shardings_match_oracle(seed):
    """Seeded random shapes, 2-4 shards at random (ragged, possibly tiny) boundaries, masks with dead
    runs, duplicates / empty slots, partial teacher mass: every rank's loss, the summed dHidden and the
    concatenated dWeight against the full-vocabulary oracle."""
    r = np.random.default_rng(seed)
    T = int(r.choice([5, 130, 300, 700]))
    H = 8 * int(r.integers(1, 30))
    K = int(r.choice([1, 4, 16, 40]))
    V = int(r.integers(max(4 * K, 64), 3000))
    R = int(r.integers(2, 5))
    cuts = sorted(int(x) for x in r.choice(np.arange(1, V), size=R - 1, replace=False))
    bounds = [0] + cuts + [V]
    tau = float(r.choice([0.7, 1.0, 2.0]))
    chunk = int(r.choice([0, 64, 100, 256]))
    g = torch.Generator().manual_seed(seed)
    idx = (torch.randint(0, V, (T, K), generator=g) if r.random() < 0.3
           else torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)])).to(torch.int32)
    if r.random() < 0.5:
        idx[torch.rand(T, K, generator=g) < 0.1] = -1
    mask = None
    if r.random() < 0.6:
        mask = (torch.rand(T, generator=g) >= 0.15).to(torch.uint8)
        if T >= 600:
            mask[100:100 + int(r.integers(256, 450))] = 0
    d = {"hidden": torch.randn(T, H, generator=g).to(torch.bfloat16),
         "weight": (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16),
         "topk_idx": idx.contiguous(), "topk_val": (torch.randn(T, K, generator=g) * 3 ** 0.5).float(), "mask": mask}
    lse = None
    if r.random() < 0.5:
        lse = torch.logsumexp(d["topk_val"].double() / tau, 1).float() + torch.rand(T, generator=g) * 0.4
    ranks, dH, dW = _run_sharded(d, T, H, V, K, bounds, chunk, tau, lse=lse)
    o = kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                    d["topk_val"].numpy(), tau=tau, mask=None if mask is None else mask.numpy(),
                    teacher_lse=None if lse is None else lse.double().numpy())
    for op in ranks:
        assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"]) + 1e-6
        np.testing.assert_allclose(op.loss_per_token.cpu().double().numpy(), o["loss_tok"], rtol=0, atol=2e-4)
        assert torch.equal(op.loss_per_token, ranks[0].loss_per_token)      # identical bits on every rank
    assert _fro(dH.cpu().double().numpy(), o["dH"]) <= 1e-2
    assert _fro(dW.cpu().double().numpy(), o["dW"]) <= 1e-2
    if mask is not None:
        assert not dH[mask == 0].abs().sum().item()


def test_sharded_without_recompute_when_one_chunk_covers_the_tokens():
    """stored_exponentials with vocabulary shards: log Z is known only after the exchange, the exponentials wait in
    each rank's buffer, and the backward of every rank forms its G slice from them (three projections)."""
    T, H, V, K, tau = 300, 264, 4120, 9, 1.0
    g = torch.Generator().manual_seed(5)
    d = {"hidden": torch.randn(T, H, generator=g).to(torch.bfloat16),
         "weight": (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16),
         "topk_idx": torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32),
         "topk_val": (torch.randn(T, K, generator=g) * 3 ** 0.5).float(),
         "mask": (torch.rand(T, generator=g) >= 0.1).to(torch.uint8)}
    ranks, dH, dW = _run_sharded(d, T, H, V, K, [0, 1000, 2500, 4120], 0, tau,
                                 opt=B.make_options(stored_exponentials=1, dhidden_dtype=1))
    o = kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(), d["topk_idx"].numpy(),
                    d["topk_val"].numpy(), tau=tau, mask=d["mask"].numpy())
    for op in ranks:
        assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
    assert _fro(dH.cpu().double().numpy(), o["dH"]) <= 1e-2
    assert _fro(dW.cpu().double().numpy(), o["dW"]) <= 1e-2
