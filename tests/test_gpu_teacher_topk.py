"""GPU parity of the teacher top-K cache kernel against its dense fp64 oracle.

The selection is decided by fp32 logits on the GPU and fp64 logits in the oracle, so two entries whose
logits differ by less than the fp32 accumulation error may swap places or membership at the K-th
boundary. What is unique is compared exactly (entries clearly above the boundary, sorted values,
the log-sum-exp); the rest is checked for validity (every returned index is a genuine near-top entry).
"""
import numpy as np
import pytest
import torch

from oracle.kdkl_oracle import kdkl_oracle
from oracle.teacher_oracle import teacher_topk_oracle
from paper_2608_03796_b200 import binding as B

pytestmark = pytest.mark.gpu
EPS = 2e-4          # fp32 accumulation error bound on a logit of magnitude O(10)


def _case(T, H, V, seed):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    return h, W


def _check(h, W, K, tau, stored=False, exact_floor=0.98):
    dev = torch.device("cuda:0")
    idx, val, lse, ws = B.kdkl_teacher_topk(h.to(dev), W.to(dev), K, temperature=tau, stored=stored)
    code, _ = B.kdkl_status(ws)
    assert code == 0
    idx, val, lse = idx.cpu().numpy(), val.cpu().double().numpy(), lse.cpu().double().numpy()
    o = teacher_topk_oracle(h.double().numpy(), W.double().numpy(), K, tau=tau)
    np.testing.assert_allclose(lse, o["lse"], rtol=0, atol=2e-4)
    T, V = o["z"].shape
    assert idx.min() >= 0 and idx.max() < V
    for t in range(T):
        assert len(set(idx[t].tolist())) == K                             # K distinct entries
        zt = o["z"][t]
        np.testing.assert_allclose(val[t], zt[idx[t]], rtol=0, atol=EPS)   # values are the logits at those indices
        assert np.all(np.diff(val[t]) <= 0)                                # sorted descending
        kth = o["val"][t, -1]
        assert np.all(zt[idx[t]] >= kth - EPS)                             # nothing below the boundary got in
        sure = o["idx"][t][o["val"][t] > kth + EPS]                        # entries clearly above it must be there
        assert set(sure.tolist()) <= set(idx[t].tolist())
    exact = (idx == o["idx"]).mean()
    assert exact >= exact_floor                                            # position-exact except at near-ties
    return idx, val, lse, o


@pytest.mark.parametrize("stored", [False, True])
@pytest.mark.parametrize("T,H,V,K,tau", [(300, 264, 4120, 16, 1.0), (70, 64, 300, 100, 2.0), (5, 8, 9, 9, 1.0),
                                         (1100, 128, 70000, 100, 1.0), (4200, 64, 4099, 8, 1.0)])
def test_teacher_topk_matches_oracle(T, H, V, K, tau, stored):
    """Both forms: two projections, and one projection with the fp32 logits of each pass kept in the workspace.
    The last shape spans two 4096-token passes with a vocabulary that is not a multiple of 4."""
    h, W = _case(T, H, V, seed=T + V)
    _check(h, W, K, tau, stored)


def test_stored_form_gives_the_same_record_bit_for_bit():
    """Same logits, same threshold, same selection: the two forms must agree exactly."""
    dev = torch.device("cuda:0")
    h, W = _case(700, 136, 9000, seed=11)
    a = B.kdkl_teacher_topk(h.to(dev), W.to(dev), 32, temperature=1.3)
    b = B.kdkl_teacher_topk(h.to(dev), W.to(dev), 32, temperature=1.3, stored=True)
    assert B.kdkl_status(a[3])[0] == 0 and B.kdkl_status(b[3])[0] == 0
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])


def test_ties_break_by_smaller_index_and_overflow_is_reported():
    dev = torch.device("cuda:0")
    T, H, V, K = 4, 64, 2048, 8
    h, W = _case(T, H, V, seed=9)
    W[100] = W[7]; W[1500] = W[7]                     # three identical vocabulary rows: exact ties
    idx, val, lse, ws = B.kdkl_teacher_topk(h.to(dev), W.to(dev), 256, temperature=1.0)
    assert B.kdkl_status(ws)[0] == 0
    idx, val = idx.cpu().numpy(), val.cpu().numpy()
    for t in range(T):
        pos = {int(v): int(np.where(idx[t] == v)[0][0]) for v in (7, 100, 1500) if v in idx[t]}
        if len(pos) == 3:
            assert pos[7] < pos[100] < pos[1500] and val[t][pos[7]] == val[t][pos[1500]]
    # a constant head: every logit ties, more candidates than the list can hold -> reported
    Wc = torch.ones(4096, H).to(torch.bfloat16)       # 16 tiles >= K = 8: threshold path, list of 256
    _, _, _, ws2 = B.kdkl_teacher_topk(h.to(dev), Wc.to(dev), 8, temperature=1.0)
    assert B.kdkl_status(ws2)[0] == -12


@pytest.mark.parametrize("stored", [False, True])
def test_large_logits_clustered_in_a_few_tiles(stored):
    """A frequency-ordered vocabulary: the first 3000 entries carry systematically larger logits, so thousands of
    logits reach the K-th largest tile maximum and the first candidate list (max(4K, 256) slots) overflows. The
    kernel tightens the threshold on the device and scans again; the record must still be the exact top-K."""
    T, H, V, K = 300, 64, 40000, 32
    g = torch.Generator().manual_seed(77)
    u = torch.randn(H, generator=g)
    u = u / u.norm()
    h = (torch.randn(T, H, generator=g) * 0.5 + 4.0 * u).to(torch.bfloat16)
    W = torch.randn(V, H, generator=g) / H ** 0.5
    W[:3000] += 1.5 * u * torch.rand(3000, 1, generator=g)          # logits of the head entries shifted up by ~0..6
    W = W.to(torch.bfloat16)
    z = h.double() @ W.double().T
    thr = torch.topk(z.view(T, -1, 250).amax(-1), K, dim=1).values[:, -1]   # roughly the tile-maxima threshold
    assert ((z >= thr[:, None]).sum(1) > 4 * max(4 * K, 256)).any()           # far more than the first list holds
    _check(h, W, K, 1.0, stored)


@pytest.mark.parametrize("stored", [False, True])
def test_vocabulary_with_fewer_tiles_than_k(stored):
    """V = 20000 is 79 tiles of 256 columns, fewer than K = 128: the tile maxima give no threshold, every logit is a
    candidate, and the record comes out of the tightening rounds alone (20000 -> about 5000 -> 1250 -> 310)."""
    h, W = _case(260, 64, 20000, seed=91)
    _check(h, W, 128, 1.0, stored)


@pytest.mark.parametrize("T,H,V,K", [(48, 64, 1 << 20, 256),      # the largest vocabulary and K the call takes
                                     (130, 64, 65000, 256)])       # 254 tiles < K: 65000 -> 16250 -> 4062 -> 1015
def test_limits_of_vocabulary_and_k(T, H, V, K):
    h, W = _case(T, H, V, seed=V % 1000 + K)
    _check(h, W, K, 1.0, False)


def _draw(seed):
    """A seeded random configuration: shape, K, temperature, and one of four logit structures - plain Gaussian, a
    head of systematically larger logits (overflowing lists), a confident teacher (one direction dominates), groups
    of identical vocabulary rows (exact ties, also at the K-th boundary)."""
    r = np.random.default_rng(seed)
    T = int(r.choice([1, 3, 37, 130, 300]))
    H = int(r.choice([8, 24, 64, 136, 256]))
    V = int(r.choice([r.integers(1, 300), r.integers(300, 9000), r.integers(9000, 70000)]))
    K = int(min(V, r.choice([1, 2, 7, 16, 50, 100, 128, 256])))
    tau = float(r.choice([1.0, 1.0, 0.7, 2.0]))
    kind = int(r.integers(0, 4))
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(T, H, generator=g)
    W = torch.randn(V, H, generator=g) / H ** 0.5
    if kind == 1:
        u = torch.randn(H, generator=g); u = u / u.norm()
        h = h * 0.5 + 4.0 * u
        n = min(V, int(r.integers(200, 4000)))
        W[:n] += 1.5 * u * torch.rand(n, 1, generator=g)
    elif kind == 2:
        W = W * 4.0
    elif kind == 3 and V >= 8:
        src = torch.randint(0, V, (max(V // 8, 1),), generator=g)
        dst = torch.randint(0, V, (len(src),), generator=g)
        W[dst] = W[src]
    return h.to(torch.bfloat16), W.to(torch.bfloat16), K, tau, bool(r.integers(0, 2))


@pytest.mark.parametrize("seed", range(2000, 2040))
def test_random_configuration(seed):
    h, W, K, tau, stored = _draw(seed)
    _check(h, W, K, tau, stored, exact_floor=0.0 if W.shape[0] < 4 * K else 0.9)


def test_cache_feeds_the_loss_with_exact_retained_mass():
    """Teacher kernel -> cache record -> fused loss with teacher_lse: the paper's un-renormalised M < 1 path,
    end to end on the GPU, against the oracles fed with their own (fp64) cache."""
    dev = torch.device("cuda:0")
    T, Ht, Hs, V, K, tau = 200, 96, 128, 3000, 20, 1.0
    ht, Wt = _case(T, Ht, V, seed=41)
    hs, Ws = _case(T, Hs, V, seed=42)
    idx, val, lse, _ = B.kdkl_teacher_topk(ht.to(dev), Wt.to(dev), K, temperature=tau)
    op = B.FusedChunkedKL(T, Hs, V, K, chunk=64, temperature=tau, device=dev)
    op.forward(hs.to(dev), Ws.to(dev), idx, val, teacher_lse=lse)
    op.backward(hs.to(dev), Ws.to(dev))
    assert op.status()[0] == 0
    ot = teacher_topk_oracle(ht.double().numpy(), Wt.double().numpy(), K, tau=tau)
    o = kdkl_oracle(hs.double().numpy(), Ws.double().numpy(), ot["idx"], ot["val"], tau=tau, teacher_lse=ot["lse"])
    assert o["M"].max() < 1.0
    assert abs(op.loss.item() - o["loss"]) <= 1e-3 * abs(o["loss"])
    dW = op.dweight.cpu().double().numpy()
    assert np.linalg.norm(dW - o["dW"]) / np.linalg.norm(o["dW"]) <= 1e-2


def test_fullsize_sampled_rows():
    """The benchmark shape (T=4096, H=4096, V=131072, K=100): the dense oracle on 24 sampled rows
    (rows are independent given the head), with the same unique / valid split as above."""
    from paper_2608_03796_b200 import inputs as I
    dev = torch.device("cuda:0")
    cfg = I.CONFIGS["c2"]
    h = I.hidden(cfg, device=dev)
    W = I.weight(cfg, device=dev)
    idx, val, lse, ws = B.kdkl_teacher_topk(h, W, cfg.K, temperature=1.0)
    assert B.kdkl_status(ws)[0] == 0
    del ws
    sidx, sval, slse, sws = B.kdkl_teacher_topk(h, W, cfg.K, temperature=1.0, stored=True)   # one projection
    assert B.kdkl_status(sws)[0] == 0
    assert torch.equal(sidx, idx) and torch.equal(sval, val) and torch.equal(slse, lse)
    del sws, sidx, sval, slse
    R = I.sample_rows(cfg, 24).to(dev)
    o = teacher_topk_oracle(h[R].cpu().double().numpy(), W.cpu().double().numpy(), cfg.K, tau=1.0)
    gi, gv = idx[R].cpu().numpy(), val[R].cpu().double().numpy()
    np.testing.assert_allclose(lse[R].cpu().double().numpy(), o["lse"], rtol=0, atol=2e-4)
    exact = 0
    for r in range(len(R)):
        zt = o["z"][r]
        assert len(set(gi[r].tolist())) == cfg.K and gi[r].min() >= 0 and gi[r].max() < cfg.V
        np.testing.assert_allclose(gv[r], zt[gi[r]], rtol=0, atol=EPS)
        assert np.all(np.diff(gv[r]) <= 0)
        kth = o["val"][r, -1]
        assert np.all(zt[gi[r]] >= kth - EPS)
        sure = o["idx"][r][o["val"][r] > kth + EPS]
        assert set(sure.tolist()) <= set(gi[r].tolist())
        exact += int((gi[r] == o["idx"][r]).sum())
    assert exact > 0.98 * len(R) * cfg.K
    # whole-run properties: every row sorted, distinct, in range; retained mass below one
    assert bool((val[:, 1:] <= val[:, :-1]).all())
    assert int(idx.min()) >= 0 and int(idx.max()) < cfg.V
    srt = idx.sort(dim=1).values
    assert bool((srt[:, 1:] != srt[:, :-1]).all())
    mass = torch.exp(val.double() - lse.double()[:, None]).sum(1)
    assert bool((mass > 0).all()) and bool((mass < 1).all())
