"""Pins for the fp64 oracle against things other than itself.

Each test names what fixes the expected value: a library routine (torch float64
kl_div / cross_entropy with autograd), a closed form, finite differences, a
pure-Python brute force, or an invariant of the mathematics. The paper prints no
worked numeric example for this loss, so there are no golden values from it.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle.kdkl_oracle import kdkl_oracle, teacher_probs


def _rand_case(T, H, V, K, seed, distinct=True):
    rng = np.random.default_rng(seed)
    h = rng.standard_normal((T, H))
    W = rng.standard_normal((V, H)) / math.sqrt(H)
    if distinct:
        idx = np.stack([rng.choice(V, size=K, replace=False) for _ in range(T)]).astype(np.int32)
    else:
        idx = rng.integers(0, V, size=(T, K)).astype(np.int32)
    val = rng.standard_normal((T, K)) * math.sqrt(3.0)
    return h, W, idx, val


def _torch_ref(h, W, idx, val, tau, mask=None, lse=None, grad_loss=1.0):
    """torch float64: Eq. "kl" via F.kl_div on a scattered dense teacher, autograd for grads."""
    ht = torch.tensor(h, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    T, V = h.shape[0], W.shape[0]
    l = torch.tensor(val, dtype=torch.float64) / tau
    lam = torch.logsumexp(l, dim=1) if lse is None else torch.tensor(lse, dtype=torch.float64)
    pk = torch.exp(l - lam[:, None])
    p = torch.zeros(T, V, dtype=torch.float64)
    p.scatter_add_(1, torch.tensor(idx, dtype=torch.int64), pk)
    logq = F.log_softmax(ht @ Wt.T / tau, dim=1)
    per_tok = F.kl_div(logq, p, reduction="none").sum(1)
    m = torch.ones(T, dtype=torch.float64) if mask is None else torch.tensor(mask, dtype=torch.float64)
    loss = (per_tok * m).sum() / m.sum()
    (loss * grad_loss).backward()
    return loss.item(), per_tok.detach().numpy() * m.numpy(), ht.grad.numpy(), Wt.grad.numpy()


@pytest.mark.parametrize("tau", [1.0, 2.0, 0.7])
def test_matches_torch_kl_div_and_autograd(tau):
    h, W, idx, val = _rand_case(37, 24, 211, 7, seed=1)
    mask = (np.arange(37) % 5 != 0).astype(np.uint8)
    o = kdkl_oracle(h, W, idx, val, tau=tau, mask=mask, grad_loss=1.7)
    loss, per_tok, dH, dW = _torch_ref(h, W, idx, val, tau, mask, grad_loss=1.7)
    assert abs(o["loss"] - loss) <= 1e-12 * abs(loss)
    np.testing.assert_allclose(o["loss_tok"], per_tok, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(o["dH"], dH, rtol=1e-9, atol=1e-13)
    np.testing.assert_allclose(o["dW"], dW, rtol=1e-9, atol=1e-13)
    assert np.all(o["dH"][mask == 0] == 0.0)


def test_duplicates_scatter_add_matches_torch():
    h, W, idx, val = _rand_case(9, 8, 13, 6, seed=2, distinct=False)
    idx[0, :] = 3                                   # a row that is all one index
    o = kdkl_oracle(h, W, idx, val)
    loss, per_tok, dH, dW = _torch_ref(h, W, idx, val, 1.0)
    np.testing.assert_allclose(o["loss_tok"], per_tok, rtol=1e-10)
    np.testing.assert_allclose(o["dW"], dW, rtol=1e-9, atol=1e-13)
    np.testing.assert_allclose(o["dH"], dH, rtol=1e-9, atol=1e-13)


def test_partial_mass_matches_torch_and_is_not_renormalised():
    h, W, idx, val = _rand_case(21, 16, 97, 5, seed=3)
    rng = np.random.default_rng(30)
    mass = rng.uniform(0.6, 1.0, size=21)
    lse = np.log(np.exp(val / 1.0).sum(1)) - np.log(mass)
    o = kdkl_oracle(h, W, idx, val, teacher_lse=lse)
    np.testing.assert_allclose(o["M"], mass, rtol=1e-12)
    loss, per_tok, dH, dW = _torch_ref(h, W, idx, val, 1.0, lse=lse)
    np.testing.assert_allclose(o["loss_tok"], per_tok, rtol=1e-10)
    np.testing.assert_allclose(o["dH"], dH, rtol=1e-9, atol=1e-13)
    np.testing.assert_allclose(o["dW"], dW, rtol=1e-9, atol=1e-13)
    # log-probability mode (values already log p) is the same thing
    o1 = kdkl_oracle(h, W, idx, val - lse[:, None], teacher_mode=1)
    np.testing.assert_allclose(o1["loss_tok"], o["loss_tok"], rtol=1e-12)
    np.testing.assert_allclose(o1["dW"], o["dW"], rtol=1e-10, atol=1e-15)


def test_k1_is_cross_entropy():
    h, W, idx, val = _rand_case(19, 12, 53, 1, seed=4)
    o = kdkl_oracle(h, W, idx, val)
    ht = torch.tensor(h, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    ce = F.cross_entropy(ht @ Wt.T, torch.tensor(idx[:, 0], dtype=torch.int64), reduction="none")
    ce.mean().backward()
    np.testing.assert_allclose(o["loss_tok"], ce.detach().numpy(), rtol=1e-12)
    np.testing.assert_allclose(o["dH"], ht.grad.numpy(), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(o["dW"], Wt.grad.numpy(), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(o["gathered_logits"][:, 0],
                               (ht @ Wt.T).detach().numpy()[np.arange(19), idx[:, 0]], rtol=1e-12)


def test_closed_form_zero_weight():
    T, H, V, K, tau = 6, 5, 31, 4, 1.3
    h, _, idx, val = _rand_case(T, H, V, K, seed=5)
    W = np.zeros((V, H))
    rng = np.random.default_rng(50)
    mass = rng.uniform(0.5, 1.0, size=T)
    lse = np.log(np.exp(val / tau).sum(1)) - np.log(mass)
    o = kdkl_oracle(h, W, idx, val, tau=tau, teacher_lse=lse, grad_loss=2.0)
    p = np.exp(val / tau - lse[:, None])
    expect = (p * np.log(p)).sum(1) + mass * math.log(V)
    np.testing.assert_allclose(o["loss_tok"], expect, rtol=1e-12)
    np.testing.assert_allclose(o["logZ"], math.log(V), rtol=1e-14)
    assert np.all(o["dH"] == 0.0)
    # dW[v,:] = sum_t (g/tau) (M/V - p_tv) h_t
    g = 2.0 / T
    dz = np.tile((mass / V)[:, None], (1, V))
    for t in range(T):
        for k in range(K):
            dz[t, idx[t, k]] -= p[t, k]
    np.testing.assert_allclose(o["dW"], (g / tau) * dz.T @ h, rtol=1e-11, atol=1e-15)


def test_zero_point_teacher_equals_student():
    T, H, V = 5, 7, 23
    h, W, _, _ = _rand_case(T, H, V, 1, seed=6)
    rng = np.random.default_rng(60)
    idx = np.stack([rng.permutation(V) for _ in range(T)]).astype(np.int32)
    z = h @ W.T
    val = np.take_along_axis(z, idx.astype(np.int64), axis=1)
    o = kdkl_oracle(h, W, idx, val, tau=1.0)
    assert abs(o["loss"]) < 1e-12
    assert np.abs(o["loss_tok"]).max() < 1e-12
    assert np.abs(o["dH"]).max() < 1e-12 and np.abs(o["dW"]).max() < 1e-12


def test_finite_differences_every_element():
    T, H, V, K, tau = 5, 6, 17, 4, 1.5
    h, W, idx, val = _rand_case(T, H, V, K, seed=7)
    mask = np.array([1, 1, 0, 1, 1], dtype=np.uint8)
    lse = np.log(np.exp(val / tau).sum(1)) + 0.2
    kw = dict(tau=tau, mask=mask, teacher_lse=lse)
    o = kdkl_oracle(h, W, idx, val, **kw)
    eps = 1e-6

    def f(hh, ww):
        return kdkl_oracle(hh, ww, idx, val, want_grads=False, **kw)["loss"]
    for arr, grad, which in ((h, o["dH"], 0), (W, o["dW"], 1)):
        num = np.zeros_like(arr)
        for i in range(arr.shape[0]):
            for j in range(arr.shape[1]):
                a1 = arr.copy(); a1[i, j] += eps
                a0 = arr.copy(); a0[i, j] -= eps
                num[i, j] = ((f(a1, W) - f(a0, W)) if which == 0 else (f(h, a1) - f(h, a0))) / (2 * eps)
        np.testing.assert_allclose(grad, num, rtol=1e-6, atol=1e-9)


def test_brute_force_python_loops():
    """Eq. "kl", Eq. "grad" and Algorithm 1's two products as explicit scalar loops."""
    T, H, V, K, tau = 3, 4, 9, 3, 0.8
    h, W, idx, val = _rand_case(T, H, V, K, seed=8, distinct=False)
    idx[1, 2] = -1                                   # an empty slot
    mask = [1, 1, 1]
    o = kdkl_oracle(h, W, idx, val, tau=tau, grad_loss=1.0)
    N = 3
    dH = [[0.0] * H for _ in range(T)]
    dW = [[0.0] * H for _ in range(V)]
    tot = 0.0
    for t in range(T):
        z = [sum(h[t][j] * W[v][j] for j in range(H)) for v in range(V)]
        s = [zz / tau for zz in z]
        mx = max(s)
        logZ = mx + math.log(sum(math.exp(x - mx) for x in s))
        ks = [k for k in range(K) if idx[t][k] >= 0]
        lam = math.log(sum(math.exp(val[t][k] / tau) for k in ks))
        p = [0.0] * V
        for k in ks:
            p[idx[t][k]] += math.exp(val[t][k] / tau - lam)
        M = sum(p)
        L = sum(p[v] * (math.log(p[v]) - (s[v] - logZ)) for v in range(V) if p[v] > 0)
        assert abs(L - o["loss_tok"][t]) < 1e-12
        for k in range(K):
            if idx[t][k] >= 0:
                assert abs(o["gathered_logits"][t][k] - z[idx[t][k]]) < 1e-13
            else:
                assert math.isnan(o["gathered_logits"][t][k])
        tot += L
        for v in range(V):
            dz = (1.0 / N / tau) * (M * math.exp(s[v] - logZ) - p[v])
            for j in range(H):
                dH[t][j] += dz * W[v][j]
                dW[v][j] += dz * h[t][j]
    assert abs(tot / N - o["loss"]) < 1e-12
    np.testing.assert_allclose(o["dH"], np.array(dH), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(o["dW"], np.array(dW), rtol=1e-10, atol=1e-14)


def test_bounds_and_invariants():
    T, H, V, K = 40, 16, 301, 9
    h, W, idx, val = _rand_case(T, H, V, K, seed=9)
    o = kdkl_oracle(h, W, idx, val)
    assert np.all(o["loss_tok"] >= -1e-12)                       # KL >= 0 when M = 1
    np.testing.assert_allclose(o["M"], 1.0, rtol=1e-12)
    assert np.abs(o["dW"].sum(axis=0)).max() < 1e-12             # sum_v dz = (g/tau)(M - M) = 0
    assert np.all(o["logZ"] >= (h @ W.T).max(1) - 1e-12)
    # partial mass: L >= M log M >= -1/e (log-sum inequality), can be negative
    rng = np.random.default_rng(90)
    mass = rng.uniform(0.3, 1.0, size=T)
    lse = np.log(np.exp(val).sum(1)) - np.log(mass)
    o2 = kdkl_oracle(h, W, idx, val, teacher_lse=lse)
    assert np.all(o2["loss_tok"] >= mass * np.log(mass) - 1e-12)
    assert np.abs(o2["dW"].sum(axis=0)).max() < 1e-12
    # adding a per-token constant to teacher values changes nothing (mode 0, no lse)
    o3 = kdkl_oracle(h, W, idx, val + rng.standard_normal((T, 1)))
    np.testing.assert_allclose(o3["loss_tok"], o["loss_tok"], rtol=1e-10, atol=1e-12)
    # permuting the K slots of each row changes nothing but the echo order
    perm = rng.permutation(K)
    o4 = kdkl_oracle(h, W, idx[:, perm], val[:, perm])
    np.testing.assert_allclose(o4["loss_tok"], o["loss_tok"], rtol=1e-12)
    np.testing.assert_allclose(o4["dW"], o["dW"], rtol=1e-10, atol=1e-15)
    np.testing.assert_allclose(o4["gathered_logits"], o["gathered_logits"][:, perm], rtol=0)
    # row blocking (memory bounding only) changes nothing beyond summation order of dW
    o5 = kdkl_oracle(h, W, idx, val, row_block=7)
    np.testing.assert_allclose(o5["loss_tok"], o["loss_tok"], rtol=1e-13)
    np.testing.assert_allclose(o5["dH"], o["dH"], rtol=1e-12, atol=1e-16)
    np.testing.assert_allclose(o5["dW"], o["dW"], rtol=1e-10, atol=1e-15)


def test_masked_rows_never_read_and_bad_indices():
    T, H, V, K = 12, 8, 50, 4
    h, W, idx, val = _rand_case(T, H, V, K, seed=10)
    mask = np.ones(T, dtype=np.uint8); mask[[2, 7]] = 0
    ref = kdkl_oracle(h, W, idx, val, mask=mask)
    idx2, val2 = idx.copy(), val.copy()
    idx2[[2, 7]] = -1; val2[[2, 7]] = np.nan
    o = kdkl_oracle(h, W, idx2, val2, mask=mask)
    assert o["loss"] == ref["loss"] and np.array_equal(o["dW"], ref["dW"])
    assert np.all(o["loss_tok"][[2, 7]] == 0) and np.all(o["dH"][[2, 7]] == 0)
    # all tokens ignored: loss 0, zero gradients
    z = kdkl_oracle(h, W, idx, val, mask=np.zeros(T, dtype=np.uint8))
    assert z["loss"] == 0.0 and not z["dW"].any() and not z["dH"].any()
    # an index >= V is dropped and counted
    idx3 = idx.copy(); idx3[0, 1] = V + 3
    o3 = kdkl_oracle(h, W, idx3, val)
    assert o3["n_bad_idx"] == 1
    idx4 = idx.copy(); idx4[0, 1] = -1
    np.testing.assert_allclose(o3["loss_tok"], kdkl_oracle(h, W, idx4, val)["loss_tok"], rtol=1e-13)


def test_teacher_probs_modes():
    val = np.array([[0.3, -1.0, 2.0]])
    p = teacher_probs(val, 2.0)
    e = np.exp(val / 2.0)
    np.testing.assert_allclose(p, e / e.sum(), rtol=1e-14)
    p = teacher_probs(val, 1.0, teacher_lse=np.array([3.0]))
    np.testing.assert_allclose(p, np.exp(val - 3.0), rtol=1e-14)
    p = teacher_probs(np.log(np.array([[0.5, 0.2, 0.1]])), 1.0, teacher_mode=1)
    np.testing.assert_allclose(p, [[0.5, 0.2, 0.1]], rtol=1e-14)
    with pytest.raises(ValueError):
        teacher_probs(val, 2.0, teacher_mode=1)


def test_statistical_sanity_on_config_generators():
    """With the benchmark generators z ~ N(0,1): logZ ~ log V + 1/2 (a gross-error alarm only)."""
    from paper_2608_03796_b200 import inputs as I
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    o = kdkl_oracle(d["hidden"].double().numpy(), d["weight"].double().numpy(),
                    d["topk_idx"].numpy(), d["topk_val"].numpy(), tau=cfg.tau, want_grads=False)
    assert abs(o["logZ"].mean() - (math.log(cfg.V) + 0.5)) < 0.1
    assert 5.0 < o["loss"] < 9.0


@pytest.mark.parametrize("seed", list(range(40)))
def test_random_configurations_match_torch_autograd(seed):
    """Seeded random shapes and options (temperature, masks, duplicates, partial mass, upstream gradient) against the
    torch float64 library expression with autograd: any dropped term, wrong sign or transposed operand that only
    shows for some combination of options fails here."""
    r = np.random.default_rng(1000 + seed)
    T, H, V = int(r.integers(1, 40)), int(r.integers(1, 30)), int(r.integers(2, 150))
    K = int(r.integers(1, min(V, 12) + 1))
    tau = float(r.choice([0.5, 1.0, 1.0, 2.5]))
    h, W, idx, val = _rand_case(T, H, V, K, seed=seed, distinct=bool(r.random() < 0.6))
    mask = (r.random(T) > 0.3).astype(np.uint8) if r.random() < 0.6 else None
    if mask is not None and mask.sum() == 0:
        mask[0] = 1
    lse = None
    if r.random() < 0.5:
        l = val / tau
        lse = np.log(np.exp(l - l.max(1, keepdims=True)).sum(1)) + l.max(1) + r.random(T) * 0.7      # mass < 1
    gl = float(r.choice([1.0, -0.5, 2.0]))
    o = kdkl_oracle(h, W, idx, val, tau=tau, mask=mask, teacher_lse=lse, grad_loss=gl)
    loss, per_tok, dH, dW = _torch_ref(h, W, idx, val, tau, mask, lse=lse, grad_loss=gl)
    assert abs(o["loss"] - loss) <= 1e-11 * max(1.0, abs(loss))
    np.testing.assert_allclose(o["loss_tok"], per_tok, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(o["dH"], dH, rtol=1e-8, atol=1e-12)
    np.testing.assert_allclose(o["dW"], dW, rtol=1e-8, atol=1e-12)
