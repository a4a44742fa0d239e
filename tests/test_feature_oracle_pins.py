"""Pins for the feature-loss oracle: torch float64 library losses with autograd, finite differences, closed forms."""
import numpy as np
import torch
import torch.nn.functional as F

from oracle.feature_oracle import KIND_COSINE, KIND_MSE, feature_loss_oracle


def _data(T=19, H=24, seed=0):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((T, H)), rng.standard_normal((T, H)) * 1.7 + 0.3


def test_mse_matches_torch_mse_loss_and_autograd():
    s, r = _data()
    o = feature_loss_oracle(s, r, KIND_MSE, weight=0.7, grad_loss=1.3)
    st = torch.tensor(s, requires_grad=True)
    loss = 0.7 * F.mse_loss(st, torch.tensor(r))                 # mean over T*H = mean over tokens of the row means
    (1.3 * loss).backward()
    assert abs(o["loss"] - loss.item()) < 1e-13 * abs(loss.item())
    np.testing.assert_allclose(o["dS"], st.grad.numpy(), rtol=1e-12, atol=1e-15)


def test_cosine_matches_torch_cosine_embedding_loss_and_autograd():
    s, r = _data(seed=1)
    o = feature_loss_oracle(s, r, KIND_COSINE, weight=2.0)
    st = torch.tensor(s, requires_grad=True)
    loss = 2.0 * F.cosine_embedding_loss(st, torch.tensor(r), torch.ones(s.shape[0], dtype=torch.float64))
    loss.backward()
    assert abs(o["loss"] - loss.item()) < 1e-12 * abs(loss.item())
    np.testing.assert_allclose(o["dS"], st.grad.numpy(), rtol=1e-9, atol=1e-13)


def test_masked_mean_matches_torch_on_the_kept_rows():
    s, r = _data(T=31, seed=2)
    mask = (np.arange(31) % 3 != 0).astype(np.uint8)
    s_bad, r_bad = s.copy(), r.copy()
    s_bad[mask == 0] = np.nan                                    # ignored rows must never reach the arithmetic
    r_bad[mask == 0] = np.inf
    keep = mask != 0
    for kind in (KIND_MSE, KIND_COSINE):
        with np.errstate(all="ignore"):
            o = feature_loss_oracle(s_bad, r_bad, kind, mask=mask)
        st = torch.tensor(s[keep], requires_grad=True)
        rt = torch.tensor(r[keep])
        loss = F.mse_loss(st, rt) if kind == KIND_MSE else (1 - F.cosine_similarity(st, rt, dim=1)).mean()
        loss.backward()
        assert o["N"] == keep.sum()
        assert abs(o["loss"] - loss.item()) < 1e-12
        np.testing.assert_allclose(o["dS"][keep], st.grad.numpy(), rtol=1e-9, atol=1e-13)
        assert not o["dS"][~keep].any() and not o["loss_tok"][~keep].any()


def test_finite_differences_every_element():
    s, r = _data(T=4, H=5, seed=3)
    mask = np.array([1, 0, 1, 1], dtype=np.uint8)
    for kind in (KIND_MSE, KIND_COSINE):
        o = feature_loss_oracle(s, r, kind, mask=mask, weight=0.9, grad_loss=1.0)
        eps = 1e-6
        for t in range(4):
            for h in range(5):
                sp, sm = s.copy(), s.copy()
                sp[t, h] += eps; sm[t, h] -= eps
                fd = (feature_loss_oracle(sp, r, kind, mask=mask, weight=0.9, want_grads=False)["loss"]
                      - feature_loss_oracle(sm, r, kind, mask=mask, weight=0.9, want_grads=False)["loss"]) / (2 * eps)
                assert abs(fd - o["dS"][t, h]) <= 1e-7 * max(1.0, abs(fd)) + 1e-9


def test_closed_forms():
    H = 8
    e0 = np.zeros(H); e0[0] = 1
    e1 = np.zeros(H); e1[1] = 1
    s = np.stack([3 * e0, 3 * e0, 3 * e0, 2 * e0 + 2 * e1])
    r = np.stack([3 * e0, -5 * e0, 7 * e1, 4 * e0])
    o = feature_loss_oracle(s, r, KIND_COSINE)
    np.testing.assert_allclose(o["loss_tok"], [0.0, 2.0, 1.0, 1 - 1 / np.sqrt(2)], atol=1e-15)
    assert not o["dS"][0].any() and not o["dS"][1].any()         # parallel and antiparallel rows are stationary
    np.testing.assert_allclose(o["dS"][2], -(1 / 4) * e1 / 3, atol=1e-16)   # -g r/(|s||r|), g = 1/N
    m = feature_loss_oracle(s, r, KIND_MSE)
    np.testing.assert_allclose(m["loss_tok"], [0.0, 64 / H, (9 + 49) / H, (4 + 4) / H], atol=1e-15)
    np.testing.assert_allclose(m["dS"][1], (1 / 4) * (2 / H) * 8 * e0, atol=1e-16)
    assert abs(m["loss"] - (64 + 58 + 8) / H / 4) < 1e-15


def test_cosine_invariants():
    s, r = _data(T=9, H=16, seed=4)
    o = feature_loss_oracle(s, r, KIND_COSINE)
    o2 = feature_loss_oracle(3.5 * s, 0.25 * r, KIND_COSINE)
    np.testing.assert_allclose(o2["loss_tok"], o["loss_tok"], rtol=1e-13)             # positive scaling changes nothing
    np.testing.assert_allclose(o2["dS"], o["dS"] / 3.5, rtol=1e-12)                    # ... and the gradient scales by 1/a
    np.testing.assert_allclose((o["dS"] * s).sum(1), 0, atol=1e-15)                    # gradient is tangent to the sphere
    assert (o["loss_tok"] >= 0).all() and (o["loss_tok"] <= 2).all()


def test_degenerate_rows_and_empty_mask():
    s, r = _data(T=3, H=8, seed=5)
    s[1] = 0
    o = feature_loss_oracle(s, r, KIND_COSINE)
    assert o["loss_tok"][1] == 1.0 and not o["dS"][1].any() and np.isfinite(o["dS"]).all()
    for kind in (KIND_MSE, KIND_COSINE):
        z = feature_loss_oracle(s, r, kind, mask=np.zeros(3, dtype=np.uint8))
        assert z["loss"] == 0.0 and not z["dS"].any()


def test_denominator_override_splits_a_batch():
    s, r = _data(T=12, H=8, seed=6)
    for kind in (KIND_MSE, KIND_COSINE):
        whole = feature_loss_oracle(s, r, kind)
        a = feature_loss_oracle(s[:5], r[:5], kind, denom=12)
        b = feature_loss_oracle(s[5:], r[5:], kind, denom=12)
        assert abs(a["loss"] + b["loss"] - whole["loss"]) < 1e-14
        np.testing.assert_allclose(np.concatenate([a["dS"], b["dS"]]), whole["dS"], rtol=1e-13, atol=1e-18)
