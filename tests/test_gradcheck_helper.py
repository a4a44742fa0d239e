"""The gradient comparison helper must (a) accept what the CUDA path's arithmetic produces - fp32 contractions of a
G that was rounded once to bf16 - and (b) reject a defect confined to one row although the whole-matrix norm
does not see it. Checked here on synthetic matrices with the structure of Eq. "grad" (a dense softmax part plus
K large sparse teacher entries per token), on the CPU."""
import numpy as np
import pytest
import torch

from gradcheck import check_grad_matrix, check_support_rows


def _dlogits(T, V, K, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.softmax(torch.randn(T, V, generator=g, dtype=torch.float64), dim=-1)
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)])
    p = torch.softmax(torch.randn(T, K, generator=g, dtype=torch.float64) * 3 ** 0.5, dim=-1)
    sparse = torch.zeros(T, V, dtype=torch.float64).scatter_add_(1, idx, p)
    return q / T, sparse / T, idx


def _bf16(x):
    return x.to(torch.float32).to(torch.bfloat16).to(torch.float64)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_accepts_one_bf16_rounding_and_rejects_a_row_without_its_teacher_term(seed):
    T, V, H, K = 1300, 2000, 64, 8
    dense, sparse, idx = _dlogits(T, V, K, seed)
    g = torch.Generator().manual_seed(100 + seed)
    h = _bf16(torch.randn(T, H, generator=g))
    W = _bf16(torch.randn(V, H, generator=g) / H ** 0.5)
    G = dense - sparse
    ref_dW, ref_dH = (G.T @ h).numpy(), (G @ W).numpy()
    Gr = _bf16(G)
    got_dW, got_dH = (Gr.T @ h).numpy(), _bf16(Gr @ W).numpy()
    rel_w, ratio_w = check_grad_matrix(got_dW, ref_dW, "dW")
    rel_h, ratio_h = check_grad_matrix(got_dH, ref_dH, "dH", out_bf16=True)
    assert rel_w < 5e-3 and rel_h < 6e-3 and ratio_w < 0.8 and ratio_h < 0.8     # with room to spare
    check_support_rows(got_dW, ref_dW, idx.numpy(), [0, 7, T - 1], "dW")

    # the defect: token 7 loses its sparse teacher term (a missed support correction in one row of 1300)
    bad = G.clone()
    bad[7] = dense[7]
    bad_r = _bf16(bad)
    bad_dW, bad_dH = (bad_r.T @ h).numpy(), _bf16(bad_r @ W).numpy()
    fro = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    assert fro(bad_dW, ref_dW) > fro(got_dW, ref_dW)
    with pytest.raises(AssertionError):
        check_grad_matrix(bad_dH, ref_dH, "dH", out_bf16=True)
    with pytest.raises(AssertionError):
        check_support_rows(bad_dW, ref_dW, idx.numpy(), [7], "dW")
    with pytest.raises(AssertionError):
        check_grad_matrix(bad_dW, ref_dW, "dW")


def test_a_defect_hidden_from_the_global_norm_is_caught():
    """One wrong run of 64 elements in a 20000 x 256 dW: 1e-2 relative Frobenius over the whole matrix stays
    green, the per-row and per-element bounds do not."""
    g = torch.Generator().manual_seed(5)
    ref = torch.randn(20000, 256, generator=g, dtype=torch.float64).numpy()
    got = ref * (1 + 1e-3)
    got[12345, 64:128] = 0.0
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 1e-2
    with pytest.raises(AssertionError):
        check_grad_matrix(got, ref, "dW")


def test_zero_rows_must_be_exact_zeros():
    ref = np.zeros((4, 8)); ref[1] = 1.0
    got = ref.copy()
    check_grad_matrix(got, ref, "dH", out_bf16=True)
    got[2, 3] = 1e-9
    with pytest.raises(AssertionError):
        check_grad_matrix(got, ref, "dH", out_bf16=True)


def test_sparse_parts_split_the_oracle_gradient():
    """oracle + sparse part = the gradient of the dense part alone, g/tau * M * softmax(z/tau), written out here;
    with duplicates, an empty slot, an out-of-range index and an ignored token."""
    from gradcheck import sparse_parts, dense_dweight
    from oracle.kdkl_oracle import kdkl_oracle
    rng = np.random.default_rng(3)
    T, H, V, K, tau = 6, 5, 11, 4, 1.7
    h, W = rng.standard_normal((T, H)), rng.standard_normal((V, H))
    idx = rng.integers(0, V, (T, K))
    idx[0, 1] = idx[0, 0]; idx[1, 2] = -1; idx[2, 3] = V + 4
    val = rng.standard_normal((T, K)) * 2
    mask = np.array([1, 1, 1, 0, 1, 1], np.uint8)
    o = kdkl_oracle(h, W, idx, val, tau=tau, mask=mask, grad_loss=-0.5, teacher_lse=np.full(T, 3.0))
    S_H, S_W = sparse_parts(o, h, W, idx, tau)
    s = (h @ W.T) / tau
    q = np.exp(s - s.max(1, keepdims=True)); q /= q.sum(1, keepdims=True)
    dz = (o["g"] / tau * o["M"])[:, None] * q
    np.testing.assert_allclose(o["dH"] + S_H, dz @ W, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(o["dW"] + S_W, dz.T @ h, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(dense_dweight(o, h, W, idx, tau), np.abs(dz.T @ h), rtol=1e-12, atol=1e-15)
    assert not S_H[3].any()


def test_cancelling_support_entry_of_a_one_token_batch():
    """T = 1: every dW row is a single product. Where M q ~ p the single-pass entry keeps the rounding error of the
    stored exponential (u times the dense part), far above u times the net value: accepted with dense_mag,
    refused without; an error of twice that size is refused either way."""
    H = 64
    hrow = np.linspace(0.5, 1.5, H)
    dense_g = np.array([1e-3, 1e-3, 1.0, 1e-3, 1e-3])     # row 2: a confident student entry that cancels to 1e-3
    net_g = np.array([1e-3, 1e-3, 1e-3, 1e-3, 1e-3])      # of its dense part; the other rows are dense-only
    ref, dense = net_g[:, None] * hrow, dense_g[:, None] * hrow
    got = ref.copy()
    got[2] += 0.9 * 2.0 ** -8 * dense[2]
    with pytest.raises(AssertionError):
        check_grad_matrix(got, ref, "dW", roundings=2)
    check_grad_matrix(got, ref, "dW", roundings=2, dense_mag=dense)
    got[2] += 1.5 * 2.0 ** -8 * dense[2]
    with pytest.raises(AssertionError):
        check_grad_matrix(got, ref, "dW", roundings=2, dense_mag=dense)


def test_term_norms_against_plain_loops():
    from gradcheck import term_norms
    from oracle.kdkl_oracle import kdkl_oracle
    rng = np.random.default_rng(11)
    T, H, V, K, tau = 5, 4, 9, 3, 0.8
    h, W = rng.standard_normal((T, H)), rng.standard_normal((V, H))
    idx = rng.integers(0, V, (T, K)); idx[1, 1] = idx[1, 0]; idx[2, 2] = -1
    val = rng.standard_normal((T, K))
    mask = np.array([1, 1, 1, 0, 1], np.uint8)
    o = kdkl_oracle(h, W, idx, val, tau=tau, mask=mask, grad_loss=2.0)
    nH, nW = term_norms(o, h, W, idx, tau)
    # the dense dlogits through the oracle's own gradient: dH = G W with W = identity gives G
    G = kdkl_oracle(np.concatenate([h, np.zeros((T, V))], 1)[:, :H], W, idx, val, tau=tau, mask=mask, grad_loss=2.0)
    s = (h @ W.T) / tau
    q = np.exp(s - s.max(1, keepdims=True)); q /= q.sum(1, keepdims=True)
    want_H, want_W = np.zeros(T), np.zeros(V)
    for t in range(T):
        for v in range(V):
            p_tv = sum(o["p_k"][t, k] for k in range(K) if idx[t, k] == v)
            g_tv = o["g"][t] / tau * (o["M"][t] * q[t, v] - p_tv)
            want_H[t] += g_tv ** 2 * (W[v] ** 2).sum()
            want_W[v] += g_tv ** 2 * (h[t] ** 2).sum()
    np.testing.assert_allclose(nH, np.sqrt(want_H), rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(nW, np.sqrt(want_W), rtol=1e-12, atol=1e-18)
    assert nH[3] == 0.0 and G["loss"] == o["loss"]


def test_row_of_a_few_cancelling_terms_is_judged_against_its_terms():
    """Three tokens with opposite signs dominate a dW row of a hidden size of 8: the row's norm is a third of the
    root-sum-square of its terms. Every term rounded by half a bf16 step (the most one rounding can do) moves the
    row by more than 1e-2 of its own norm, and by 2^-9 of its terms' norm."""
    from gradcheck import check_grad_matrix
    H = 8
    hs = np.array([[1.0, -2.0, 0.5, 1.5, -1.0, 2.0, 0.25, -0.5],
                   [1.1, -1.9, 0.4, 1.6, -0.9, 2.1, 0.30, -0.6],
                   [0.9, -2.1, 0.6, 1.4, -1.1, 1.9, 0.20, -0.4]])
    g = np.array([1.0, -1.5, 0.8])                        # dlogits of the three tokens at this vocabulary row
    terms = g[:, None] * hs
    ref = np.vstack([terms.sum(0), np.ones(H), np.ones(H)])
    scale = np.array([np.sqrt((terms ** 2).sum()), 0.0, 0.0])
    got = ref.copy()
    got[0] = (terms * (1 + 2.0 ** -9 * np.array([[1.0], [-1.0], [1.0]]))).sum(0)
    assert np.linalg.norm(got[0] - ref[0]) > 1e-2 * np.linalg.norm(ref[0])
    with pytest.raises(AssertionError):
        check_grad_matrix(got, ref, "dW")
    check_grad_matrix(got, ref, "dW", row_scale=scale)
    got[0] = (terms * (1 + 12 * 2.0 ** -9 * np.array([[1.0], [-1.0], [1.0]]))).sum(0)
    with pytest.raises(AssertionError):
        check_grad_matrix(got, ref, "dW", row_scale=scale)
