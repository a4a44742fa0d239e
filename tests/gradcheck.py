"""Gradient comparison beyond one global norm (a helper for the GPU parity tests; not a test itself).

The CUDA path's only rounding of consequence is G (the chunk's dlogits), rounded once to bf16 before the two
output contractions; everything else is fp32 accumulation of exact bf16 products. bf16 keeps 8 significand
bits, so a rounding moves a value by at most u = 2^-8 of itself. For an output element

    out[r, c] = sum_j G[j] * x[j]        (dH: j = vocabulary, x = W[:, c];  dW: j = token, x = h[:, c])

the error is sum_j delta_j G[j] x[j] with |delta_j| <= u and no preferred sign. Two regimes:
  * one term dominates (a support entry with a large teacher probability): |error| <= u |out|;
  * many comparable terms: the error is a sum of independent zero-mean terms, standard deviation at most
    u / sqrt(3) times the root-mean-square of the row (x is N(0, s^2) along c, so the row's rms is
    s * |G|_2 and the error's deviation is (u / sqrt 3) * s * |G|_2).
Hence, element by element,

    |cuda - oracle| <= u_out |oracle| + u |oracle| + C_SIGMA * n^(1/2) * (u / sqrt 3) * rms(oracle row)

with u_out = 2^-8 when the output itself is stored in bf16 (dH by default) and 0 for fp32 outputs, n the number
of bf16 roundings inside G (1; 2 for the single-pass step, whose stored exponential is rounded as well), and
C_SIGMA = 8 standard deviations (5e8 elements of a full-size dW never reach it by chance). Row by row, the
relative Frobenius error must stay below the tolerance stated for the whole matrix (1e-2): about three times
what the model predicts (u / sqrt 3 = 2.3e-3, plus the output rounding), so a row whose sparse teacher term
or tail columns went missing fails although it vanishes inside the whole-matrix norm.

Two roundings (single-pass step). The first rounding is of the stored exponential, so its error scales with the
dense softmax part a_t q_v of an entry, not with G itself; at a support entry where the student already matches
the teacher (M q ~ p) G is much smaller than that part, and a vocabulary row of dW made of such entries has a
small norm with an error of ordinary size. With roundings >= 2 every row is therefore judged against at least
the median row's scale (norm and rms), which is the scale of the dense part, and the relative term of the
element-wise bound is taken on the dense part where the caller supplies it (`dense_mag`, the magnitude of the
output computed from M q alone: |oracle + sparse part|, see sparse_parts): u * (dense_mag + 2 |oracle|) - one
rounding of e, one of the patched entry, one of the scaled hidden row; the per-row relative error is then taken
against the larger of the row's own norm and its dense part's.

Rows made of a few cancelling terms. The bounds above take a row's own norm as the scale of its error, which holds
when many comparable terms add up. A dW row that three tokens dominate with opposite signs (hidden size 8 in the
randomized tests) has a norm well below the root-sum-square of its terms, while every term still carries its own
rounding error: the per-row relative error is taken against that root-sum-square where the caller supplies it
(`row_scale`, see term_norms), and spread over the row it stands in for the row's rms in the element-wise bound - the usual forward error bound of a sum, |sum delta_i x_i| <= u sum |x_i|.

Absolute floor. The logits themselves are fp32 sums of bf16 products pushed through exp2: a relative error of about
2^-16 on M q and on p separately. Where the two cancel almost completely the element is far below its row-mates and
its error is set by that, not by its own size: every element is allowed 2e-5 of the largest row's rms.
"""
import numpy as np

U_BF16 = 2.0 ** -8
C_SIGMA = 8.0
ROW_FRO = 1e-2
ABS_EPS = 2e-5


def sparse_parts(o, hidden, weight, topk_idx, tau):
    """The sparse teacher terms of Eq. "grad" on their own, from the oracle's per-slot probabilities p_k and
    upstream factors g: S_H[t,:] = (g_t / tau) sum_k p_tk W[idx_tk,:] and S_W[v,:] = sum_{t,k: idx_tk = v}
    (g_t / tau) p_tk h_t, so that oracle + S is the gradient of the dense part M q alone. float64 numpy."""
    h = np.asarray(hidden, dtype=np.float64)
    W = np.asarray(weight, dtype=np.float64)
    idx = np.asarray(topk_idx).astype(np.int64)
    T, K = idx.shape
    V = W.shape[0]
    coef = (o["g"][:, None] / float(tau)) * o["p_k"]                 # [T, K], 0 at unusable slots
    ok = coef != 0
    ii = np.where(ok, np.clip(idx, 0, V - 1), 0)
    S_H = np.einsum("tk,tkh->th", coef, W[ii]) if T * K * W.shape[1] <= (1 << 27) else \
        np.stack([coef[t] @ W[ii[t]] for t in range(T)])
    S_W = np.zeros_like(W)
    tt = np.repeat(np.arange(T), K).reshape(T, K)
    np.add.at(S_W, ii[ok], coef[ok][:, None] * h[tt[ok]])
    return S_H, S_W


def term_norms(o, hidden, weight, topk_idx, tau):
    """Root-sum-square of the terms each output row is a sum of (float64 numpy, the dense dlogits of Eq. "grad"
    rebuilt from the oracle's logZ, M, p_k and g): for dH row t, sqrt(sum_v G_tv^2 |W_v|^2); for dW row v,
    sqrt(sum_t G_tv^2 |h_t|^2). A rounding error of relative size u in every term gives an error of about u times
    this norm, however much the terms cancel in the sum: the scale a row's error is judged against when only a
    few tokens (or a tiny hidden size) make up the row."""
    h = np.asarray(hidden, dtype=np.float64)
    W = np.asarray(weight, dtype=np.float64)
    idx = np.asarray(topk_idx).astype(np.int64)
    T, K = idx.shape
    V = W.shape[0]
    q = np.exp((h @ W.T) / float(tau) - o["logZ"][:, None])
    p = np.zeros((T, V))
    ok = o["p_k"] != 0
    tt = np.repeat(np.arange(T), K).reshape(T, K)
    np.add.at(p, (tt[ok], np.clip(idx, 0, V - 1)[ok]), o["p_k"][ok])
    G2 = ((o["g"] / float(tau))[:, None] * (o["M"][:, None] * q - p)) ** 2
    return np.sqrt(G2 @ (W * W).sum(axis=1)), np.sqrt(G2.T @ (h * h).sum(axis=1))


def dense_dweight(o, hidden, weight, topk_idx, tau):
    """|dW| of the dense part M q alone (see sparse_parts): the `dense_mag` of a single-pass dW comparison."""
    return np.abs(o["dW"] + sparse_parts(o, hidden, weight, topk_idx, tau)[1])


def elementwise_tolerance(ref_block, out_bf16=False, roundings=1, rms_floor=0.0, dense_block=None, abs_floor=0.0,
                          row_scale=None):
    """The bound above for a block of whole rows of the oracle's matrix (float64 [rows, cols]). row_scale [rows]:
    the root-sum-square of the terms of each row (term_norms); spread over the row it replaces a smaller rms."""
    rms = np.maximum(np.sqrt(np.mean(ref_block * ref_block, axis=1, keepdims=True)), rms_floor)
    if row_scale is not None:
        rms = np.maximum(rms, np.asarray(row_scale, dtype=np.float64)[:, None] / np.sqrt(ref_block.shape[1]))
    rel = U_BF16 * ((2.0 if out_bf16 else 1.0) + (1.0 if dense_block is not None else 0.0))
    tol = rel * np.abs(ref_block) + C_SIGMA * np.sqrt(float(roundings)) * (U_BF16 / np.sqrt(3.0)) * rms + abs_floor
    if dense_block is not None:
        tol = tol + U_BF16 * np.abs(dense_block)
    return tol


def check_grad_matrix(got, ref, name, out_bf16=False, roundings=1, row_fro=ROW_FRO, block=4096, extra_tol=None,
                      dense_mag=None, abs_scale=None, row_scale=None):
    """got, ref: [rows, cols] (anything np.asarray takes; compared in float64, row block by row block so that a
    full-size dW does not need several float64 copies). extra_tol (scalar or [rows, cols]) is added to every
    element's bound: the fp32 rounding of `dW +=` onto existing contents. dense_mag ([rows, cols], single-pass
    step): the output of the dense part alone. abs_scale: the largest row rms of the WHOLE matrix when `ref` is only
    some of its rows (default: taken from ref). row_scale ([rows], see term_norms): the per-row relative error is
    taken against at least this. Raises AssertionError naming the worst row / element.
    Returns (largest per-row relative error, largest elementwise error / tolerance)."""
    rows = ref.shape[0]
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    norms = np.empty(rows)
    errs = np.empty(rows)
    dnorms = np.zeros(rows)
    worst_ratio, worst_at = 0.0, None
    norm_floor = 0.0
    for r0 in range(0, rows, block):
        b = np.asarray(ref[r0:r0 + block], dtype=np.float64)
        norms[r0:r0 + len(b)] = np.sqrt((b * b).sum(axis=1))
    if roundings >= 2 and rows:
        norm_floor = float(np.median(norms))
    rms_floor = norm_floor / np.sqrt(ref.shape[1])
    if abs_scale is None:
        abs_scale = float(norms.max()) / np.sqrt(ref.shape[1]) if rows else 0.0
    abs_floor = ABS_EPS * abs_scale
    for r0 in range(0, rows, block):
        b = np.asarray(ref[r0:r0 + block], dtype=np.float64)
        a = np.asarray(got[r0:r0 + block], dtype=np.float64)
        assert np.isfinite(a).all(), f"{name}: non-finite values in rows {r0}..{r0 + len(a) - 1}"
        diff = np.abs(a - b)
        errs[r0:r0 + len(b)] = np.sqrt((diff * diff).sum(axis=1))
        dense = None if dense_mag is None else np.asarray(dense_mag[r0:r0 + block], dtype=np.float64)
        if dense is not None:
            dnorms[r0:r0 + len(b)] = np.sqrt((dense * dense).sum(axis=1))
        tol = elementwise_tolerance(b, out_bf16, roundings, rms_floor, dense, abs_floor,
                                    None if row_scale is None else np.asarray(row_scale)[r0:r0 + block])
        tol = np.where(norms[r0:r0 + len(b), None] > 0, tol, 0.0)
        if extra_tol is not None:
            tol = tol + (extra_tol if np.ndim(extra_tol) == 0 else np.asarray(extra_tol)[r0:r0 + block])
        # rows the oracle holds as exact zeros (ignored tokens) must be exact zeros
        ratio = np.where(tol > 0, diff / np.where(tol > 0, tol, 1.0), np.where(diff > 0, np.inf, 0.0))
        k = int(np.argmax(ratio))
        if ratio.flat[k] > worst_ratio:
            worst_ratio = float(ratio.flat[k])
            rr, cc = np.unravel_index(k, ratio.shape)
            worst_at = (r0 + int(rr), int(cc), float(a[rr, cc]), float(b[rr, cc]), float(tol[rr, cc]))
    assert worst_ratio <= 1.0, (f"{name}: element (row, col, got, oracle, tolerance) = {worst_at} is "
                                f"{worst_ratio:.2f} x its tolerance")
    # per-row relative Frobenius error, on every row whose norm is not negligible next to the largest
    live = norms > 1e-6 * norms.max() if rows and norms.max() > 0 else np.zeros(rows, bool)
    denom = np.maximum(np.maximum(np.where(live, norms, 1.0), norm_floor), dnorms)
    if row_scale is not None:
        denom = np.maximum(denom, np.asarray(row_scale, dtype=np.float64))
    rel = np.where(live, errs / denom, 0.0)
    r = int(np.argmax(rel)) if rows else 0
    assert not rows or rel[r] <= row_fro, f"{name}: row {r} relative error {rel[r]:.3e} > {row_fro:.0e}"
    return (float(rel[r]) if rows else 0.0), worst_ratio


def check_support_rows(got_dw, ref_dw, topk_idx, tokens, name, roundings=1, dense_mag=None, row_scale=None):
    """The rows of dW at the teacher indices of the given tokens: the place where the sparse -p term of
    Eq. "grad" lands. Compared like any other rows, but named, so that a missing support correction is
    reported as such."""
    V = ref_dw.shape[0]
    rows = sorted({int(v) for t in tokens for v in np.asarray(topk_idx[t]).tolist() if 0 <= v < V})
    if not rows:
        return
    sel = np.asarray(rows)
    ref = np.asarray(ref_dw)
    whole = float(np.sqrt((ref * ref).mean(axis=1).max()))     # the floor is set by the whole matrix, not by the selection
    check_grad_matrix(np.asarray(got_dw)[sel], ref[sel], f"{name} (support rows)", False, roundings, block=len(sel),
                      dense_mag=None if dense_mag is None else np.asarray(dense_mag)[sel], abs_scale=whole,
                      row_scale=None if row_scale is None else np.asarray(row_scale)[sel])
