"""fp64 CPU oracle for the fused chunked KL distillation loss.

TEST INFRASTRUCTURE ONLY. This file is the slow, dense, obviously-correct statement
of what the CUDA path must compute. Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product never does, and it shares
no code with the CUDA path.

The fused loss is not an approximation: the paper states that its three offline
implementations are equivalent evaluations of one identity (section "Offline
Distillation with a Top-K Teacher", Eq. "decomp"). So the oracle is the plain
definition written out: it materialises the dense logit matrix, the dense teacher
and the dense softmax in float64 and applies Eq. "kl" and Eq. "grad" to them.
numpy's float64 matrix product serves as the projection step; nothing is tiled,
fused or reordered (``row_block`` only bounds memory: rows are independent, and
dW is the plain sum of the per-block sums).

Pins (tests/test_oracle_pins.py): torch float64 kl_div + autograd, cross-entropy
for K=1, closed form for W=0, the zero point K=V with teacher = student, central
finite differences, a pure-Python brute force on tiny inputs, the bound of the
log-sum inequality, and chunk/slot-order/offset invariances. Every function in
this file is covered by at least one of them.

Readings of the paper taken here (each is listed in the design notes too):
  * teacher values l[t,k] become probabilities p_k = exp(l_k/tau - Lambda_t) with
    Lambda_t = teacher_lse[t] when given (retained mass M_t < 1 possible, never
    renormalised: section "Offline Distillation with a Top-K Teacher"), else the
    logsumexp over the row's K values (M_t = 1), else 0 in log-probability mode;
  * student q = softmax(z/tau); no tau^2 factor on the loss; gradient carries 1/tau;
  * duplicate indices in a row add (scatter-add, section "Sparse KL and
    Forward-Chunked Loss"); idx < 0 is an empty slot; idx >= V is ignored and counted;
  * the loss is the mean over positions with mask = 1 (text below Eq. "kl").
"""
from __future__ import annotations

import numpy as np


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def teacher_probs(topk_val, tau, teacher_lse=None, teacher_mode=0, valid=None):
    """p[t,k] from cached teacher values (reading Q1 above). Invalid slots get p = 0.

    Section "Offline Distillation with a Top-K Teacher": p lives on the support S,
    M = sum_S p <= 1, not renormalised.
    """
    l = _f64(topk_val)
    if valid is None:
        valid = np.ones(l.shape, dtype=bool)
    u = np.where(valid, l, -np.inf) / float(tau)
    if teacher_mode == 1:
        if float(tau) != 1.0:
            raise ValueError("log-probability mode needs tau = 1")
        lam = np.zeros(l.shape[0])
    elif teacher_lse is not None:
        lam = _f64(teacher_lse)
    else:
        mx = np.max(u, axis=1)
        mx = np.where(np.isfinite(mx), mx, 0.0)
        with np.errstate(divide="ignore"):
            lam = mx + np.log(np.sum(np.exp(u - mx[:, None]), axis=1))
    with np.errstate(invalid="ignore"):
        p = np.exp(u - lam[:, None])
    return np.where(valid, p, 0.0)


def kdkl_oracle(hidden, weight, topk_idx, topk_val, tau=1.0, mask=None, teacher_lse=None,
                teacher_mode=0, grad_loss=1.0, denom=None, want_grads=True, row_block=None):
    """Dense fp64 evaluation of loss and gradients.

    hidden [T,H], weight [V,H] (any float dtype, widened exactly), topk_idx int [T,K],
    topk_val [T,K], mask [T] (1 = counted) or None, denom = divisor of the mean
    (default: number of counted tokens).

    Returns a dict with: loss, loss_tok [T] (0 at ignored rows), logZ [T] (of z/tau),
    M [T], p_k [T,K] (the teacher probability of every slot, 0 at unusable slots) and g [T] (the upstream
    factor grad_loss * mask / N of every token), gathered_logits [T,K] (z at the teacher indices, unscaled; NaN at empty
    slots), gathered_idx [T,K], n_bad_idx, and with want_grads: dH [T,H], dW [V,H].
    """
    h = _f64(hidden)
    W = _f64(weight)
    idx = np.asarray(topk_idx).astype(np.int64)
    T, H = h.shape
    V = W.shape[0]
    K = idx.shape[1]
    tau = float(tau)
    msk = np.ones(T, dtype=bool) if mask is None else (np.asarray(mask) != 0)
    N = float(msk.sum()) if denom is None else float(denom)

    valid = (idx >= 0) & (idx < V) & msk[:, None]
    n_bad = int(((idx >= V) & msk[:, None]).sum())
    lse_in = None if teacher_lse is None else np.where(msk, _f64(teacher_lse), 0.0)
    p_k = teacher_probs(np.where(valid, _f64(topk_val), 0.0), tau, lse_in, teacher_mode, valid)
    M = p_k.sum(axis=1)                                   # retained mass

    loss_tok = np.zeros(T)
    logZ = np.zeros(T)
    zg = np.full((T, K), np.nan)
    dH = np.zeros((T, H)) if want_grads else None
    dW = None
    g = np.where(msk, float(grad_loss) / N, 0.0) if N > 0 else np.zeros(T)

    step = T if not row_block else int(row_block)
    for r0 in range(0, T, max(step, 1)):
        r1 = min(T, r0 + step)
        R = r1 - r0
        z = h[r0:r1] @ W.T                                # Algorithm 1: z = h W^T
        s = z / tau
        mx = s.max(axis=1)
        lz = mx + np.log(np.exp(s - mx[:, None]).sum(axis=1))   # log Z (text above Eq. "kl")
        logq = s - lz[:, None]
        logZ[r0:r1] = lz

        # dense teacher by scatter-add (section "Full Dense KL Computation")
        p = np.zeros((R, V))
        rr = np.repeat(np.arange(R), K).reshape(R, K)
        vv = valid[r0:r1]
        np.add.at(p, (rr[vv], idx[r0:r1][vv]), p_k[r0:r1][vv])

        # Eq. "kl": sum_v p_v (log p_v - log q_v) over the support
        with np.errstate(divide="ignore", invalid="ignore"):
            term = np.where(p > 0, p * (np.log(p) - logq), 0.0)
        L_def = term.sum(axis=1)
        # Eq. "decomp": H - C + M log Z
        with np.errstate(divide="ignore", invalid="ignore"):
            Hent = np.where(p > 0, p * np.log(p), 0.0).sum(axis=1)
        Cx = (p * s).sum(axis=1)
        L_dec = Hent - Cx + M[r0:r1] * lz
        if not np.allclose(L_def, L_dec, rtol=1e-10, atol=1e-10):
            raise AssertionError("definition and decomposition disagree")
        loss_tok[r0:r1] = np.where(msk[r0:r1], L_def, 0.0)

        ii = np.clip(idx[r0:r1], 0, V - 1)
        zsel = np.take_along_axis(z, ii, axis=1)
        okslot = (idx[r0:r1] >= 0) & (idx[r0:r1] < V)
        zg[r0:r1] = np.where(okslot, zsel, np.nan)

        if want_grads:
            # Eq. "grad": dL/dz_v = M q_v - p_v, times g/tau (chain rule through s = z/tau)
            dz = (g[r0:r1, None] / tau) * (M[r0:r1, None] * np.exp(logq) - p)
            dH[r0:r1] = dz @ W                            # Algorithm 1: dh = G W
            dWb = dz.T @ h[r0:r1]                         # Algorithm 1: dW += G^T h
            dW = dWb if dW is None else dW + dWb

    loss = float(loss_tok.sum() / N) if N > 0 else 0.0
    out = {"loss": loss, "loss_tok": loss_tok, "logZ": logZ, "M": M, "p_k": p_k, "g": g, "gathered_logits": zg,
           "gathered_idx": np.asarray(topk_idx).astype(np.int32).copy(), "n_bad_idx": n_bad, "N": N}
    if want_grads:
        out["dH"] = dH
        out["dW"] = dW if dW is not None else np.zeros((V, H))
    return out
