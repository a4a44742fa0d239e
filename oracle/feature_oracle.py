"""fp64 CPU oracle for the hidden-state feature loss that is added to the logit KL.

TEST INFRASTRUCTURE ONLY (same rules as kdkl_oracle.py: never imported by the product path, no
code shared with the CUDA path).

The paper (section "Additional Ablations", paragraph "Loss design") recommends adding a
hidden-state feature loss to the logit KL and names two variants, mean-squared error and cosine,
without printing a formula. The oracle therefore writes out the textbook definitions, per token t
with student row s_t and teacher row r_t of width H:

    MSE     f_t = (1/H) sum_h (s_th - r_th)^2
    cosine  f_t = 1 - <s_t, r_t> / (|s_t| |r_t|)        (f_t = 1 when |s_t| |r_t| <= eps)

reduced like the KL term (mean over the mask = 1 positions, N = number of them, N = 0 gives 0):

    loss = weight * sum_t mask_t f_t / N

and the gradient with respect to the student rows, g_t = grad_loss * weight * mask_t / N:

    MSE     d s_t = g_t (2/H) (s_t - r_t)
    cosine  d s_t = -g_t ( r_t / (|s_t||r_t|) - <s_t,r_t> s_t / (|s_t|^3 |r_t|) )   (0 on degenerate rows)

Pins (tests/test_feature_oracle_pins.py): torch float64 mse_loss / cosine_embedding_loss with
autograd, central finite differences, and closed forms (equal rows, opposite rows, orthogonal
rows, scale invariance of the cosine variant, gradient orthogonal to s for the cosine variant).
"""
from __future__ import annotations

import numpy as np

KIND_MSE = 0
KIND_COSINE = 1
COS_EPS = 1e-12


def feature_loss_oracle(student, teacher, kind=KIND_MSE, mask=None, weight=1.0, grad_loss=1.0, denom=None,
                        want_grads=True):
    """student, teacher: [T,H] (any real dtype, widened to float64). Returns dict(loss, loss_tok [T], N, dS [T,H])."""
    s = np.asarray(student, dtype=np.float64)
    r = np.asarray(teacher, dtype=np.float64)
    T, H = s.shape
    m = np.ones(T) if mask is None else (np.asarray(mask) != 0).astype(np.float64)
    N = float(m.sum()) if denom is None else float(denom)
    if kind == KIND_MSE:
        diff = s - r
        f = (diff * diff).sum(axis=1) / H
    elif kind == KIND_COSINE:
        dot = (s * r).sum(axis=1)
        ns = np.sqrt((s * s).sum(axis=1))
        nr = np.sqrt((r * r).sum(axis=1))
        ok = ns * nr > COS_EPS
        den = np.where(ok, ns * nr, 1.0)
        f = np.where(ok, 1.0 - dot / den, 1.0)
    else:
        raise ValueError("kind")
    f = np.where(m != 0, f, 0.0)                     # ignored rows may hold anything, NaN included
    loss = float(weight) * f.sum() / N if N > 0 else 0.0
    out = {"loss": loss, "loss_tok": f, "N": N}
    if want_grads:
        g = (float(grad_loss) * float(weight) / N) * m if N > 0 else np.zeros(T)
        if kind == KIND_MSE:
            dS = g[:, None] * (2.0 / H) * diff
        else:
            ns_ = np.where(ok, ns, 1.0)
            nr_ = np.where(ok, nr, 1.0)
            dS = -g[:, None] * (r / (ns_ * nr_)[:, None] - (dot / (ns_ ** 3 * nr_))[:, None] * s)
            dS = np.where(ok[:, None], dS, 0.0)
        out["dS"] = np.where(m[:, None] != 0, dS, 0.0)
    return out
