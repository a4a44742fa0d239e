"""fp64 CPU oracle for the teacher top-K cache record.

TEST INFRASTRUCTURE ONLY (same rules as kdkl_oracle.py: never imported by the product path, no
code shared with the CUDA path).

What the cache holds per position (paper, section "Offline Distillation with a Top-K Teacher"):
the K largest teacher entries of the position's distribution over the vocabulary, plus, so that
the retained mass M < 1 can be kept exact instead of renormalised, the normaliser of the full
distribution. With teacher logits z = W h this is, written out:

    lse_t      = log sum_v exp(z_tv / tau)
    (idx, val) = the K largest z_tv, ordered by value descending, ties by smaller index first

The oracle is that definition: a dense float64 product, a full sort per row.
Pins (tests/test_teacher_oracle_pins.py): torch.topk / torch.logsumexp in float64, a brute-force
selection loop, and the identity sum_k exp(val_k / tau - lse) = retained mass <= 1.
"""
from __future__ import annotations

import numpy as np


def teacher_topk_oracle(hidden, weight, K, tau=1.0):
    """Returns dict(idx int32 [T,K], val float64 [T,K] (raw logits), lse float64 [T] (of z/tau), z [T,V])."""
    h = np.asarray(hidden, dtype=np.float64)
    W = np.asarray(weight, dtype=np.float64)
    z = h @ W.T
    s = z / float(tau)
    mx = s.max(axis=1)
    lse = mx + np.log(np.exp(s - mx[:, None]).sum(axis=1))
    T, V = z.shape
    idx = np.empty((T, K), dtype=np.int32)
    val = np.empty((T, K))
    cols = np.arange(V)
    for t in range(T):
        order = np.lexsort((cols, -z[t]))        # value descending, then index ascending
        idx[t] = order[:K]
        val[t] = z[t, order[:K]]
    return {"idx": idx, "val": val, "lse": lse, "z": z}
