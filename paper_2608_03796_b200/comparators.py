"""The paper's two comparison losses, as plain torch programs for measurement only.

The fused chunked loss is measured against the two other offline implementations the paper describes:

  dense_kl            section "Full Dense KL Computation": the [T, V] logits, a dense log-softmax and the teacher
                      scattered into a dense [T, V] probability tensor; O(T V) memory several times over.
  forward_chunked_kl  section "Sparse KL and Forward-Chunked Loss": the standard output projection (logits and
                      their gradient held in full), the normaliser computed chunk by chunk, the teacher kept
                      sparse (gather / scatter-add over its K entries).

They are comparison systems, not part of the library: library GEMMs and torch element-wise kernels, bf16 logits,
no hand-written kernel. Nothing in the package imports this module; bench.py times them next to the fused path
(iteration rate and peak memory versus sequence length) and one GPU test checks them against the fp64 oracle, so
that the comparison is between verified programs. Assumes distinct teacher indices per row (what a top-K cache
holds); empty slots (index < 0), a loss mask and a full-vocabulary teacher log-sum-exp are supported.
"""
from __future__ import annotations

from typing import Optional

import torch


def _teacher(topk_idx, topk_val, teacher_lse, mask, tau):
    """Sparse teacher of Eq. "kl": p [T, K] (0 in empty slots and ignored rows), clamped indices, counted rows."""
    T = topk_idx.shape[0]
    counted = torch.ones(T, dtype=torch.bool, device=topk_idx.device) if mask is None else mask != 0
    usable = (topk_idx >= 0) & counted[:, None]
    u = torch.where(usable, topk_val / tau, torch.full_like(topk_val, float("-inf")))
    if teacher_lse is None:
        lam = torch.logsumexp(torch.where(counted[:, None], u, torch.zeros_like(u)), dim=-1)
    else:
        lam = torch.where(counted, teacher_lse, torch.zeros_like(teacher_lse))
    p = torch.where(usable, torch.exp(u - lam[:, None]), torch.zeros_like(u))
    return p, topk_idx.long().clamp(min=0), counted


def dense_kl(hidden, weight, topk_idx, topk_val, *, teacher_lse=None, mask=None, tau=1.0, grad_loss=1.0):
    """Dense KL, forward + backward by autograd. Returns (loss, dhidden, dweight) as detached tensors."""
    h = hidden.detach().clone().requires_grad_(True)
    W = weight.detach().clone().requires_grad_(True)
    p_k, idx, counted = _teacher(topk_idx, topk_val, teacher_lse, mask, tau)
    z = (h @ W.T).float() / tau
    logq = torch.log_softmax(z, dim=-1)
    p = torch.zeros_like(logq).scatter_add_(1, idx, p_k)
    per_tok = torch.nn.functional.kl_div(logq, p, reduction="none").sum(-1)
    n = counted.sum().clamp(min=1)
    loss = (per_tok * counted).sum() / n
    (loss * grad_loss).backward()
    return loss.detach(), h.grad, W.grad


class _SparseChunked(torch.autograd.Function):
    """Eq. "decomp" on full logits z [T, V]: log Z per chunk of rows, sparse teacher terms over the K entries;
    the backward writes dz = (M q - p) g / tau chunk by chunk (Eq. "grad")."""

    @staticmethod
    def forward(ctx, z, p_k, idx, counted, tau, chunk):
        T = z.shape[0]
        logZ = torch.empty(T, device=z.device)
        for s0 in range(0, T, chunk):
            logZ[s0:s0 + chunk] = torch.logsumexp(z[s0:s0 + chunk].float() / tau, dim=-1)
        cross = (p_k * z.gather(1, idx).float() / tau).sum(-1)
        Msum = p_k.sum(-1)
        Hent = torch.where(p_k > 0, p_k * p_k.clamp_min(1e-38).log(), torch.zeros_like(p_k)).sum(-1)
        inv_n = 1.0 / float(counted.sum().clamp(min=1).item())
        ctx.save_for_backward(z, logZ, p_k, idx, counted, Msum)
        ctx.tau, ctx.chunk, ctx.inv_n = tau, chunk, inv_n
        return ((Hent - cross + Msum * logZ) * counted).sum() * inv_n

    @staticmethod
    def backward(ctx, g):
        z, logZ, p_k, idx, counted, Msum = ctx.saved_tensors
        tau, chunk = ctx.tau, ctx.chunk
        dz = torch.empty_like(z)
        coef = (g * ctx.inv_n / tau) * counted
        for s0 in range(0, z.shape[0], chunk):
            e = slice(s0, s0 + chunk)
            q = torch.exp(z[e].float() / tau - logZ[e, None])
            dz[e] = (q * (coef[e] * Msum[e])[:, None]).to(z.dtype)
        dz.scatter_add_(1, idx, (-(p_k * coef[:, None])).to(z.dtype))
        return dz, None, None, None, None, None


def forward_chunked_kl(hidden, weight, topk_idx, topk_val, *, teacher_lse=None, mask=None, tau=1.0, chunk=4096,
                       grad_loss=1.0):
    """Forward-chunked sparse KL, forward + backward. Returns (loss, dhidden, dweight) as detached tensors."""
    h = hidden.detach().clone().requires_grad_(True)
    W = weight.detach().clone().requires_grad_(True)
    p_k, idx, counted = _teacher(topk_idx, topk_val, teacher_lse, mask, tau)
    loss = _SparseChunked.apply(h @ W.T, p_k, idx, counted, tau, chunk)
    (loss * grad_loss).backward()
    return loss.detach(), h.grad, W.grad


METHODS = {"dense": dense_kl, "fwdchunk": forward_chunked_kl}


def run(method: str, d: dict, tau: float, chunk: int, teacher_lse: Optional[torch.Tensor] = None):
    """One forward + backward of a comparator on an inputs dict (hidden, weight, topk_idx, topk_val, mask)."""
    kw = dict(teacher_lse=teacher_lse, mask=d["mask"], tau=tau)
    if method == "fwdchunk":
        kw["chunk"] = chunk
    return METHODS[method](d["hidden"], d["weight"], d["topk_idx"], d["topk_val"], **kw)
