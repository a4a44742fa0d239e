"""torch.autograd entry to the fused chunked KL loss (and the optional feature loss).

    loss = fused_chunked_kl(hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None,
                            chunk=4096, temperature=1.0)
    loss.backward()          # hidden.grad [T,H] bf16, weight.grad [V,H] bf16 (rounded from the fp32 dW)

Marshalling only: forward runs kdkl_forward, backward runs kdkl_backward; nothing of the loss arithmetic
happens in torch ops. Neither call waits for the device: the upstream gradient stays where autograd holds it
(kdkl_options.grad_loss_device), and the device status of a step (a bounded wait that ran out, a state mismatch)
is copied to pinned host memory behind the step's kernels and looked at when the same buffers are next used, or
by check_status() - an error of step i is therefore raised during step i+1. `sync_status=True` reads the status
at the end of backward instead (one stream synchronisation per step). The single-pass form compares the upstream
gradient with `expected_grad` on the host and so reads it once (`grad.item()`).
Workspace and gradient buffers are pooled per shape, so repeated steps allocate nothing. A forward call takes a
buffer set out of the pool and owns it until its backward has run: two losses of one shape that are both alive
(loss1 + loss2, pipelined micro-batches, activation checkpointing) therefore never share the saved state of
Algorithm 1, and a backward whose buffer set has been reused in the meantime (a second backward through a freed
graph) raises instead of returning gradients of another batch. `weight_grad_fp32=True` hands the fp32 dW
buffer over to the caller (the pool allocates a new one next time) instead of a bf16 copy; with `dweight_out`
given, dW is accumulated into that fp32 tensor in place.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B

_free: dict = {}          # key -> buffer sets (FusedChunkedKL holders) no live loss is using
_probed: list = []        # buffer sets whose last step's status has not been looked at yet


def clear_cache() -> None:
    """Drops the pooled workspaces and gradient buffers (sets in use by a live loss are unaffected)."""
    try:
        check_status()
    finally:
        _free.clear()


def _probe(op) -> None:
    """Enqueue a copy of the workspace header's status words to pinned host memory behind the step's kernels."""
    if getattr(op, "probe", None) is None:
        op.probe = torch.zeros(4, dtype=torch.int32).pin_memory()
        op.probe_event = torch.cuda.Event()
    op.probe.copy_(op.workspace[:16].view(torch.int32), non_blocking=True)
    op.probe_event.record()
    if not getattr(op, "probe_pending", False):
        op.probe_pending = True
        _probed.append(op)


def _collect(op) -> None:
    """Look at the status a finished earlier step left (waits for that step's kernels only if they still run)."""
    if not getattr(op, "probe_pending", False):
        return
    op.probe_event.synchronize()
    op.probe_pending = False
    if op in _probed:
        _probed.remove(op)
    code, where = int(op.probe[0]), int(op.probe[1])
    if code not in (0, -10):                                      # -10: out-of-range teacher indices were ignored
        raise B.KdklError(code, f"device status of an earlier fused_chunked_kl step, detail {where}")


def check_status() -> None:
    """Raises if any step whose status has not been looked at yet failed on the device (waits for those steps)."""
    first = None
    for op in list(_probed):                   # every pending status is collected, the first failure is raised
        try:
            _collect(op)
        except B.KdklError as e:
            first = first or e
    if first is not None:
        raise first


def _acquire(T, H, V, K, chunk, tau, accumulate, device):
    """A buffer set for this shape that nothing else is using: out of the pool, or a new one."""
    key = (T, H, V, K, chunk, tau, accumulate, str(device))
    pool = _free.setdefault(key, [])
    if pool:
        op = pool.pop()
        _collect(op)                                              # the status its last step left
        if op.dweight is None:                                    # handed over to a caller last time
            op.dweight = torch.empty(V, H, dtype=torch.float32, device=device)
    else:
        op = B.FusedChunkedKL(T, H, V, K, chunk=chunk, temperature=tau,
                              opt=B.make_options(accumulate_dweight=accumulate), device=device)
        op.generation = 0
    op.generation += 1
    return key, op


def _release(key, op) -> None:
    _free.setdefault(key, []).append(op)


class _FusedChunkedKL(torch.autograd.Function):
    @staticmethod
    def forward(ctx, hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask, chunk, temperature, dweight_out,
                weight_grad_fp32, single_pass, expected_grad, sync_status):
        T, H = hidden.shape
        V, K = weight.shape[0], topk_idx.shape[1]
        # single pass: the gradients for an upstream gradient of 1 come out of the forward call (three projections
        # instead of four); it writes dW itself, so it is not combined with accumulation into a caller's buffer
        ctx.done = bool(single_pass) and dweight_out is None
        key, op = _acquire(T, H, V, K, int(chunk), float(temperature), 1 if dweight_out is not None else 0,
                           hidden.device)
        ctx.expected = float(expected_grad)
        if ctx.done:
            op.forward_backward(hidden, weight, topk_idx, topk_val, teacher_lse=teacher_lse, loss_mask=loss_mask,
                                grad_loss=ctx.expected)
        else:
            op.forward(hidden, weight, topk_idx, topk_val, teacher_lse=teacher_lse, loss_mask=loss_mask)
        loss = op.loss.clone().squeeze(0)
        if not (ctx.needs_input_grad[0] or ctx.needs_input_grad[1]):
            _release(key, op)                                     # no backward will come: the set is free again
            return loss
        ctx.op, ctx.key, ctx.generation, ctx.mask = op, key, op.generation, loss_mask
        ctx.dweight_out, ctx.weight_grad_fp32, ctx.sync_status = dweight_out, weight_grad_fp32, bool(sync_status)
        ctx.save_for_backward(hidden, weight)
        return loss

    @staticmethod
    def backward(ctx, grad):
        hidden, weight = ctx.saved_tensors
        op = ctx.op
        if op.generation != ctx.generation:
            raise RuntimeError("fused_chunked_kl: this loss's saved state has been reused by a later forward call "
                               "(backward ran twice without retain_graph semantics the buffers can honour)")
        if not (ctx.done and float(grad.item()) == ctx.expected):   # any other upstream gradient: the recompute path
            if ctx.dweight_out is not None:
                saved, op.dweight = op.dweight, ctx.dweight_out   # dW += into the caller's fp32 buffer
            try:                                                  # the upstream gradient stays on the device
                op.backward(hidden, weight, loss_mask=ctx.mask,
                            grad_loss=grad.detach().to(torch.float32).contiguous())
            finally:
                if ctx.dweight_out is not None:
                    op.dweight = saved
        if ctx.sync_status:
            code, detail = op.status()
            if code not in (0, -10):                              # -10: out-of-range teacher indices were ignored
                raise B.KdklError(code, f"device status, detail {detail}")
        else:
            _probe(op)
        if ctx.dweight_out is not None:
            dW = None
        elif ctx.weight_grad_fp32:
            dW, op.dweight = op.dweight, None                     # ownership passes to the caller
        else:
            dW = op.dweight.to(weight.dtype)
        dH = op.dhidden.clone()
        _release(ctx.key, op)          # free for the next forward; a second backward of this graph before that
        return dH, dW, None, None, None, None, None, None, None, None, None, None, None   # still finds its state intact


def fused_chunked_kl(hidden, weight, topk_idx, topk_val, teacher_lse: Optional[torch.Tensor] = None,
                     loss_mask: Optional[torch.Tensor] = None, chunk: int = 4096, temperature: float = 1.0,
                     dweight_out: Optional[torch.Tensor] = None, weight_grad_fp32: bool = False,
                     single_pass: bool = False, expected_grad: float = 1.0, sync_status: bool = False) -> torch.Tensor:
    """Mean forward KL between the cached top-K teacher and softmax(hidden @ weight.T / temperature).
    single_pass=True computes the gradients during the forward call (kdkl_forward_backward) for an upstream
    gradient of `expected_grad` (the weight this loss carries in the total); if backward then sees another
    value, the gradients are recomputed by kdkl_backward."""
    return _FusedChunkedKL.apply(hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask, chunk, temperature,
                                 dweight_out, weight_grad_fp32, single_pass, expected_grad, sync_status)


class _FeatureLoss(torch.autograd.Function):
    @staticmethod
    def forward(ctx, student, teacher, loss_mask, kind, weight):
        T, H = student.shape
        ws = torch.empty(B.kdkl_feature_loss_workspace_bytes(T), dtype=torch.uint8, device=student.device)
        loss = torch.zeros(1, dtype=torch.float32, device=student.device)
        B.kdkl_feature_loss(student, teacher, ws, loss, kind=kind, loss_mask=loss_mask, weight=weight)   # loss only
        ctx.save_for_backward(student, teacher, ws)
        ctx.args = (loss_mask, kind, weight)
        return loss.squeeze(0)

    @staticmethod
    def backward(ctx, g):
        # one more pass of the same kernel writes grad * d loss / d student; the upstream gradient stays on the device
        student, teacher, ws = ctx.saved_tensors
        loss_mask, kind, weight = ctx.args
        grad = torch.empty_like(student)
        scratch = torch.zeros(1, dtype=torch.float32, device=student.device)
        B.kdkl_feature_loss(student, teacher, ws, scratch, kind=kind, loss_mask=loss_mask, weight=weight,
                            grad_loss=g.detach().to(torch.float32).contiguous(), dstudent=grad)
        return grad, None, None, None, None


def feature_loss(student, teacher, loss_mask=None, kind=B.FEATURE_MSE, weight=1.0) -> torch.Tensor:
    """Hidden-state feature loss (MSE or cosine) between student and cached teacher hidden states."""
    return _FeatureLoss.apply(student, teacher, loss_mask, kind, weight)
