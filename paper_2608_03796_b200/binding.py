"""ctypes binding over the kdkl C ABI (include/kdkl.h): argument marshalling only.

Every step of the loss runs in the library's CUDA kernels. torch is used here for device
memory and the current stream, nothing else. If the shared library has not been built the
first call raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkdkl.so")

KDKL_OK = 0
ERRORS = {
    -1: "KDKL_ERR_NULL", -2: "KDKL_ERR_SHAPE", -3: "KDKL_ERR_ALIGN", -4: "KDKL_ERR_WORKSPACE",
    -5: "KDKL_ERR_ARG", -6: "KDKL_ERR_ARCH", -7: "KDKL_ERR_CUDA", -8: "KDKL_ERR_TIMEOUT",
    -9: "KDKL_ERR_STATE", -10: "KDKL_ERR_INDEX", -11: "KDKL_ERR_NONFINITE", -12: "KDKL_ERR_OVERFLOW",
    -13: "KDKL_ERR_RANGE",
}

EXPORTS = [
    "kdkl_workspace_bytes", "kdkl_forward", "kdkl_backward", "kdkl_status", "kdkl_saved_state",
    "kdkl_host_arena_bytes", "kdkl_forward_backward_host", "kdkl_profile_stages", "kdkl_gemm_bf16", "kdkl_last_error",
    "kdkl_last_launch_count", "kdkl_logz_noalloc", "kdkl_forward_shard", "kdkl_forward_finish",
    "kdkl_wait_selftest", "kdkl_teacher_topk", "kdkl_teacher_topk_workspace_bytes",
    "kdkl_feature_loss", "kdkl_feature_loss_device_grad", "kdkl_feature_loss_workspace_bytes", "kdkl_step_host_record", "kdkl_record_staging_bytes",
    "kdkl_forward_backward", "kdkl_profile_single_pass", "kdkl_teacher_topk_stored",
    "kdkl_teacher_topk_stored_workspace_bytes", "kdkl_workspace_layout", "kdkl_count_tokens",
    "kdkl_debug_guard_bytes",
]

FEATURE_MSE, FEATURE_COSINE = 0, 1


class KdklError(RuntimeError):
    def __init__(self, code: int, text: str = ""):
        self.code = code
        super().__init__(f"{ERRORS.get(code, code)} {text}".strip())


class kdkl_options(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_int32), ("teacher_mode", ctypes.c_int32),
                ("accumulate_dweight", ctypes.c_int32), ("dhidden_dtype", ctypes.c_int32),
                ("denom_override", ctypes.c_float), ("stored_exponentials", ctypes.c_int32),
                ("denom_device", ctypes.c_void_p), ("dw_chunks_per_pass", ctypes.c_int32),
                ("grad_loss_device", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library (once). Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it first (python -c 'import __graft_entry__ as g; g.build()')")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, f32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float, ctypes.c_size_t
    L.kdkl_workspace_bytes.restype = sz
    L.kdkl_workspace_bytes.argtypes = [i64, i64, i64, i32, i64, vp]
    L.kdkl_workspace_layout.restype = ctypes.c_int
    L.kdkl_workspace_layout.argtypes = [i64, i64, i64, i32, i64, vp, ctypes.POINTER(ctypes.c_int64),
                                        ctypes.POINTER(ctypes.c_int64), i32]
    L.kdkl_debug_guard_bytes.restype = ctypes.c_int64
    L.kdkl_debug_guard_bytes.argtypes = [i64]
    L.kdkl_count_tokens.restype = ctypes.c_int
    L.kdkl_count_tokens.argtypes = [vp, i64, vp, vp]
    L.kdkl_forward.restype = ctypes.c_int
    L.kdkl_forward.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, vp, sz, vp, vp, vp, vp, vp]
    L.kdkl_forward_shard.restype = ctypes.c_int
    L.kdkl_forward_shard.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i32, i64, f32, vp, vp, sz,
                                     vp, vp, vp, vp]
    L.kdkl_forward_finish.restype = ctypes.c_int
    L.kdkl_forward_finish.argtypes = [vp, i32, vp, i64, i64, i64, i32, i64, f32, vp, vp, sz, vp, vp, vp]
    L.kdkl_backward.restype = ctypes.c_int
    L.kdkl_backward.argtypes = [vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, f32, vp, sz, vp, vp, vp]
    L.kdkl_status.restype = ctypes.c_int
    L.kdkl_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)]
    L.kdkl_saved_state.restype = ctypes.c_int
    L.kdkl_saved_state.argtypes = [vp, i64, i64, i64, i32, i64, vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    L.kdkl_host_arena_bytes.restype = sz
    L.kdkl_host_arena_bytes.argtypes = [i64, i64, i64, i32, i64, vp]
    L.kdkl_forward_backward_host.restype = ctypes.c_int
    L.kdkl_forward_backward_host.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, f32, vp, sz,
                                             vp, vp, vp, vp]
    L.kdkl_forward_backward.restype = ctypes.c_int
    L.kdkl_forward_backward.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, f32, vp, sz, vp, vp,
                                        vp, vp, vp]
    L.kdkl_record_staging_bytes.restype = sz
    L.kdkl_record_staging_bytes.argtypes = [i64, i32]
    L.kdkl_step_host_record.restype = ctypes.c_int
    L.kdkl_step_host_record.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, f32, vp, sz, vp, sz,
                                        vp, vp, vp, vp]
    L.kdkl_profile_stages.restype = ctypes.c_int
    L.kdkl_profile_stages.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, f32, vp, sz,
                                      vp, vp, vp, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
    L.kdkl_profile_single_pass.restype = ctypes.c_int
    L.kdkl_profile_single_pass.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i64, f32, vp, f32, vp, sz,
                                           vp, vp, vp, vp, ctypes.POINTER(ctypes.c_float),
                                           ctypes.POINTER(ctypes.c_int32)]
    L.kdkl_gemm_bf16.restype = ctypes.c_int
    L.kdkl_gemm_bf16.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, vp, vp]
    L.kdkl_logz_noalloc.restype = ctypes.c_int
    L.kdkl_logz_noalloc.argtypes = [vp, vp, i64, i64, i64, f32, vp, vp]
    L.kdkl_teacher_topk_workspace_bytes.restype = sz
    L.kdkl_teacher_topk_workspace_bytes.argtypes = [i64, i64, i64, i32]
    L.kdkl_teacher_topk_stored_workspace_bytes.restype = sz
    L.kdkl_teacher_topk_stored_workspace_bytes.argtypes = [i64, i64, i64, i32]
    L.kdkl_teacher_topk_stored.restype = ctypes.c_int
    L.kdkl_teacher_topk_stored.argtypes = [vp, vp, i64, i64, i64, i32, f32, vp, sz, vp, vp, vp, vp]
    L.kdkl_teacher_topk.restype = ctypes.c_int
    L.kdkl_teacher_topk.argtypes = [vp, vp, i64, i64, i64, i32, f32, vp, sz, vp, vp, vp, vp]
    L.kdkl_feature_loss_workspace_bytes.restype = sz
    L.kdkl_feature_loss_workspace_bytes.argtypes = [i64]
    L.kdkl_feature_loss.restype = ctypes.c_int
    L.kdkl_feature_loss.argtypes = [vp, vp, vp, i64, i64, i32, f32, f32, f32, i32, vp, sz, vp, vp, vp, vp]
    L.kdkl_feature_loss_device_grad.restype = ctypes.c_int
    L.kdkl_feature_loss_device_grad.argtypes = [vp, vp, vp, i64, i64, i32, f32, vp, f32, i32, vp, sz, vp, vp, vp, vp]
    L.kdkl_wait_selftest.restype = ctypes.c_int
    L.kdkl_wait_selftest.argtypes = [vp, i64, vp]
    L.kdkl_last_error.restype = ctypes.c_char_p
    L.kdkl_last_error.argtypes = []
    L.kdkl_last_launch_count.restype = ctypes.c_int64
    L.kdkl_last_launch_count.argtypes = []
    _lib = L
    return L


def _check(rc: int):
    if rc != KDKL_OK:
        raise KdklError(rc, lib().kdkl_last_error().decode() if rc == -7 else "")


def _dptr(t: Optional[torch.Tensor], dtype=None, shape=None, name="tensor"):
    """Device pointer of a contiguous CUDA tensor, optionally of a given dtype and shape. Anything else is
    refused here: the library would hand the address to a kernel as it is, and a narrower element type or a
    smaller tensor than the kernel assumes would be read out of bounds."""
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"kdkl: {name}: expected a CUDA tensor, got a tensor on {t.device}")
    if t.device.index != torch.cuda.current_device():
        # the library launches on the current device and stream: a pointer into another GPU's memory would reach
        # a kernel (and a tensor map) as it is
        raise TypeError(f"kdkl: {name}: tensor on {t.device}, but the current device is "
                        f"cuda:{torch.cuda.current_device()} (one process per GPU: torch.cuda.set_device first)")
    if not t.is_contiguous():
        raise TypeError(f"kdkl: {name}: expected a contiguous tensor")
    if dtype is not None and t.dtype not in (dtype if isinstance(dtype, tuple) else (dtype,)):
        raise TypeError(f"kdkl: {name}: expected dtype {dtype}, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise TypeError(f"kdkl: {name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


_BF16, _F32, _I32, _U8 = torch.bfloat16, torch.float32, torch.int32, torch.uint8


def _hptr(t: Optional[torch.Tensor]):
    """Host pointer of a contiguous CPU tensor (the host-buffer entry point)."""
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise TypeError("kdkl: expected a contiguous host tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_options(teacher_mode=0, accumulate_dweight=0, dhidden_dtype=0, denom_override=0.0,
                 stored_exponentials=0, denom_device: Optional[torch.Tensor] = None,
                 dw_chunks_per_pass=0) -> kdkl_options:
    """denom_device: a CUDA float64 tensor of one element holding the divisor of the mean (read on the device
    when the kernels run); the caller keeps it alive until they have run."""
    ptr = None
    if denom_device is not None:
        ptr = _dptr(denom_device, torch.float64, (1,), "denom_device").value
    return kdkl_options(ctypes.sizeof(kdkl_options), teacher_mode, accumulate_dweight, dhidden_dtype, denom_override,
                        stored_exponentials, ptr, dw_chunks_per_pass, None)


def _grad_args(opt: Optional[kdkl_options], grad_loss):
    """grad_loss as a number travels by value; as a CUDA float32 tensor of one element it stays on the device
    (kdkl_options.grad_loss_device: no host read) - the options are copied with the pointer set."""
    if not isinstance(grad_loss, torch.Tensor):
        return opt, float(grad_loss)
    out = kdkl_options()
    if opt is not None:
        ctypes.memmove(ctypes.byref(out), ctypes.byref(opt), ctypes.sizeof(kdkl_options))
    out.struct_size = ctypes.sizeof(kdkl_options)
    out.grad_loss_device = _dptr(grad_loss.reshape(1), _F32, (1,), "grad_loss").value
    return out, 0.0


def kdkl_count_tokens(loss_mask: Optional[torch.Tensor], T: int, count_out: torch.Tensor) -> None:
    """Number of counted tokens (T without a mask) as one float64 on the device; enqueue-only."""
    _check(lib().kdkl_count_tokens(_dptr(loss_mask, _U8, (T,), "loss_mask"), T,
                                   _dptr(count_out, torch.float64, (1,), "count_out"), _stream()))


def kdkl_debug_guard_bytes(n: int) -> int:
    """Test hook: n untouched bytes after every workspace slab from now on (0 = compact); returns the old value."""
    return int(lib().kdkl_debug_guard_bytes(n))


def _opt_ptr(opt: Optional[kdkl_options]):
    return None if opt is None else ctypes.cast(ctypes.pointer(opt), ctypes.c_void_p)


def kdkl_workspace_bytes(T, H, V, K, chunk=0, opt=None) -> int:
    return lib().kdkl_workspace_bytes(T, H, V, K, chunk, _opt_ptr(opt))


def kdkl_workspace_layout(T, H, V, K, chunk=0, opt=None):
    """[(offset, used length)] of every workspace slab, in layout order (debug aid; see include/kdkl.h)."""
    off = (ctypes.c_int64 * 32)()
    ln = (ctypes.c_int64 * 32)()
    n = lib().kdkl_workspace_layout(T, H, V, K, chunk, _opt_ptr(opt), off, ln, 32)
    return [(int(off[i]), int(ln[i])) for i in range(n)]


def kdkl_forward(hidden, weight, topk_idx, topk_val, workspace, loss_out, *, teacher_lse=None, loss_mask=None,
                 chunk=0, temperature=1.0, opt=None, loss_per_token=None, gathered_logits=None,
                 gathered_idx=None) -> None:
    T, H = hidden.shape
    V = weight.shape[0]
    K = topk_idx.shape[1]
    _check(lib().kdkl_forward(_dptr(hidden, _BF16, (T, H), "hidden"), _dptr(weight, _BF16, (V, H), "weight"),
                              _dptr(topk_idx, _I32, (T, K), "topk_idx"), _dptr(topk_val, _F32, (T, K), "topk_val"),
                              _dptr(teacher_lse, _F32, (T,), "teacher_lse"), _dptr(loss_mask, _U8, (T,), "loss_mask"),
                              T, H, V, K, chunk, temperature, _opt_ptr(opt), _dptr(workspace, _U8, None, "workspace"),
                              workspace.numel(), _dptr(loss_out, _F32, (1,), "loss_out"),
                              _dptr(loss_per_token, _F32, (T,), "loss_per_token"),
                              _dptr(gathered_logits, _F32, (T, K), "gathered_logits"),
                              _dptr(gathered_idx, _I32, (T, K), "gathered_idx"), _stream()))


def kdkl_backward(hidden, weight, K, workspace, dhidden, dweight, *, loss_mask=None, chunk=0, temperature=1.0,
                  opt=None, grad_loss=1.0) -> None:
    T, H = hidden.shape
    V = weight.shape[0]
    dh_dtype = _F32 if (opt is not None and opt.dhidden_dtype == 1) else _BF16
    opt, grad_loss = _grad_args(opt, grad_loss)
    _check(lib().kdkl_backward(_dptr(hidden, _BF16, (T, H), "hidden"), _dptr(weight, _BF16, (V, H), "weight"),
                               _dptr(loss_mask, _U8, (T,), "loss_mask"), T, H, V, K, chunk, temperature,
                               _opt_ptr(opt), grad_loss, _dptr(workspace, _U8, None, "workspace"), workspace.numel(),
                               _dptr(dhidden, dh_dtype, (T, H), "dhidden"), _dptr(dweight, _F32, (V, H), "dweight"),
                               _stream()))


def kdkl_forward_backward(hidden, weight, topk_idx, topk_val, workspace, loss_out, dhidden, dweight, *,
                          teacher_lse=None, loss_mask=None, chunk=0, temperature=1.0, opt=None, grad_loss=1.0,
                          loss_per_token=None) -> None:
    """Single-pass forward + backward: three projections instead of four (see include/kdkl.h)."""
    T, H = hidden.shape
    V = weight.shape[0]
    K = topk_idx.shape[1]
    dh_dtype = _F32 if (opt is not None and opt.dhidden_dtype == 1) else _BF16
    opt, grad_loss = _grad_args(opt, grad_loss)
    _check(lib().kdkl_forward_backward(
        _dptr(hidden, _BF16, (T, H), "hidden"), _dptr(weight, _BF16, (V, H), "weight"),
        _dptr(topk_idx, _I32, (T, K), "topk_idx"), _dptr(topk_val, _F32, (T, K), "topk_val"),
        _dptr(teacher_lse, _F32, (T,), "teacher_lse"), _dptr(loss_mask, _U8, (T,), "loss_mask"), T, H, V, K, chunk,
        temperature, _opt_ptr(opt), grad_loss, _dptr(workspace, _U8, None, "workspace"), workspace.numel(),
        _dptr(loss_out, _F32, (1,), "loss_out"), _dptr(loss_per_token, _F32, (T,), "loss_per_token"),
        _dptr(dhidden, dh_dtype, (T, H), "dhidden"), _dptr(dweight, _F32, (V, H), "dweight"), _stream()))


def kdkl_forward_shard(hidden, weight_local, topk_idx, topk_val, workspace, shard_stats, *, vocab_offset, V_total,
                       teacher_lse=None, loss_mask=None, chunk=0, temperature=1.0, opt=None, gathered_logits=None,
                       gathered_idx=None) -> None:
    """The local sweep of one vocabulary shard; fills shard_stats [2, T] (see include/kdkl.h)."""
    T, H = hidden.shape
    V_local = weight_local.shape[0]
    K = topk_idx.shape[1]
    _check(lib().kdkl_forward_shard(_dptr(hidden, _BF16, (T, H), "hidden"),
                                    _dptr(weight_local, _BF16, (V_local, H), "weight_local"),
                                    _dptr(topk_idx, _I32, (T, K), "topk_idx"), _dptr(topk_val, _F32, (T, K), "topk_val"),
                                    _dptr(teacher_lse, _F32, (T,), "teacher_lse"),
                                    _dptr(loss_mask, _U8, (T,), "loss_mask"), T, H, V_local, vocab_offset, V_total, K,
                                    chunk, temperature, _opt_ptr(opt), _dptr(workspace, _U8, None, "workspace"),
                                    workspace.numel(), _dptr(shard_stats, _F32, (2, T), "shard_stats"),
                                    _dptr(gathered_logits, _F32, (T, K), "gathered_logits"),
                                    _dptr(gathered_idx, _I32, (T, K), "gathered_idx"), _stream()))


def kdkl_forward_finish(all_stats, n_shards, T, H, V_local, K, workspace, loss_out, *, loss_mask=None, chunk=0,
                        temperature=1.0, opt=None, loss_per_token=None) -> None:
    """Completes the sharded forward from the gathered statistics [n_shards, 2, T]."""
    _check(lib().kdkl_forward_finish(_dptr(all_stats, _F32, (n_shards, 2, T), "all_stats"), n_shards,
                                     _dptr(loss_mask, _U8, (T,), "loss_mask"), T, H, V_local, K, chunk, temperature,
                                     _opt_ptr(opt), _dptr(workspace, _U8, None, "workspace"), workspace.numel(),
                                     _dptr(loss_out, _F32, (1,), "loss_out"),
                                     _dptr(loss_per_token, _F32, (T,), "loss_per_token"), _stream()))


def kdkl_status(workspace):
    """(code, [site_or_row, counted_tokens, ignored_indices]); synchronises the current stream."""
    code = ctypes.c_int32(0)
    detail = (ctypes.c_int64 * 3)()
    _check(lib().kdkl_status(_dptr(workspace), _stream(), ctypes.byref(code), detail))
    return code.value, list(detail)


def kdkl_saved_state(workspace, T, H, V, K, chunk=0, opt=None):
    """Views of the saved log Z [T] and retained mass M [T] inside the workspace."""
    a, b = ctypes.c_void_p(), ctypes.c_void_p()
    _check(lib().kdkl_saved_state(_dptr(workspace), T, H, V, K, chunk, _opt_ptr(opt), ctypes.byref(a), ctypes.byref(b)))
    base = workspace.data_ptr()
    ws_f = workspace.view(torch.uint8)
    def view(p):
        off = p.value - base
        return ws_f[off:off + 4 * T].view(torch.float32)
    return view(a), view(b)


def kdkl_host_arena_bytes(T, H, V, K, chunk=0, opt=None) -> int:
    return lib().kdkl_host_arena_bytes(T, H, V, K, chunk, _opt_ptr(opt))


def kdkl_forward_backward_host(hidden, weight, topk_idx, topk_val, arena, loss_out, dhidden_out, dweight_out, *,
                               teacher_lse=None, loss_mask=None, chunk=0, temperature=1.0, opt=None,
                               grad_loss=1.0) -> None:
    """All tensors except ``arena`` are HOST tensors (pinned for full copy speed)."""
    T, H = hidden.shape
    V = weight.shape[0]
    K = topk_idx.shape[1]
    _check(lib().kdkl_forward_backward_host(_hptr(hidden), _hptr(weight), _hptr(topk_idx), _hptr(topk_val),
                                            _hptr(teacher_lse), _hptr(loss_mask), T, H, V, K, chunk, temperature,
                                            _opt_ptr(opt), grad_loss, _dptr(arena),
                                            arena.numel() * arena.element_size(), _hptr(loss_out), _hptr(dhidden_out),
                                            _hptr(dweight_out), _stream()))


def kdkl_record_staging_bytes(T, K) -> int:
    return lib().kdkl_record_staging_bytes(T, K)


def kdkl_step_host_record(hidden, weight, topk_idx_host, topk_val_host, staging, workspace, loss_out_host, dhidden,
                          dweight, *, teacher_lse_host=None, loss_mask_host=None, chunk=0, temperature=1.0, opt=None,
                          grad_loss=1.0) -> None:
    """One step with the cached teacher record (and mask) in HOST memory and everything else on the device."""
    T, H = hidden.shape
    V = weight.shape[0]
    K = topk_idx_host.shape[1]
    dh_dtype = _F32 if (opt is not None and opt.dhidden_dtype == 1) else _BF16
    _check(lib().kdkl_step_host_record(
        _dptr(hidden, _BF16, (T, H), "hidden"), _dptr(weight, _BF16, (V, H), "weight"), _hptr(topk_idx_host),
        _hptr(topk_val_host), _hptr(teacher_lse_host), _hptr(loss_mask_host), T, H, V, K, chunk, temperature,
        _opt_ptr(opt), grad_loss, _dptr(staging, _U8, None, "staging"), staging.numel(),
        _dptr(workspace, _U8, None, "workspace"), workspace.numel(), _hptr(loss_out_host),
        _dptr(dhidden, dh_dtype, (T, H), "dhidden"), _dptr(dweight, _F32, (V, H), "dweight"), _stream()))


STAGES = ["prep", "fwd_gemm_lse", "combine", "loss_reduce", "bwd_coef", "bwd_gemm_dlogits", "dhidden_gemm",
          "dweight_gemm"]


def kdkl_profile_stages(hidden, weight, topk_idx, topk_val, workspace, loss_out, dhidden, dweight, *,
                        teacher_lse=None, loss_mask=None, chunk=0, temperature=1.0, opt=None, grad_loss=1.0):
    """Forward + backward with an event between kernels: {stage: (ms, launches)}. Synchronises."""
    T, H = hidden.shape
    V = weight.shape[0]
    K = topk_idx.shape[1]
    ms = (ctypes.c_float * 8)()
    nl = (ctypes.c_int32 * 8)()
    _check(lib().kdkl_profile_stages(_dptr(hidden), _dptr(weight), _dptr(topk_idx), _dptr(topk_val), _dptr(teacher_lse),
                                     _dptr(loss_mask), T, H, V, K, chunk, temperature, _opt_ptr(opt), grad_loss,
                                     _dptr(workspace), workspace.numel() * workspace.element_size(), _dptr(loss_out),
                                     _dptr(dhidden), _dptr(dweight), _stream(), ms, nl))
    return {STAGES[i]: (float(ms[i]), int(nl[i])) for i in range(8)}


STAGES_SINGLE = ["prep", "fwd_gemm_lse_exp", "combine", "loss_reduce", "bwd_coef", "scale_and_patch", "dhidden_gemm",
                 "dweight_gemm"]


def kdkl_profile_single_pass(hidden, weight, topk_idx, topk_val, workspace, loss_out, dhidden, dweight, *,
                             teacher_lse=None, loss_mask=None, chunk=0, temperature=1.0, opt=None, grad_loss=1.0):
    """The single-pass step with an event between kernels: {stage: (ms, launches)}. Synchronises."""
    T, H = hidden.shape
    V = weight.shape[0]
    K = topk_idx.shape[1]
    ms = (ctypes.c_float * 8)()
    nl = (ctypes.c_int32 * 8)()
    _check(lib().kdkl_profile_single_pass(_dptr(hidden), _dptr(weight), _dptr(topk_idx), _dptr(topk_val),
                                          _dptr(teacher_lse), _dptr(loss_mask), T, H, V, K, chunk, temperature,
                                          _opt_ptr(opt), grad_loss, _dptr(workspace), workspace.numel(),
                                          _dptr(loss_out), _dptr(dhidden), _dptr(dweight), _stream(), ms, nl))
    return {STAGES_SINGLE[i]: (float(ms[i]), int(nl[i])) for i in range(8) if nl[i] > 0}


def kdkl_gemm_bf16(A, B, C, M, N, K, a_mn=0, b_mn=0, status=None) -> None:
    _check(lib().kdkl_gemm_bf16(_dptr(A), _dptr(B), _dptr(C), M, N, K, a_mn, b_mn, _dptr(status), _stream()))


def kdkl_logz_noalloc(hidden, weight, logz_out, temperature=1.0) -> None:
    """log Z per token with no device allocation by anyone: the scratch is a fixed array inside the
    library (V <= 262144). For callers that may not call cudaMalloc (a plugin inside a server whose
    pool owns the device, a latency-critical callback). Calls sharing a GPU must not overlap."""
    T, H = hidden.shape
    V = weight.shape[0]
    _check(lib().kdkl_logz_noalloc(_dptr(hidden), _dptr(weight), T, H, V, temperature, _dptr(logz_out), _stream()))


def kdkl_teacher_topk(hidden, weight, K, temperature=1.0, workspace=None, stored=False):
    """The teacher cache record: (topk_idx int32 [T,K], topk_val fp32 [T,K] descending, lse fp32 [T], workspace).
    stored=True keeps the fp32 logits of each 4096-token pass in the workspace (one projection instead of two)."""
    T, H = hidden.shape
    V = weight.shape[0]
    size_fn = lib().kdkl_teacher_topk_stored_workspace_bytes if stored else lib().kdkl_teacher_topk_workspace_bytes
    call = lib().kdkl_teacher_topk_stored if stored else lib().kdkl_teacher_topk
    if workspace is None:
        workspace = torch.empty(size_fn(T, H, V, K), dtype=torch.uint8, device=hidden.device)
    idx = torch.empty(T, K, dtype=torch.int32, device=hidden.device)
    val = torch.empty(T, K, dtype=torch.float32, device=hidden.device)
    lse = torch.empty(T, dtype=torch.float32, device=hidden.device)
    _check(call(_dptr(hidden), _dptr(weight), T, H, V, K, temperature, _dptr(workspace), workspace.numel(),
                _dptr(idx), _dptr(val), _dptr(lse), _stream()))
    return idx, val, lse, workspace


def kdkl_feature_loss_workspace_bytes(T) -> int:
    return lib().kdkl_feature_loss_workspace_bytes(T)


def kdkl_feature_loss(student, teacher, workspace, loss_out, *, kind=FEATURE_MSE, loss_mask=None, weight=1.0,
                      grad_loss=1.0, denom_override=0.0, accumulate=0, loss_per_token=None, dstudent=None) -> None:
    """Hidden-state feature loss (MSE or cosine) and its gradient in one pass; see include/kdkl.h.
    grad_loss: a number, or a CUDA float32 tensor of one element that is read on the device."""
    T, H = student.shape
    if isinstance(grad_loss, torch.Tensor):
        _check(lib().kdkl_feature_loss_device_grad(
            _dptr(student, _BF16, (T, H), "student"), _dptr(teacher, _BF16, (T, H), "teacher"),
            _dptr(loss_mask, _U8, (T,), "loss_mask"), T, H, kind, weight,
            _dptr(grad_loss.reshape(1), _F32, (1,), "grad_loss"), denom_override, accumulate,
            _dptr(workspace, _U8, None, "workspace"), workspace.numel(), _dptr(loss_out, _F32, (1,), "loss_out"),
            _dptr(loss_per_token, _F32, (T,), "loss_per_token"), _dptr(dstudent, _BF16, (T, H), "dstudent"), _stream()))
        return
    _check(lib().kdkl_feature_loss(_dptr(student, _BF16, (T, H), "student"), _dptr(teacher, _BF16, (T, H), "teacher"),
                                   _dptr(loss_mask, _U8, (T,), "loss_mask"), T, H, kind, weight, grad_loss,
                                   denom_override, accumulate, _dptr(workspace, _U8, None, "workspace"),
                                   workspace.numel(), _dptr(loss_out, _F32, (1,), "loss_out"),
                                   _dptr(loss_per_token, _F32, (T,), "loss_per_token"),
                                   _dptr(dstudent, _BF16, (T, H), "dstudent"), _stream()))


def kdkl_wait_selftest(status, limit_ns: int) -> None:
    """A wait nobody satisfies must expire into status = {KDKL_ERR_TIMEOUT, 99} (see include/kdkl.h)."""
    _check(lib().kdkl_wait_selftest(_dptr(status), limit_ns, _stream()))


def kdkl_last_launch_count() -> int:
    return lib().kdkl_last_launch_count()


class FusedChunkedKL:
    """Convenience holder: allocates workspace and outputs with torch once, then runs the two calls."""

    def __init__(self, T, H, V, K, chunk=0, temperature=1.0, opt=None, device="cuda", want_gathered=False,
                 want_per_token=False):
        self.T, self.H, self.V, self.K = T, H, V, K
        self.chunk, self.temperature, self.opt = chunk, temperature, opt
        nbytes = kdkl_workspace_bytes(T, H, V, K, chunk, opt)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.loss = torch.zeros(1, dtype=torch.float32, device=device)
        dh_dtype = torch.float32 if (opt is not None and opt.dhidden_dtype == 1) else torch.bfloat16
        self.dhidden = torch.empty(T, H, dtype=dh_dtype, device=device)
        self.dweight = torch.empty(V, H, dtype=torch.float32, device=device)
        self.loss_per_token = torch.empty(T, dtype=torch.float32, device=device) if want_per_token else None
        self.gathered_logits = torch.empty(T, K, dtype=torch.float32, device=device) if want_gathered else None
        self.gathered_idx = torch.empty(T, K, dtype=torch.int32, device=device) if want_gathered else None
        self.launches = 0

    def forward(self, hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None):
        kdkl_forward(hidden, weight, topk_idx, topk_val, self.workspace, self.loss, teacher_lse=teacher_lse,
                     loss_mask=loss_mask, chunk=self.chunk, temperature=self.temperature, opt=self.opt,
                     loss_per_token=self.loss_per_token, gathered_logits=self.gathered_logits,
                     gathered_idx=self.gathered_idx)
        self.launches = kdkl_last_launch_count()
        return self.loss

    def backward(self, hidden, weight, loss_mask=None, grad_loss=1.0):
        kdkl_backward(hidden, weight, self.K, self.workspace, self.dhidden, self.dweight, loss_mask=loss_mask,
                      chunk=self.chunk, temperature=self.temperature, opt=self.opt, grad_loss=grad_loss)
        self.launches += kdkl_last_launch_count()
        return self.dhidden, self.dweight

    def forward_backward(self, hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None, grad_loss=1.0):
        """Single-pass step (three projections): loss, dhidden and dweight from one call."""
        kdkl_forward_backward(hidden, weight, topk_idx, topk_val, self.workspace, self.loss, self.dhidden,
                              self.dweight, teacher_lse=teacher_lse, loss_mask=loss_mask, chunk=self.chunk,
                              temperature=self.temperature, opt=self.opt, grad_loss=grad_loss,
                              loss_per_token=self.loss_per_token)
        self.launches = kdkl_last_launch_count()
        return self.loss, self.dhidden, self.dweight

    def status(self):
        return kdkl_status(self.workspace)

    def saved_state(self):
        return kdkl_saved_state(self.workspace, self.T, self.H, self.V, self.K, self.chunk, self.opt)


class ShardedFusedChunkedKL:
    """One rank of the vocabulary-sharded loss (the paper's tensor-parallel variant).

    The kernels do the local work; the two exchanges of Algorithm 1 are the caller's collectives:
    an all-gather of the [2, T] shard statistics between the local sweep and the finish, and a sum of
    the fp32 partial dhidden over ranks after backward. By default they go through torch.distributed
    (NCCL); ``all_gather(out[n,2,T], local[2,T])`` and ``all_reduce_sum(tensor)`` can be injected.
    """

    def __init__(self, T, H, V_local, vocab_offset, V_total, K, n_shards, chunk=0, temperature=1.0, device="cuda",
                 all_gather=None, all_reduce_sum=None, want_per_token=False, opt=None):
        self.T, self.H, self.V_local, self.K = T, H, V_local, K
        self.vocab_offset, self.V_total, self.n_shards = vocab_offset, V_total, n_shards
        self.chunk, self.temperature = chunk, temperature
        # fp32 partial dhidden: summed over ranks in fp32 (an option struct passed in must ask for it too)
        self.opt = opt if opt is not None else make_options(dhidden_dtype=1)
        if self.opt.dhidden_dtype != 1:
            raise ValueError("ShardedFusedChunkedKL: opt.dhidden_dtype must be 1 (fp32 partial sums)")
        self.workspace = torch.empty(kdkl_workspace_bytes(T, H, V_local, K, chunk, self.opt), dtype=torch.uint8,
                                     device=device)
        self.stats_local = torch.empty(2, T, dtype=torch.float32, device=device)
        self.stats_all = torch.empty(n_shards, 2, T, dtype=torch.float32, device=device)
        self.loss = torch.zeros(1, dtype=torch.float32, device=device)
        self.loss_per_token = torch.empty(T, dtype=torch.float32, device=device) if want_per_token else None
        self.dhidden = torch.empty(T, H, dtype=torch.float32, device=device)
        self.dweight = torch.empty(V_local, H, dtype=torch.float32, device=device)
        self._all_gather = all_gather or self._dist_all_gather
        self._all_reduce_sum = all_reduce_sum or self._dist_all_reduce
        self._launches = [0, 0, 0]

    @staticmethod
    def _dist_all_gather(out, local):
        import torch.distributed as dist
        dist.all_gather_into_tensor(out.view(-1, out.shape[-1]), local)   # [R*2, T]: rank r's rows at 2r, 2r+1

    @staticmethod
    def _dist_all_reduce(t):
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.SUM)

    def forward_local(self, hidden, weight_local, topk_idx, topk_val, teacher_lse=None, loss_mask=None):
        kdkl_forward_shard(hidden, weight_local, topk_idx, topk_val, self.workspace, self.stats_local,
                           vocab_offset=self.vocab_offset, V_total=self.V_total, teacher_lse=teacher_lse,
                           loss_mask=loss_mask, chunk=self.chunk, temperature=self.temperature, opt=self.opt)
        self._launches = [kdkl_last_launch_count(), 0, 0]

    def forward_finish(self, loss_mask=None):
        kdkl_forward_finish(self.stats_all, self.n_shards, self.T, self.H, self.V_local, self.K, self.workspace,
                            self.loss, loss_mask=loss_mask, chunk=self.chunk, temperature=self.temperature,
                            opt=self.opt, loss_per_token=self.loss_per_token)
        self._launches[1] = kdkl_last_launch_count()
        return self.loss

    def launches_total(self) -> int:
        """Kernels this rank's last step enqueued (local sweep + finish + backward)."""
        return sum(self._launches)

    def forward(self, hidden, weight_local, topk_idx, topk_val, teacher_lse=None, loss_mask=None):
        self.forward_local(hidden, weight_local, topk_idx, topk_val, teacher_lse, loss_mask)
        self._all_gather(self.stats_all, self.stats_local)          # Algorithm 1: distributed max / reduce sigma
        return self.forward_finish(loss_mask)

    def backward_local(self, hidden, weight_local, loss_mask=None, grad_loss=1.0):
        kdkl_backward(hidden, weight_local, self.K, self.workspace, self.dhidden, self.dweight, loss_mask=loss_mask,
                      chunk=self.chunk, temperature=self.temperature, opt=self.opt, grad_loss=grad_loss)
        self._launches[2] = kdkl_last_launch_count()

    def backward(self, hidden, weight_local, loss_mask=None, grad_loss=1.0):
        self.backward_local(hidden, weight_local, loss_mask, grad_loss)
        self._all_reduce_sum(self.dhidden)                          # Algorithm 1: reduce dh across shards
        return self.dhidden, self.dweight

    def status(self):
        return kdkl_status(self.workspace)


class TokenShardedFusedKL:
    """One rank of the token-sharded (data-parallel) loss: this rank holds T_local tokens and the whole head.

    Rows are independent given the weight, so the only exchanges are three sums over ranks: the number of
    counted tokens (before forward: it is the divisor of the mean), the loss, and the fp32 dweight.
    dhidden needs no communication. ``all_reduce_sum(tensor)`` defaults to torch.distributed (NCCL).
    The count is taken by the library's kernel and stays on the device: its sum over ranks reaches the
    kernels through ``kdkl_options.denom_device``, so a step has no host read.
    """

    def __init__(self, T_local, H, V, K, chunk=0, temperature=1.0, device="cuda", all_reduce_sum=None):
        self.T, self.H, self.V, self.K = T_local, H, V, K
        self.chunk, self.temperature, self.device = chunk, temperature, device
        self.workspace = torch.empty(kdkl_workspace_bytes(T_local, H, V, K, chunk), dtype=torch.uint8, device=device)
        self.loss = torch.zeros(1, dtype=torch.float32, device=device)
        self.dhidden = torch.empty(T_local, H, dtype=torch.bfloat16, device=device)
        self.dweight = torch.empty(V, H, dtype=torch.float32, device=device)
        self._all_reduce_sum = all_reduce_sum or ShardedFusedChunkedKL._dist_all_reduce
        self._launches = [0, 0, 0]
        self.n_global = torch.zeros(1, dtype=torch.float64, device=device)
        self.opt = make_options(denom_device=self.n_global)    # every rank divides by the global count

    def count_tokens(self, loss_mask=None):
        """Global number of counted tokens, left on the device (one kernel, one small all-reduce)."""
        kdkl_count_tokens(loss_mask, self.T, self.n_global)
        self._launches = [kdkl_last_launch_count(), 0, 0]
        self._all_reduce_sum(self.n_global)
        return self.n_global

    def launches_total(self) -> int:
        """Kernels this rank's last step enqueued (count + forward + backward)."""
        return sum(self._launches)

    def forward_local(self, hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None):
        kdkl_forward(hidden, weight, topk_idx, topk_val, self.workspace, self.loss, teacher_lse=teacher_lse,
                     loss_mask=loss_mask, chunk=self.chunk, temperature=self.temperature, opt=self.opt)
        self._launches[1] = kdkl_last_launch_count()

    def forward(self, hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None):
        self.count_tokens(loss_mask)
        self.forward_local(hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask)
        self._all_reduce_sum(self.loss)                        # partial means add up to the global mean
        return self.loss

    def backward_local(self, hidden, weight, loss_mask=None, grad_loss=1.0):
        kdkl_backward(hidden, weight, self.K, self.workspace, self.dhidden, self.dweight, loss_mask=loss_mask,
                      chunk=self.chunk, temperature=self.temperature, opt=self.opt, grad_loss=grad_loss)
        self._launches[2] = kdkl_last_launch_count()

    def backward(self, hidden, weight, loss_mask=None, grad_loss=1.0):
        self.backward_local(hidden, weight, loss_mask, grad_loss)
        self._all_reduce_sum(self.dweight)                     # the data-parallel gradient reduction
        return self.dhidden, self.dweight

    def forward_backward_local(self, hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None,
                               grad_loss=1.0):
        """Single-pass step of this rank (three projections) with the global divisor."""
        kdkl_forward_backward(hidden, weight, topk_idx, topk_val, self.workspace, self.loss, self.dhidden,
                              self.dweight, teacher_lse=teacher_lse, loss_mask=loss_mask, chunk=self.chunk,
                              temperature=self.temperature, opt=self.opt, grad_loss=grad_loss)
        self._launches[1], self._launches[2] = kdkl_last_launch_count(), 0

    def forward_backward(self, hidden, weight, topk_idx, topk_val, teacher_lse=None, loss_mask=None, grad_loss=1.0):
        self.count_tokens(loss_mask)
        self.forward_backward_local(hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask, grad_loss)
        self._all_reduce_sum(self.loss)
        self._all_reduce_sum(self.dweight)
        return self.loss, self.dhidden, self.dweight

    def status(self):
        return kdkl_status(self.workspace)
