"""The C-ABI library builds for sm_100a, loads, and exports every symbol include/kdkl.h declares."""
import os
import re

import __graft_entry__ as entry
from paper_2608_03796_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    src = open(os.path.join(ROOT, "include", "kdkl.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(kdkl_[a-z0-9_]+)\s*\(", src)))


def test_library_builds_loads_and_exports_declared_symbols():
    entry.build()
    L = binding.lib()
    names = _declared_symbols()
    assert len(names) >= 8
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(binding.EXPORTS)


def test_sizes_without_a_gpu():
    entry.build()
    # workspace grows linearly with T at fixed chunk: the vocabulary-sized part is per chunk
    a = binding.kdkl_workspace_bytes(32768, 4096, 131072, 100, 4096)
    b = binding.kdkl_workspace_bytes(65536, 4096, 131072, 100, 4096)
    c = binding.kdkl_workspace_bytes(131072, 4096, 131072, 100, 4096)
    assert abs((c - b) - 2 * (b - a)) <= 4096
    per_token = (b - a) / 32768
    assert per_token < 2500                      # bytes of saved state per token at K = 100
    assert a - 32768 * per_token < 2.5 * 2 ** 30  # constant part: two [chunk, V] bf16 buffers + dH partials
    assert binding.kdkl_workspace_bytes(0, 1, 1, 1) == 0
    assert binding.kdkl_host_arena_bytes(256, 256, 4096, 16, 64) > binding.kdkl_workspace_bytes(256, 256, 4096, 16, 64)


def test_options_struct_layout():
    o = binding.make_options(teacher_mode=1, denom_override=3.0)
    assert o.struct_size == 48 and o.teacher_mode == 1 and o.denom_override == 3.0 and o.stored_exponentials == 0
    assert o.denom_device is None and binding.kdkl_options.denom_device.offset == 24
    assert o.grad_loss_device is None and binding.kdkl_options.grad_loss_device.offset == 40


def test_host_side_argument_checks_without_a_gpu():
    """Argument errors are detected before any CUDA call, so they can be checked on a CPU-only box.
    Pointers are fake but non-null and aligned: nothing dereferences them on these paths."""
    entry.build()
    L = binding.lib()
    P, Q = 0x10000, 0x20000                       # 16-byte aligned dummies
    T, H, V, K = 64, 64, 512, 4
    ws = binding.kdkl_workspace_bytes(T, H, V, K)

    def fwd(hidden=P, weight=P, idx=P, val=P, T=T, H=H, V=V, K=K, chunk=0, tau=1.0, opt=None, wsp=Q, wsb=ws, loss=P):
        return L.kdkl_forward(hidden, weight, idx, val, None, None, T, H, V, K, chunk, tau, opt, wsp, wsb, loss,
                              None, None, None, None)
    assert fwd(hidden=None) == -1 and fwd(loss=None) == -1 and fwd(idx=None) == -1
    assert fwd(T=0) == -2 and fwd(H=60) == -2 and fwd(K=0) == -2 and fwd(K=2000) == -2
    assert fwd(tau=0.0) == -5 and fwd(tau=-1.0) == -5 and fwd(chunk=-1) == -5
    assert fwd(hidden=P + 2) == -3 and fwd(wsp=Q + 8) == -3
    assert fwd(wsb=ws - 1) == -4
    bad_opt = binding.make_options()
    bad_opt.struct_size = 7
    assert fwd(opt=binding._opt_ptr(bad_opt)) == -5
    assert fwd(opt=binding._opt_ptr(binding.make_options(teacher_mode=1)), tau=2.0) == -5
    old_size = binding.make_options()
    old_size.struct_size = 20                     # the struct before stored_exponentials was added is still accepted
    assert fwd(opt=binding._opt_ptr(old_size), wsb=ws - 1) == -4
    for size in (24, 32, 40):                     # ... and so are the later, shorter layouts
        old_size.struct_size = size
        assert fwd(opt=binding._opt_ptr(old_size), wsb=ws - 1) == -4
    # stored exponentials need one chunk over all tokens
    assert fwd(opt=binding._opt_ptr(binding.make_options(stored_exponentials=1)), chunk=32) == -5
    assert fwd(opt=binding._opt_ptr(binding.make_options(stored_exponentials=2))) == -5
    # backward: same checks plus its own outputs
    def bwd(dh=P, dw=P, **kw):
        a = dict(hidden=P, weight=P, T=T, H=H, V=V, K=K, chunk=0, tau=1.0, wsp=Q, wsb=ws)
        a.update(kw)
        return L.kdkl_backward(a["hidden"], a["weight"], None, a["T"], a["H"], a["V"], a["K"], a["chunk"], a["tau"],
                               None, 1.0, a["wsp"], a["wsb"], dh, dw, None)
    assert bwd(dh=None) == -1 and bwd(dw=None) == -1 and bwd(V=0) == -2 and bwd(wsb=16) == -4 and bwd(dw=P + 4) == -3
    # sharded entry: window must lie inside the vocabulary
    assert L.kdkl_forward_shard(P, P, P, P, None, None, T, H, 256, 300, V, K, 0, 1.0, None, Q, ws, P, None, None,
                                None) == -2
    assert L.kdkl_gemm_bf16(P, P, P, 64, 64, 60, 0, 0, None, None) == -2
    assert L.kdkl_wait_selftest(P, 0, None) == -5
    assert L.kdkl_logz_noalloc(P, P, 8, 64, 262144 + 256, 1.0, P, None) == -4
    # feature loss
    fws = binding.kdkl_feature_loss_workspace_bytes(T)
    assert fws >= 256 + 4 * T and fws % 16 == 0

    def feat(s=P, r=P, T=T, H=H, kind=0, weight=1.0, acc=0, wsp=Q, wsb=fws, loss=P, dst=P):
        return L.kdkl_feature_loss(s, r, None, T, H, kind, weight, 1.0, 0.0, acc, wsp, wsb, loss, None, dst, None)
    assert feat(s=None) == -1 and feat(r=None) == -1 and feat(loss=None) == -1 and feat(wsp=None) == -1
    assert feat(T=0) == -2 and feat(H=12) == -2
    assert feat(kind=2) == -5 and feat(acc=3) == -5 and feat(weight=float("nan")) == -5
    assert feat(s=P + 8) == -3 and feat(dst=P + 2) == -3
    assert feat(wsb=fws - 1) == -4


def test_header_is_plain_c99(tmp_path):
    """The boundary is a C ABI: the header must compile as C, with no C++ or torch types."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        import pytest
        pytest.skip("no gcc")
    src = tmp_path / "use.c"
    src.write_text('#include "kdkl.h"\nint main(void) { kdkl_options o; o.struct_size = (int32_t)sizeof(o); '
                   'return kdkl_workspace_bytes(1, 8, 8, 1, 0, &o) == 0; }\n')
    subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                    "-I", os.path.join(ROOT, "include"), str(src)], check=True)


def test_binding_refuses_host_tensors_where_device_pointers_are_expected():
    """A CPU tensor (or a strided view) handed to a device entry point must raise before the library sees
    the address: there is no CPU path to fall back to, and a kernel must never get a host pointer."""
    import pytest
    import torch
    from paper_2608_03796_b200 import autograd
    entry.build()
    h = torch.zeros(8, 64, dtype=torch.bfloat16)
    W = torch.zeros(128, 64, dtype=torch.bfloat16)
    idx = torch.zeros(8, 4, dtype=torch.int32)
    val = torch.zeros(8, 4)
    ws = torch.empty(binding.kdkl_workspace_bytes(8, 64, 128, 4), dtype=torch.uint8)
    loss = torch.zeros(1)
    with pytest.raises(TypeError):
        binding.kdkl_forward(h, W, idx, val, ws, loss)
    with pytest.raises(TypeError):
        binding.kdkl_feature_loss(h, h, ws, loss)
    with pytest.raises(TypeError):
        autograd.fused_chunked_kl(h.requires_grad_(False), W, idx, val)
    assert binding._dptr(None) is None and binding._hptr(None) is None
    with pytest.raises(TypeError):
        binding._hptr(torch.zeros(4, 4).t())          # strided view
