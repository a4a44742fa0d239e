"""Out-of-bounds write detection without a sanitizer: guard bytes after every workspace slab and around every
output buffer are pre-filled with a pattern and must survive a forward + backward (both forms).

kdkl_debug_guard_bytes makes the library leave untouched bytes after each slab of its workspace layout;
kdkl_workspace_layout gives the slab table, so everything between a slab's used length and the next slab's start
can be checked. Outputs are views into one larger buffer with 1 KiB guard zones before and after each.
"""
import numpy as np
import pytest
import torch

from paper_2608_03796_b200 import binding as B

pytestmark = pytest.mark.gpu
PATTERN = 0xA5


class Carver:
    """Views at 256-byte aligned offsets inside one pattern-filled byte buffer, 1 KiB apart."""

    def __init__(self, nbytes, dev):
        self.buf = torch.full((nbytes,), PATTERN, dtype=torch.uint8, device=dev)
        self.off = 1024
        self.used = []

    def take(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        v = self.buf[self.off:self.off + n].view(dtype).view(*shape)
        self.used.append((self.off, n))
        self.off = (self.off + n + 1024 + 255) // 256 * 256
        return v

    def guards_intact(self):
        keep = torch.ones(self.buf.numel(), dtype=torch.bool, device=self.buf.device)
        for o, n in self.used:
            keep[o:o + n] = False
        return bool((self.buf[keep] == PATTERN).all())


@pytest.fixture
def guard_bytes():
    """4 KiB of guard bytes after every workspace slab for the duration of one test."""
    before = B.kdkl_debug_guard_bytes(4096)
    yield 4096
    B.kdkl_debug_guard_bytes(before)


@pytest.mark.parametrize("single_pass", [False, True])
@pytest.mark.parametrize("T,H,V,K,chunk,masked", [
    (300, 72, 1001, 7, 100, True),       # ragged everything, three chunks, dead row tiles
    (257, 264, 4120, 100, 0, False),     # one chunk, rows one past a pair tile
    (1300, 128, 520, 33, 512, True),     # several chunks, a dead chunk
    (64, 4104, 300, 5, 0, False),        # ragged last k-block
])
def test_no_kernel_writes_outside_its_buffers(guard_bytes, T, H, V, K, chunk, masked, single_pass):
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(T + V)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16).to(dev)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16).to(dev)
    idx = torch.stack([torch.randperm(V, generator=g)[:K] for _ in range(T)]).to(torch.int32).to(dev)
    val = torch.randn(T, K, generator=g).to(dev)
    mask = None
    if masked:
        mask = torch.ones(T, dtype=torch.uint8)
        mask[::7] = 0
        mask[T // 3: T // 3 + 290] = 0
        mask = mask.to(dev)
    nbytes = B.kdkl_workspace_bytes(T, H, V, K, chunk)
    slabs = B.kdkl_workspace_layout(T, H, V, K, chunk)
    assert len(slabs) >= 10 and slabs[-1][0] + slabs[-1][1] <= nbytes
    ws = torch.full((nbytes,), PATTERN, dtype=torch.uint8, device=dev)
    out = Carver(T * H * 2 + V * H * 4 + T * 4 + 2 * T * K * 4 + 64 * 1024, dev)
    dh = out.take((T, H), torch.bfloat16)
    dw = out.take((V, H), torch.float32)
    loss = out.take((1,), torch.float32)
    tok = out.take((T,), torch.float32)
    if single_pass:
        B.kdkl_forward_backward(h, W, idx, val, ws, loss, dh, dw, loss_mask=mask, chunk=chunk, loss_per_token=tok)
    else:
        gl = out.take((T, K), torch.float32)
        gi = out.take((T, K), torch.int32)
        B.kdkl_forward(h, W, idx, val, ws, loss, loss_mask=mask, chunk=chunk, loss_per_token=tok, gathered_logits=gl,
                       gathered_idx=gi)
        B.kdkl_backward(h, W, K, ws, dh, dw, loss_mask=mask, chunk=chunk)
    torch.cuda.synchronize()
    assert B.kdkl_status(ws)[0] == 0
    assert torch.isfinite(dw).all() and torch.isfinite(dh.float()).all() and torch.isfinite(loss).all()
    # every byte between the used end of a slab and the start of the next one (>= 4096 of them) is untouched
    ends = [o for o, _ in slabs[1:]] + [nbytes]
    for (o, n), nxt in zip(slabs, ends):
        assert nxt - (o + n) >= 4096
        assert bool((ws[o + n:nxt] == PATTERN).all()), f"write past the slab at offset {o} (+{n})"
    assert out.guards_intact()


@pytest.mark.parametrize("T,H,kind", [(37, 72, 0), (257, 4096, 1), (19, 20000, 1), (130, 1032, 0)])
def test_feature_loss_stays_inside_its_buffers(T, H, kind):
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(T + H)
    s = torch.randn(T, H, generator=g).to(torch.bfloat16).to(dev)
    r = torch.randn(T, H, generator=g).to(torch.bfloat16).to(dev)
    mask = (torch.arange(T) % 3 != 0).to(torch.uint8).to(dev)
    wsb = B.kdkl_feature_loss_workspace_bytes(T)
    out = Carver(wsb + T * H * 2 + T * 4 + 16 * 1024, dev)
    ws = out.take((wsb,), torch.uint8)
    d = out.take((T, H), torch.bfloat16)
    tok = out.take((T,), torch.float32)
    loss = out.take((1,), torch.float32)
    B.kdkl_feature_loss(s, r, ws, loss, kind=kind, loss_mask=mask, loss_per_token=tok, dstudent=d)
    torch.cuda.synchronize()
    assert torch.isfinite(loss).all() and out.guards_intact()


@pytest.mark.parametrize("stored", [False, True])
def test_teacher_topk_stays_inside_its_buffers(stored):
    dev = torch.device("cuda:0")
    T, H, V, K = 300, 264, 4120, 16
    g = torch.Generator().manual_seed(3)
    h = torch.randn(T, H, generator=g).to(torch.bfloat16).to(dev)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16).to(dev)
    size_fn = B.lib().kdkl_teacher_topk_stored_workspace_bytes if stored else B.lib().kdkl_teacher_topk_workspace_bytes
    wsb = size_fn(T, H, V, K)
    out = Carver(wsb + 64 * 1024, dev)
    ws = out.take((wsb,), torch.uint8)
    idx, val, lse, _ = B.kdkl_teacher_topk(h, W, K, workspace=ws, stored=stored)
    torch.cuda.synchronize()
    assert B.kdkl_status(ws)[0] == 0 and int(idx.min()) >= 0 and int(idx.max()) < V
    assert out.guards_intact()
