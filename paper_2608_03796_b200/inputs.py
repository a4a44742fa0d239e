"""Seeded synthetic inputs for the fused chunked KL loss.

This module holds only input generation: hidden states, LM-head weight, teacher
top-K records and loss masks. It contains none of the loss arithmetic and is the
one piece of code the CUDA path's tests, the benchmark and the CPU oracle's tests
all use, so both sides always see identical bit patterns.

The generator is counter based: every value is a pure function of
(seed, stream, index), so a row's data does not depend on T, on the device it was
produced on, or on how the work was split. It is written with torch integer ops
and runs on CPU or CUDA tensors alike (the 64-bit multiply wraps, logical shifts
are emulated on int64).

The inputs stand in for the paper's loss-only benchmark (section "Isolating
Loss-Kernel Scaling" and its appendix table), which is itself synthetic:
deterministic random hidden states, projection weights and sparse top-100
teacher targets.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

# stream ids
S_HIDDEN, S_WEIGHT, S_TIDX, S_TVAL, S_TOFF, S_DOC, S_MASS, S_ROWS, S_THID = 1, 2, 3, 4, 5, 6, 7, 8, 9

_MASK64 = (1 << 64) - 1


def _i64(x: int) -> int:
    """Python int -> the signed 64-bit value with the same bit pattern."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_C1 = _i64(0x9E3779B97F4A7C15)
_C2 = _i64(0xD1B54A32D192ED03)
_M1 = _i64(0xBF58476D1CE4E5B9)
_M2 = _i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """A 64-bit finaliser (xor-shift / multiply rounds) on int64 tensors."""
    x = x ^ _lsr(x, 30)
    x = x * _M1
    x = x ^ _lsr(x, 27)
    x = x * _M2
    x = x ^ _lsr(x, 31)
    return x


def _key(seed: int, stream: int) -> int:
    return _i64(seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03)


def uniform(seed: int, stream: int, index: torch.Tensor) -> torch.Tensor:
    """u in (0,1), float64, one per int64 counter in ``index``."""
    r = _mix64(_mix64(index + _key(seed, stream)) ^ _C2)
    return (_lsr(r, 11).to(torch.float64) + 0.5) * (2.0 ** -53)


def normal(seed: int, stream: int, index: torch.Tensor) -> torch.Tensor:
    """Standard normal (float64) by Box-Muller on counters 2i and 2i+1."""
    u1 = uniform(seed, stream, index * 2)
    u2 = uniform(seed, stream, index * 2 + 1)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)


def bf16_bits(x: torch.Tensor) -> torch.Tensor:
    """Round float values to bfloat16 (nearest even) and return a bf16 tensor."""
    return x.to(torch.float32).to(torch.bfloat16)


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    T: int
    H: int
    V: int
    K: int
    chunk: int
    tau: float = 1.0
    seed: int = 1234
    idx_dist: str = "uniform"      # "uniform" | "zipf"
    tok_offset: bool = True        # per-token N(0,1) offset on teacher values
    packed_docs: int = 0           # >0: packing mask with that many documents
    pad_frac: float = 0.0

    @property
    def flops(self) -> float:
        return 8.0 * self.T * self.H * self.V


CONFIGS = {
    "c1": Config("c1", T=256, H=256, V=4096, K=16, chunk=64, tok_offset=False),
    "c2": Config("c2", T=4096, H=4096, V=131072, K=100, chunk=4096),
    "c3": Config("c3", T=32768, H=4096, V=131072, K=100, chunk=4096),
    "c4a": Config("c4a", T=65536, H=4096, V=131072, K=100, chunk=4096),
    "c4b": Config("c4b", T=131072, H=4096, V=131072, K=100, chunk=4096),
    "c4c": Config("c4c", T=262144, H=4096, V=131072, K=100, chunk=4096),
    # a reduced case for profiler captures: operands still larger than L2, about 1.5 GB on the device
    "prof": Config("prof", T=2048, H=4096, V=32768, K=100, chunk=2048),
    # four full-size chunks over a quarter of the vocabulary: every GEMM launch has the benchmark's chunk and H (so a
    # launch's DRAM traffic is the benchmark's scaled by V / 131072) and the second dW pass accumulates; about 2 GB
    # on the device
    "prof2": Config("prof2", T=16384, H=4096, V=32768, K=100, chunk=4096),
    "c5": Config("c5", T=32768, H=3072, V=128256, K=100, chunk=2048, tau=2.0,
                 idx_dist="zipf", tok_offset=False, packed_docs=8, pad_frac=0.05),
    # a ragged large head (hidden 2880 = 11.25 x 256, vocabulary 201088 = 785.5 x 256: the last tile of every GEMM is
    # partial in both directions) with a token count that leaves a short last chunk and an odd chunk out of the
    # pairs one dW pass covers; packing mask as in c5
    "c6": Config("c6", T=20000, H=2880, V=201088, K=100, chunk=4096,
                 idx_dist="zipf", packed_docs=5, pad_frac=0.03),
}


def _rows(T: int, rows: Optional[torch.Tensor], device) -> torch.Tensor:
    if rows is None:
        return torch.arange(T, dtype=torch.int64, device=device)
    return rows.to(device=device, dtype=torch.int64)


def _blocked(fn, rows: torch.Tensor, width: int, budget: int = 1 << 25):
    """Apply fn(row_block) over row blocks so temporaries stay bounded."""
    step = max(1, budget // max(1, width))
    outs = [fn(rows[i:i + step]) for i in range(0, rows.numel(), step)]
    if not outs:
        return fn(rows)
    return torch.cat(outs, dim=0)


def hidden(cfg: Config, rows: Optional[torch.Tensor] = None, device="cpu") -> torch.Tensor:
    """Student final hidden states, bf16 [len(rows), H], N(0,1)."""
    r = _rows(cfg.T, rows, device)
    col = torch.arange(cfg.H, dtype=torch.int64, device=device)
    return _blocked(lambda rb: bf16_bits(normal(cfg.seed, S_HIDDEN, rb[:, None] * cfg.H + col[None, :])),
                    r, cfg.H)


def teacher_hidden(cfg: Config, rows: Optional[torch.Tensor] = None, device="cpu") -> torch.Tensor:
    """Cached teacher hidden states for the feature loss, bf16 [len(rows), H]: 0.8 x the student's
    N(0,1) draw + 0.6 x an independent N(0,1) draw, i.e. unit variance and correlation 0.8 with the
    student row (a student that already tracks its teacher, as in healing)."""
    r = _rows(cfg.T, rows, device)
    col = torch.arange(cfg.H, dtype=torch.int64, device=device)

    def block(rb):
        at = rb[:, None] * cfg.H + col[None, :]
        return bf16_bits(0.8 * normal(cfg.seed, S_HIDDEN, at) + 0.6 * normal(cfg.seed, S_THID, at))
    return _blocked(block, r, cfg.H)


def weight(cfg: Config, rows: Optional[torch.Tensor] = None, device="cpu") -> torch.Tensor:
    """LM-head weight, bf16 [len(rows), H], N(0, 1/H) (variance 1/H)."""
    r = _rows(cfg.V, rows, device)
    col = torch.arange(cfg.H, dtype=torch.int64, device=device)
    s = 1.0 / math.sqrt(cfg.H)
    return _blocked(lambda rb: bf16_bits(normal(cfg.seed, S_WEIGHT, rb[:, None] * cfg.H + col[None, :]) * s),
                    r, cfg.H)


_ZIPF_CACHE: dict = {}


def _zipf_cdf(V: int, device) -> torch.Tensor:
    k = (V, str(device))
    if k not in _ZIPF_CACHE:
        w = torch.arange(1, V + 1, dtype=torch.float64, device=device) ** (-1.1)
        c = torch.cumsum(w, 0)
        _ZIPF_CACHE[k] = c / c[-1]
    return _ZIPF_CACHE[k]


def _first_k_distinct(cand: torch.Tensor, K: int) -> torch.Tensor:
    """Per row, the first K distinct values of cand [R, Kc] in draw order."""
    R, Kc = cand.shape
    order = torch.argsort(cand, dim=1, stable=True)
    srt = torch.gather(cand, 1, order)
    dup_sorted = torch.zeros_like(srt, dtype=torch.bool)
    dup_sorted[:, 1:] = srt[:, 1:] == srt[:, :-1]
    dup = torch.zeros_like(dup_sorted)
    dup.scatter_(1, order, dup_sorted)
    keep = ~dup
    rank = torch.cumsum(keep.to(torch.int64), 1) - 1
    if int(rank[:, -1].min()) + 1 < K:
        raise RuntimeError("not enough distinct candidates; raise the candidate count")
    sel = keep & (rank < K)
    out = torch.empty((R, K), dtype=cand.dtype, device=cand.device)
    rr = torch.arange(R, device=cand.device)[:, None].expand(R, Kc)
    out[rr[sel], rank[sel]] = cand[sel]
    return out


def teacher_topk(cfg: Config, rows: Optional[torch.Tensor] = None, device="cpu"):
    """Teacher record per token: (idx int32 [R,K] distinct, values fp32 [R,K] sorted descending).

    Uniform configs: indices are the first K distinct floor(u*V) draws. Zipf config:
    draws by inverse CDF of P(rank r) ~ r^-1.1, vocabulary id = r-1. Values: K draws
    of N(0, 3) (variance 3) sorted descending, k-th value to k-th drawn index, plus an
    optional per-token N(0,1) offset.
    """
    r = _rows(cfg.T, rows, device)
    K, V = cfg.K, cfg.V
    Kc = 2048 if cfg.idx_dist == "zipf" else K + 48

    def idx_block(rb):
        ctr = rb[:, None] * Kc + torch.arange(Kc, dtype=torch.int64, device=device)[None, :]
        u = uniform(cfg.seed, S_TIDX, ctr)
        if cfg.idx_dist == "zipf":
            cand = torch.searchsorted(_zipf_cdf(V, device), u.reshape(-1)).reshape(u.shape)
            cand = cand.clamp_(max=V - 1)
        else:
            cand = torch.floor(u * V).to(torch.int64).clamp_(max=V - 1)
        return _first_k_distinct(cand, K)

    idx = _blocked(idx_block, r, Kc, budget=1 << 23).to(torch.int32)
    ctr = r[:, None] * K + torch.arange(K, dtype=torch.int64, device=device)[None, :]
    val = normal(cfg.seed, S_TVAL, ctr) * math.sqrt(3.0)
    val, _ = torch.sort(val, dim=1, descending=True)
    if cfg.tok_offset:
        val = val + normal(cfg.seed, S_TOFF, r)[:, None]
    return idx.contiguous(), val.to(torch.float32).contiguous()


def loss_mask(cfg: Config, device="cpu") -> Optional[torch.Tensor]:
    """uint8 [T] (1 = counted) or None when every token counts.

    Packed config: a padding tail of round(pad_frac*T) - docs tokens; the rest is cut
    into ``packed_docs`` documents (each >= 16 tokens) by sorted distinct cut points;
    the last token of every document and the padding are ignored.
    """
    if cfg.packed_docs <= 0:
        return None
    T, D = cfg.T, cfg.packed_docs
    pad = int(round(cfg.pad_frac * T)) - D
    body = T - pad
    u = uniform(cfg.seed, S_DOC, torch.arange(D - 1, dtype=torch.int64)).tolist()
    # cut points over the slack left after giving every document 16 tokens
    slack = body - 16 * D
    cuts = sorted(int(x * slack) for x in u)
    ends = [c + 16 * (i + 1) for i, c in enumerate(cuts)] + [body]
    m = torch.ones(T, dtype=torch.uint8)
    for e in ends:
        m[e - 1] = 0
    m[body:] = 0
    return m.to(device)


def partial_mass_lse(cfg: Config, idx_vals: torch.Tensor, rows: Optional[torch.Tensor] = None) -> torch.Tensor:
    """A synthetic full-vocabulary teacher logsumexp per token, fp32 [R].

    Chosen so the retained mass is m_t ~ U(0.6, 1): lse = logsumexp_K(values/tau) - log m_t.
    (logsumexp here only manufactures an input value; the loss never calls it.)
    """
    device = idx_vals.device
    r = _rows(cfg.T, rows, device)
    m = 0.6 + 0.4 * uniform(cfg.seed, S_MASS, r)
    lse = torch.logsumexp(idx_vals.to(torch.float64) / cfg.tau, dim=1) - torch.log(m)
    return lse.to(torch.float32)


def sample_rows(cfg: Config, n: int, chunk: Optional[int] = None) -> torch.Tensor:
    """Row subset for sampled parity: first/last row of every chunk plus n seeded rows."""
    chunk = chunk or cfg.chunk
    T = cfg.T
    edges = []
    for s0 in range(0, T, chunk):
        edges += [s0, min(T, s0 + chunk) - 1]
    u = uniform(cfg.seed, S_ROWS, torch.arange(n, dtype=torch.int64))
    pick = torch.floor(u * T).to(torch.int64).clamp_(max=T - 1).tolist()
    return torch.tensor(sorted(set(edges) | set(pick)), dtype=torch.int64)


def poison_masked(idx: torch.Tensor, val: torch.Tensor, mask: Optional[torch.Tensor]):
    """Overwrite teacher rows at ignored positions with idx=-1 / NaN (they must never be read)."""
    if mask is None:
        return idx, val
    dead = mask.to(idx.device) == 0
    idx = idx.clone()
    val = val.clone()
    idx[dead] = -1
    val[dead] = float("nan")
    return idx, val


def make_inputs(cfg: Config, device="cpu", rows: Optional[torch.Tensor] = None):
    """All inputs of one config as a dict of tensors on ``device``.

    ``rows`` restricts the token-indexed tensors (hidden, teacher, mask) to a subset;
    the weight is always whole.
    """
    h = hidden(cfg, rows, device)
    w = weight(cfg, None, device)
    idx, val = teacher_topk(cfg, rows, device)
    mask = loss_mask(cfg, device)
    if mask is not None:
        msub = mask if rows is None else mask[rows.to(mask.device)]
        idx, val = poison_masked(idx, val, msub)
        mask = msub
    return {"hidden": h, "weight": w, "topk_idx": idx, "topk_val": val, "mask": mask}
