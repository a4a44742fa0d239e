"""The seeded generators: shapes, distributions and structure of each config."""
import math

import torch

from paper_2608_03796_b200 import inputs as I


def test_c1_shapes_and_distributions():
    cfg = I.CONFIGS["c1"]
    d = I.make_inputs(cfg)
    assert d["hidden"].shape == (256, 256) and d["hidden"].dtype == torch.bfloat16
    assert d["weight"].shape == (4096, 256)
    assert d["topk_idx"].dtype == torch.int32 and d["topk_val"].dtype == torch.float32
    assert abs(d["hidden"].float().std().item() - 1.0) < 0.02
    assert abs(d["weight"].float().std().item() * math.sqrt(cfg.H) - 1.0) < 0.02
    s = torch.sort(d["topk_idx"], 1)[0]
    assert not (s[:, 1:] == s[:, :-1]).any()
    assert int(d["topk_idx"].min()) >= 0 and int(d["topk_idx"].max()) < cfg.V
    assert (d["topk_val"][:, 1:] <= d["topk_val"][:, :-1]).all()
    assert d["mask"] is None


def test_rows_do_not_depend_on_T_or_on_subsetting():
    c2, c3 = I.CONFIGS["c2"], I.CONFIGS["c3"]
    r = torch.tensor([0, 5, 4095])
    assert torch.equal(I.hidden(c2, r), I.hidden(c3, r))
    i2, v2 = I.teacher_topk(c2, r)
    i3, v3 = I.teacher_topk(c3, r)
    assert torch.equal(i2, i3) and torch.equal(v2, v3)
    c1 = I.CONFIGS["c1"]
    assert torch.equal(I.hidden(c1)[r[:2]], I.hidden(c1, r[:2]))
    assert torch.equal(I.weight(c1)[r[:2]], I.weight(c1, r[:2]))


def test_c5_mask_and_zipf_and_poison():
    cfg = I.CONFIGS["c5"]
    m = I.loss_mask(cfg)
    assert m.numel() == cfg.T and int((m == 0).sum()) == 1638
    pad = int(round(0.05 * cfg.T)) - 8
    assert not m[cfg.T - pad:].any() and int((m[:cfg.T - pad] == 0).sum()) == 8
    rows = torch.arange(0, 32)
    idx, val = I.teacher_topk(cfg, rows)
    s = torch.sort(idx, 1)[0]
    assert not (s[:, 1:] == s[:, :-1]).any()
    assert (idx < 256).float().mean() > 0.3          # hits concentrate in the first vocab tile
    pi, pv = I.poison_masked(idx, val, torch.tensor([0] + [1] * 31, dtype=torch.uint8))
    assert (pi[0] == -1).all() and torch.isnan(pv[0]).all() and torch.equal(pi[1:], idx[1:])


def test_partial_mass_and_sample_rows():
    cfg = I.CONFIGS["c1"]
    idx, val = I.teacher_topk(cfg)
    lse = I.partial_mass_lse(cfg, val)
    mass = torch.exp(torch.logsumexp(val.double(), 1) - lse.double())
    assert mass.min() > 0.59 and mass.max() < 1.001
    r = I.sample_rows(cfg, 16)
    for s0 in range(0, cfg.T, cfg.chunk):
        assert s0 in r.tolist() and s0 + cfg.chunk - 1 in r.tolist()
    assert torch.equal(r, I.sample_rows(cfg, 16))
