"""Seeded generator: value ranges, determinism, recipe structure (CPU)."""
import numpy as np
import scipy.special
import torch

import bebop_gen as G


def test_open_uniforms_are_exact_and_open():
    g = torch.Generator().manual_seed(1)
    u = G.open_uniform((100000,), g, "cpu")
    assert u.dtype == torch.float32 and float(u.min()) > 0 and float(u.max()) < 1
    k = u.double() * 2 ** 24
    assert torch.equal(k, k.round()) and bool(((k.long() % 2) == 1).all())
    assert abs(float(u.mean()) - 0.5) < 5e-3


def test_tiny_config_is_deterministic_and_shaped():
    cfg = G.get_config("tiny")
    a, b = G.make_inputs(cfg), G.make_inputs(cfg)
    assert a["target"].shape == (4, 4, 1024) and a["draft"].shape == (4, 3, 1024)
    assert a["target"].dtype == torch.float32 and a["draft_tokens"].dtype == torch.int32
    for k in ("target", "draft", "draft_tokens", "u_accept", "u_final"):
        assert torch.equal(a[k], b[k])
    assert G.checksum(a["target"]) == G.checksum(b["target"])
    c = G.make_inputs(G.get_config("tiny", seed=9))
    assert not torch.equal(a["target"], c["target"])
    assert abs(float(a["target"].std()) - 2.0) < 0.1
    assert abs(float((a["draft"] - a["target"][:, :3]).std()) - 0.5) < 0.05
    assert a["draft_len"] is None and a["temperature"] is None and a["temperature_all"] == 1.0


def test_peaks_ragged_and_temperatures():
    cfg = G.get_config("full_batch", B=12, V=4096)
    x = G.make_inputs(cfg)
    assert x["target"].dtype == torch.bfloat16
    dl = x["draft_len"]
    assert dl.dtype == torch.int32 and int(dl.min()) >= 1 and int(dl.max()) <= cfg.K
    t = x["temperature"]
    assert float(t.min()) >= 0.6 and float(t.max()) <= 1.2
    # eight peaks per row, heights 8 * i^(-2/3), at distinct ids (checked in f32, same noise stream)
    a = G.make_inputs(G.get_config("full_batch", B=3, V=4096, dtype="f32"))["target"]
    b = G.make_inputs(G.get_config("full_batch", B=3, V=4096, dtype="f32", peaks=False))["target"]
    d = (a - b)
    assert bool(((d.abs() > 1e-3).sum(-1) == 8).all())
    top = d.topk(8, dim=-1).values
    want = 8.0 * torch.arange(1, 9, dtype=torch.float32) ** (-2.0 / 3.0)
    assert torch.allclose(top, want.expand_as(top), atol=1e-4)
    assert abs(float(want[-1]) - 2.0) < 1e-6
    half = G.make_inputs(G.get_config("large_vocab", B=6, V=2048))
    assert half["temperature"].tolist() == [0.7, 0.7, 0.7, 1.0, 1.0, 1.0] or \
        np.allclose(half["temperature"].numpy(), [0.7] * 3 + [1.0] * 3)


def test_padded_rows_view():
    cfg = G.get_config("tiny", V=1000)
    x = G.make_inputs(cfg, pad_ld=24)
    assert x["ld"] == 1024 and x["target"].stride(1) == 1024 and x["target"].shape[-1] == 1000
    y = G.make_inputs(cfg)
    assert torch.equal(x["target"], y["target"]) and torch.equal(x["draft_tokens"], y["draft_tokens"])


def test_draft_tokens_follow_q():
    """Gumbel-max drafts are distributed as softmax(z_q / tau) (chi-squared, V = 8)."""
    cfg = G.Config("t", 40000, 1, 8, "f32", 1.0, False, 0.0, 0.8, seed=3)
    x = G.make_inputs(cfg)
    # make every row identical so that the empirical histogram estimates one q
    z = x["draft"][0, 0].clone()
    g = torch.Generator().manual_seed(5)
    e = torch.empty((cfg.B, 8)).exponential_(generator=g)
    tok = (z[None] / 0.8 - e.log()).argmax(-1).numpy()
    q = scipy.special.softmax(z.double().numpy() / np.float64(np.float32(0.8)))
    cnt = np.bincount(tok, minlength=8)
    chi2 = float(((cnt - cfg.B * q) ** 2 / (cfg.B * q)).sum())
    assert chi2 < 24.32
    assert int(x["draft_tokens"].min()) >= 0 and int(x["draft_tokens"].max()) < 8


def test_argmax_drafts_take_lowest_index():
    z = torch.tensor([[1.0, 3.0, 3.0, 2.0], [5.0, 5.0, 5.0, 5.0]])
    assert G.first_argmax(z).tolist() == [1, 0]
    cfg = G.get_config("tiny")
    x = G.make_inputs(cfg, draft_mode="argmax")
    assert torch.equal(x["draft_tokens"].long(), G.first_argmax(x["draft"].float()))


def test_rows_read():
    cfg = G.get_config("rollout")
    assert G.rows_read(cfg, None) == 448
    assert G.rows_read(cfg, torch.tensor([1, 2, 3], dtype=torch.int32)) == 15
