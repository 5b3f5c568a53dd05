"""Seeded synthetic inputs for the verify step: logits, draft tokens, uniforms.

This module only manufactures inputs.  It holds none of the verify arithmetic
(no softmax, no acceptance test, no CDF): draft tokens are drawn from
softmax(z_q / tau) with the Gumbel-max identity, argmax(z_q / tau + G), on the
stored (already rounded) draft logits, so neither the oracle nor the kernels
share code with it.  Both sides then read the very same tensors.

The shapes follow the five benchmark configurations plus the headline case;
the logits stand in for the rollout logits of a production-size vocabulary
(V = 151936 or 262144), which are not available offline.

Determinism: every tensor has its own torch.Generator stream derived from
(seed, stream id); logits are produced in fixed chunks of CHUNK sequences, so a
(config, seed, device type) triple always yields the same bits.  CPU and CUDA
generators yield different bits for the same seed; a test only ever compares
implementations on one stored tensor set.
"""
from dataclasses import dataclass, replace
from typing import Optional, Tuple, Union

import torch

CHUNK = 8  # sequences generated per step (bounds the fp32 staging memory)

_STREAMS = dict(target=1, draft=2, peaks=3, gumbel=4, u_accept=5, u_final=6, lengths=7,
                temperature=8, noise_std=9, peak_perm=10)


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    K: int
    V: int
    dtype: str                                   # "f32" | "bf16"
    target_std: float
    peaks: bool                                  # 8 Zipf-ranked peaks per row, h_i = 8 * i^(-2/3)
    noise_std: Union[float, Tuple[float, float]]  # draft = target + N(0, s^2); (lo, hi) -> per-row U(lo, hi)
    temperature: Union[float, str, Tuple[float, float]]  # float | "half_0.7_1.0" | (lo, hi) per row
    ragged: bool = False                         # draft_len ~ uniform{1..K}
    seed: int = 0


CONFIGS = {
    "tiny": Config("tiny", 4, 3, 1024, "f32", 2.0, False, 0.5, 1.0, seed=0),
    "rollout": Config("rollout", 64, 3, 151936, "bf16", 3.0, True, 1.0, 1.0, seed=1),
    "high_entropy": Config("high_entropy", 256, 5, 151936, "bf16", 1.0, False, 1.5, 1.0, seed=2),
    "large_vocab": Config("large_vocab", 512, 3, 262144, "bf16", 3.0, True, (0.2, 2.0), "half_0.7_1.0", seed=3),
    "full_batch": Config("full_batch", 1024, 4, 151936, "bf16", 3.0, True, (0.3, 1.5), (0.6, 1.2),
                         ragged=True, seed=4),
    # the configuration the headline metric is quoted on: "rollout" recipe at B = 256
    "headline": Config("headline", 256, 3, 151936, "bf16", 3.0, True, 1.0, 1.0, seed=5),
}


def get_config(name: str, **overrides) -> Config:
    return replace(CONFIGS[name], **overrides)


def _gen(seed: int, stream: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed + 1) * 1_000_003 + _STREAMS[stream])
    return g


def open_uniform(shape, g, device) -> torch.Tensor:
    """u = (2 r + 1) * 2^-24 with r a 23-bit integer: exact in fp32, never 0 or 1."""
    r = torch.randint(0, 1 << 23, shape, generator=g, device=device, dtype=torch.int64)
    return ((2 * r + 1).to(torch.float32) * (2.0 ** -24)).contiguous()


def torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def first_argmax(z: torch.Tensor) -> torch.Tensor:
    """Lowest index attaining the row maximum along the last dimension."""
    m = z.max(dim=-1, keepdim=True).values
    idx = torch.arange(z.shape[-1], device=z.device).expand_as(z)
    return torch.where(z == m, idx, z.shape[-1]).min(dim=-1).values


def make_inputs(cfg: Config, device="cpu", draft_mode: str = "sample", pad_ld: int = 0) -> dict:
    """Build the tensors of one verify call.

    draft_mode: "sample" (x_k ~ softmax(z_q/tau)) or "argmax" (x_k = argmax z_q,
    lowest index; the greedy-draft run).  pad_ld > 0 makes the row stride V + pad_ld
    elements (the padding is filled with a large finite value that must never be read).
    Returns target [B,K+1,V], draft [B,K,V] (views with row stride ld), draft_tokens
    [B,K] i32, draft_len [B] i32 or None, temperature [B] f32 or None,
    temperature_all, u_accept [B,K] f32, u_final [B] f32.
    """
    device = torch.device(device)
    B, K, V = cfg.B, cfg.K, cfg.V
    dt = torch_dtype(cfg.dtype)
    ld = V + pad_ld
    tgt_store = torch.empty((B, K + 1, ld), dtype=dt, device=device)
    drf_store = torch.empty((B, max(K, 1), ld), dtype=dt, device=device)
    if pad_ld:
        tgt_store.fill_(1e4)
        drf_store.fill_(1e4)
    target = tgt_store[:, :, :V]
    draft = drf_store[:, :K, :V]

    # per-row scalars
    if isinstance(cfg.noise_std, tuple):
        lo, hi = cfg.noise_std
        nstd = lo + (hi - lo) * torch.rand(B, generator=_gen(cfg.seed, "noise_std", device), device=device)
    else:
        nstd = torch.full((B,), float(cfg.noise_std), device=device)
    temperature: Optional[torch.Tensor]
    temperature_all = 1.0
    if isinstance(cfg.temperature, tuple):
        lo, hi = cfg.temperature
        temperature = (lo + (hi - lo) * torch.rand(B, generator=_gen(cfg.seed, "temperature", device),
                                                   device=device)).to(torch.float32)
    elif cfg.temperature == "half_0.7_1.0":
        temperature = torch.ones(B, dtype=torch.float32, device=device)
        temperature[: B // 2] = 0.7
    else:
        temperature = None
        temperature_all = float(cfg.temperature)
    tau_rows = temperature if temperature is not None else torch.full((B,), temperature_all, device=device)
    if cfg.ragged:
        draft_len = torch.randint(1, K + 1, (B,), generator=_gen(cfg.seed, "lengths", device),
                                  device=device, dtype=torch.int64).to(torch.int32)
    else:
        draft_len = None

    g_t, g_d = _gen(cfg.seed, "target", device), _gen(cfg.seed, "draft", device)
    g_p, g_pp = _gen(cfg.seed, "peaks", device), _gen(cfg.seed, "peak_perm", device)
    g_g = _gen(cfg.seed, "gumbel", device)
    heights = 8.0 * torch.arange(1, 9, device=device, dtype=torch.float32) ** (-2.0 / 3.0)
    tokens = torch.zeros((B, K), dtype=torch.int32, device=device)
    for b0 in range(0, B, CHUNK):
        b1 = min(B, b0 + CHUNK)
        n = b1 - b0
        t = torch.randn((n, K + 1, V), generator=g_t, device=device) * cfg.target_std
        if cfg.peaks and V >= 16:
            # 8 distinct ids per row: sorted draws from [0, V-8] plus offsets 0..7
            ids = torch.randint(0, V - 7, (n, K + 1, 8), generator=g_p, device=device).sort(dim=-1).values
            ids = ids + torch.arange(8, device=device)
            perm = torch.rand((n, K + 1, 8), generator=g_pp, device=device).argsort(dim=-1)
            t.scatter_add_(2, ids, heights[perm])
        target[b0:b1] = t.to(dt)
        if K == 0:
            continue
        d = t[:, :K] + torch.randn((n, K, V), generator=g_d, device=device) * nstd[b0:b1, None, None]
        d = d.to(dt)
        draft[b0:b1] = d
        if draft_mode == "argmax":
            tokens[b0:b1] = first_argmax(d.float()).to(torch.int32)
        else:
            e = torch.empty((n, K, V), device=device).exponential_(generator=g_g).clamp_min_(1e-30)
            key = d.float() / tau_rows[b0:b1, None, None] - e.log()
            tokens[b0:b1] = key.argmax(dim=-1).to(torch.int32)
        del t, d
    u_accept = open_uniform((B, K), _gen(cfg.seed, "u_accept", device), device)
    u_final = open_uniform((B,), _gen(cfg.seed, "u_final", device), device)
    return dict(cfg=cfg, target=target, draft=draft, ld=ld, draft_tokens=tokens, draft_len=draft_len,
                temperature=temperature, temperature_all=temperature_all,
                u_accept=u_accept, u_final=u_final)


def checksum(t: Optional[torch.Tensor]) -> Optional[int]:
    """64-bit wrap-around sum of the tensor's raw 16- or 32-bit words."""
    if t is None:
        return None
    t = t.contiguous()
    w = t.view(torch.int16) if t.element_size() == 2 else t.view(torch.int32)
    return int(w.to(torch.int64).sum().item())


def rows_read(cfg: Config, draft_len: Optional[torch.Tensor]) -> int:
    """Logit rows the method must read: sum_b (2 * len_b + 1)."""
    if draft_len is None:
        return cfg.B * (2 * cfg.K + 1)
    return int((2 * draft_len.to(torch.int64) + 1).sum().item())
