"""Seeded synthetic inputs shaped like the paper's prefill workloads.

This module holds no arithmetic of the method: it only draws N(0,1) tensors,
scales a few K channels to mimic the head-invariant K outlier stripe described
in the paper's outlier analysis, and names the five evaluation configurations.
Both the CUDA path's tests and the CPU oracle's tests draw inputs from here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import torch


@dataclass(frozen=True)
class Config:
    name: str
    B: int
    Hq: int
    Hkv: int
    N: int
    d: int
    causal: bool
    dtype: str              # "fp16" | "bf16"
    outlier_channels: int   # K channels per KV head that are scaled
    outlier_gain: float
    smooth_mode: int        # 0 bypass, 1 strong (alpha .5), 2 mild (alpha .25)
    Br: int
    Bc: int              # key-tile width of the online softmax (part of the result); 64 is the fastest path
    seed: int = 0
    fixed_outliers: tuple = ()   # explicit channel list (same for every head)
    cal_samples: int = 4
    cal_tokens: int = 128


CONFIGS = {
    # Tiny: fp16, four fixed outlier channels, 64x64 tiles, 4 calibration draws
    "C1": Config("C1-tiny", 1, 1, 1, 128, 128, False, "fp16", 4, 20.0, 1, 64, 64,
                 fixed_outliers=(3, 17, 64, 101), cal_samples=4, cal_tokens=128),
    # Qwen3-8B-shaped GQA prefill, 4 of 128 K channels x20 per KV head
    "C2": Config("C2-qwen3-8b-4k", 1, 32, 8, 4096, 128, True, "bf16", 4, 20.0, 1, 128, 64,
                 cal_samples=32, cal_tokens=1024),
    # LLaMA3.1-8B-shaped, no outliers, smoothing bypassed
    "C3": Config("C3-llama31-8b-8k", 1, 32, 8, 8192, 128, True, "bf16", 0, 1.0, 0, 128, 64),
    # Gemma2-9B-shaped, d=256, 2 of 256 channels x8, mild smoothing
    "C4": Config("C4-gemma2-9b-8k", 1, 16, 8, 8192, 256, True, "bf16", 2, 8.0, 2, 128, 64,
                 cal_samples=8, cal_tokens=1024),
    # sequence sweep base point (N and causal are overridden by the caller)
    "C5": Config("C5-sweep", 4, 32, 8, 1024, 128, True, "bf16", 4, 20.0, 1, 128, 64,
                 cal_samples=8, cal_tokens=1024),
}


def config(name: str, **over) -> Config:
    return replace(CONFIGS[name], **over)


def torch_dtype(cfg: Config):
    return torch.float16 if cfg.dtype == "fp16" else torch.bfloat16


def outlier_channels(cfg: Config, g: int):
    """Channel indices of KV head g whose K values are multiplied by outlier_gain."""
    if cfg.fixed_outliers:
        return list(cfg.fixed_outliers)
    if cfg.outlier_channels == 0:
        return []
    gen = torch.Generator().manual_seed(100 + g)
    return torch.randperm(cfg.d, generator=gen)[: cfg.outlier_channels].tolist()


def _draw(shape, gen, dt):
    return torch.randn(shape, generator=gen, dtype=torch.float32).to(dt)


def _apply_outliers(cfg: Config, k: torch.Tensor):
    # k [..., Hkv, N, d]
    for g in range(cfg.Hkv):
        ch = outlier_channels(cfg, g)
        if ch:
            k[..., g, :, ch] = (k[..., g, :, ch].float() * cfg.outlier_gain).to(k.dtype)
    return k


def make_qkv(cfg: Config, seed: int | None = None):
    """Q [B,Hq,N,d], K,V [B,Hkv,N,d] on the CPU in the config's 16-bit dtype."""
    gen = torch.Generator().manual_seed(cfg.seed if seed is None else seed)
    dt = torch_dtype(cfg)
    q = _draw((cfg.B, cfg.Hq, cfg.N, cfg.d), gen, dt)
    k = _draw((cfg.B, cfg.Hkv, cfg.N, cfg.d), gen, dt)
    v = _draw((cfg.B, cfg.Hkv, cfg.N, cfg.d), gen, dt)
    return q, _apply_outliers(cfg, k), v


def make_calibration(cfg: Config, samples: int | None = None, tokens: int | None = None):
    """Calibration activations: q_cal [S,Hq,Ncal,d], k_cal [S,Hkv,Ncal,d].

    Sample n uses seed n+1, the same distribution and outlier channels as make_qkv."""
    S = cfg.cal_samples if samples is None else samples
    T = cfg.cal_tokens if tokens is None else tokens
    dt = torch_dtype(cfg)
    qs, ks = [], []
    for n in range(S):
        gen = torch.Generator().manual_seed(n + 1)
        qs.append(_draw((cfg.Hq, T, cfg.d), gen, dt))
        ks.append(_apply_outliers(cfg, _draw((cfg.Hkv, T, cfg.d), gen, dt)))
    return torch.stack(qs), torch.stack(ks)


def make_qkv_device(cfg: Config, device, seed: int | None = None):
    """Same distribution drawn on the device (for sizes too large to draw on the host).

    The values differ from make_qkv (a different generator).  Used for timing and for parity on sampled
    rows at sizes where only those rows and their K/V head are copied back to the host."""
    gen = torch.Generator(device=device).manual_seed(cfg.seed if seed is None else seed)
    dt = torch_dtype(cfg)

    def draw(shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32, device=device).to(dt)

    q = draw((cfg.B, cfg.Hq, cfg.N, cfg.d))
    k = draw((cfg.B, cfg.Hkv, cfg.N, cfg.d))
    v = draw((cfg.B, cfg.Hkv, cfg.N, cfg.d))
    return q, _apply_outliers(cfg, k), v
