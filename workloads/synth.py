"""Seeded Q/K/V draws for the workloads.

Everything is drawn with torch's generator on the requested device, in fp32,
given the structure a model would have applied before attention (rotary
rotation, heavy-hitter direction), then rounded to fp16.  The consumer copies
the tensors wherever it needs them, so the CUDA library and the CPU oracle see
bit-identical fp16 inputs.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from .configs import Workload

_KIND = {"q": 1, "k": 2, "v": 3, "hh_dir": 4, "hh_mask": 5}


def _gen(wl: Workload, layer: int, kind: str, step: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    seed = (wl.data_seed * 1_000_003 + layer) * 1_000_033 + step * 16 + _KIND[kind]
    g.manual_seed(seed & 0x7FFFFFFFFFFFFFFF)
    return g


def _randn(shape, g, device):
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def _rotary(x: torch.Tensor, positions: torch.Tensor, rot_dims: int) -> torch.Tensor:
    """Rotate interleaved pairs of the first rot_dims features by position * base^(-2i/rot_dims)."""
    if rot_dims <= 0:
        return x
    half = rot_dims // 2
    inv_freq = 10000.0 ** (-torch.arange(half, device=x.device, dtype=torch.float32) * 2.0 / rot_dims)
    ang = positions.to(torch.float32)[..., None] * inv_freq            # [..., half]
    cos, sin = torch.cos(ang), torch.sin(ang)
    xr = x[..., :rot_dims]
    even, odd = xr[..., 0::2], xr[..., 1::2]
    rot = torch.stack((even * cos - odd * sin, even * sin + odd * cos), dim=-1).flatten(-2)
    return torch.cat((rot, x[..., rot_dims:]), dim=-1)


def _heavy_direction(wl: Workload, layer: int, device) -> torch.Tensor:
    """Per (batch, key/value head) unit vector along which heavy-hitter keys are shifted."""
    e = _randn((wl.batch, wl.kv_heads, wl.head_dim), _gen(wl, layer, "hh_dir", 0, device), device)
    return e / e.norm(dim=-1, keepdim=True)


def _heavy_amplitude(wl: Workload) -> float:
    # (q + a e).(k + a e) / sqrt(d) gains a^2 / sqrt(d) on a heavy key: choose a so that equals heavy_logit
    return math.sqrt(wl.heavy_logit * math.sqrt(wl.head_dim))


def _per_query_head(wl: Workload, e: torch.Tensor) -> torch.Tensor:
    """[B, Hkv, ...] -> [B, H, ...]: every query head of a group sees its key/value head's entry."""
    return e.repeat_interleave(wl.group, dim=1) if wl.group > 1 else e


def make_prompt(wl: Workload, layer: int, device="cpu"):
    """Prompt tensors of one layer: Q fp16 [B, H, n, d]; K, V fp16 [B, Hkv, n, d] (Hkv = H without shared heads)."""
    B, H, Hkv, n, d = wl.batch, wl.n_heads, wl.kv_heads, wl.prompt_len, wl.head_dim
    q = _randn((B, H, n, d), _gen(wl, layer, "q", 0, device), device)
    k = _randn((B, Hkv, n, d), _gen(wl, layer, "k", 0, device), device)
    v = _randn((B, Hkv, n, d), _gen(wl, layer, "v", 0, device), device)
    if wl.heavy_frac > 0:
        e = _heavy_direction(wl, layer, device)[:, :, None, :]
        a = _heavy_amplitude(wl)
        mask = torch.rand((B, Hkv, n), generator=_gen(wl, layer, "hh_mask", 0, device), device=device) < wl.heavy_frac
        q = q + a * _per_query_head(wl, e)
        k = k + a * e * mask[..., None].to(torch.float32)
    if wl.positional == "rotary" and not wl.rotary_in_library:
        pos = torch.arange(n, device=device)
        q = _rotary(q, pos, wl.rotary_dims)
        k = _rotary(k, pos, wl.rotary_dims)
    return q.half().contiguous(), k.half().contiguous(), v.half().contiguous()


def make_step(wl: Workload, layer: int, step: int, device="cpu", prompt_len: int | None = None):
    """Decode-step tensors of one layer: q fp16 [B, H, d]; k_new, v_new fp16 [B, Hkv, d]; step = 1..T."""
    B, H, Hkv, d = wl.batch, wl.n_heads, wl.kv_heads, wl.head_dim
    n = wl.prompt_len if prompt_len is None else prompt_len
    q = _randn((B, H, d), _gen(wl, layer, "q", step, device), device)
    k = _randn((B, Hkv, d), _gen(wl, layer, "k", step, device), device)
    v = _randn((B, Hkv, d), _gen(wl, layer, "v", step, device), device)
    if wl.heavy_frac > 0:
        e = _heavy_direction(wl, layer, device)
        a = _heavy_amplitude(wl)
        mask = torch.rand((B, Hkv), generator=_gen(wl, layer, "hh_mask", step, device), device=device) < wl.heavy_frac
        q = q + a * _per_query_head(wl, e)
        k = k + a * e * mask[..., None].to(torch.float32)
    if wl.positional == "rotary" and not wl.rotary_in_library:
        pos = torch.full((1,), n + step - 1, device=device)
        q = _rotary(q, pos, wl.rotary_dims)
        k = _rotary(k, pos, wl.rotary_dims)
    return q.half().contiguous(), k.half().contiguous(), v.half().contiguous()


def unit_list(wl: Workload, layer: int | None = None) -> np.ndarray:
    """All (layer, batch, key/value head) triples of the workload (or of one layer), int32 [U, 3]."""
    layers = range(wl.n_layers) if layer is None else [layer]
    out = [(l, b, h) for l in layers for b in range(wl.batch) for h in range(wl.kv_heads)]
    return np.asarray(out, dtype=np.int32).reshape(-1, 3)


def sample_units(wl: Workload, count: int, seed: int = 0, layer: int | None = None) -> np.ndarray:
    """A seeded sample (without replacement, sorted) of the workload's units."""
    units = unit_list(wl, layer)
    if count >= units.shape[0]:
        return units
    rng = np.random.default_rng(seed)
    idx = np.sort(rng.choice(units.shape[0], size=count, replace=False))
    return units[idx]
