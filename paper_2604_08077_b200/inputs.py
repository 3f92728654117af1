"""Seeded synthetic workloads for AdaS-Attn (shared by the tests, the bench and the oracle checks).

This module draws random tensors and nothing else: it contains none of the method's
arithmetic (no cube index formula, no pooling, no scoring, no selection).  The per-cube
structure of the keys is produced purely by *viewing* the raster video grid as
``[T/ct, ct, H/ch, ch, W/cw, cw]`` and broadcasting one offset vector over the three window
axes, so it does not depend on how any implementation numbers its cubes.

All tensors are drawn in fp32 on the CPU from ``torch.Generator(seed)``, then rounded to
bf16 exactly once.  The CUDA path consumes the bf16 bytes; the oracle consumes the same
values widened to fp32/fp64, so both sides see identical real numbers.

Layout of every returned tensor: raster order ``[B, S, heads, D]`` with
``S = n_prefix + T*H*W + n_text``; video token ``(t, y, x)`` sits at ``s = n_prefix + (t*H + y)*W + x``
and the text tokens follow the video tokens (Sec. 3.1 / Algorithm 1 of the paper: video cubes
first, text after them); ``n_prefix`` (0 in the benchmark configurations) text tokens may precede
the video, as a prompt does.  The grid need not be a multiple of the cube window.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Tuple

import torch


@dataclass
class Workload:
    """One AdaS-Attn problem instance (prefill), plus optional decode-step tensors."""

    name: str
    B: int
    T: int
    H: int
    W: int
    cube: Tuple[int, int, int]  # (ct, ch, cw)
    n_text: int
    Hq: int
    Hkv: int
    D: int
    top_p: float
    top_k: int = 0  # > 0: Top-K selection instead of Top-p
    n_prefix: int = 0  # text tokens before the video
    q: Optional[torch.Tensor] = None  # bf16 [B, S, Hq, D]   (None for cache-only workloads)
    k: Optional[torch.Tensor] = None  # bf16 [B, S, Hkv, D]
    v: Optional[torch.Tensor] = None  # bf16 [B, S, Hkv, D]
    # decode step (one new text token per sequence); None for prefill-only workloads
    q_new: Optional[torch.Tensor] = None  # bf16 [B, 1, Hq, D]
    k_new: Optional[torch.Tensor] = None  # bf16 [B, 1, Hkv, D]
    v_new: Optional[torch.Tensor] = None  # bf16 [B, 1, Hkv, D]
    meta: dict = field(default_factory=dict)

    @property
    def S_v(self) -> int:
        return self.T * self.H * self.W

    @property
    def S(self) -> int:
        return self.n_prefix + self.S_v + self.n_text

    @property
    def C(self) -> int:
        return self.cube[0] * self.cube[1] * self.cube[2]

    @property
    def N(self) -> int:
        ct, ch, cw = self.cube
        return (-(-self.T // ct)) * (-(-self.H // ch)) * (-(-self.W // cw))


def _gen(seed: int, device: str = "cpu") -> torch.Generator:
    """Seeded generator.  Tests draw on the CPU (the oracle reads the same bytes); the bench may
    draw the largest workloads directly on the GPU (same recipe, a different stream of draws)."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(g: torch.Generator, *shape: int, std: float = 1.0) -> torch.Tensor:
    x = torch.randn(*shape, generator=g, dtype=torch.float32, device=g.device)
    if std != 1.0:
        x.mul_(std)
    return x


def _add_cube_offsets(k_video: torch.Tensor, g: torch.Generator, T: int, H: int, W: int,
                      cube: Tuple[int, int, int], std: float) -> None:
    """In place: add one N(0, std^2 I) vector per (cube window, head) to video keys or queries.

    ``k_video`` is ``[B, T*H*W, heads, D]`` in raster order.
    """
    ct, ch, cw = cube
    B, _, Hkv, D = k_video.shape
    nT, nH, nW = -(-T // ct), -(-H // ch), -(-W // cw)         # windows along each axis (the last may be cut)
    off = _randn(g, B, nT, 1, nH, 1, nW, 1, Hkv, D, std=std)
    if (nT * ct, nH * ch, nW * cw) == (T, H, W):
        k_video.view(B, nT, ct, nH, ch, nW, cw, Hkv, D).add_(off)
    else:   # broadcast over whole windows, then keep the part of the grid that exists
        full = off.expand(B, nT, ct, nH, ch, nW, cw, Hkv, D).reshape(B, nT * ct, nH * ch, nW * cw, Hkv, D)
        k_video.view(B, T, H, W, Hkv, D).add_(full[:, :T, :H, :W])


def make_prefill(name: str, *, seed: int, B: int, T: int, H: int, W: int,
                 cube: Tuple[int, int, int], n_text: int, Hq: int, Hkv: int, D: int,
                 top_p: float, offset_std: float, with_q: bool = True,
                 device: str = "cpu", q_offset_std: float = 0.0, q_noise_std: float = 1.0,
                 n_prefix: int = 0) -> Workload:
    """i.i.d. N(0,1) Q/K/V; video K gets a per-cube shared offset of std ``offset_std``.

    ``q_offset_std`` > 0 additionally gives the video queries of one cube a shared offset (per query
    head) on top of their own N(0, q_noise_std^2) part: queries of a cube then score the cubes alike
    and select overlapping sets, the cohesion inside a spatio-temporal cube that the paper's
    partition assumes (Sec. 3.1).  Text queries stay N(0,1)."""
    g = _gen(seed, device)
    S_v = T * H * W
    S = S_v + n_text
    k = _randn(g, B, S, Hkv, D)
    v = _randn(g, B, S, Hkv, D)
    if offset_std > 0:
        _add_cube_offsets(k[:, :S_v], g, T, H, W, cube, offset_std)
    q = None
    if with_q:
        q = _randn(g, B, S, Hq, D)
        if q_offset_std > 0:
            if q_noise_std != 1.0:
                q[:, :S_v].mul_(q_noise_std)
            _add_cube_offsets(q[:, :S_v], g, T, H, W, cube, q_offset_std)
    if n_prefix > 0:   # drawn last, so that the video and text part equals the workload without a prefix
        k = torch.cat([_randn(g, B, n_prefix, Hkv, D), k], dim=1)
        v = torch.cat([_randn(g, B, n_prefix, Hkv, D), v], dim=1)
        if with_q:
            q = torch.cat([_randn(g, B, n_prefix, Hq, D), q], dim=1)
    if with_q:
        q = q.to(torch.bfloat16)
    return Workload(name=name, B=B, T=T, H=H, W=W, cube=cube, n_text=n_text, Hq=Hq, Hkv=Hkv,
                    D=D, top_p=top_p, n_prefix=n_prefix, q=q, k=k.to(torch.bfloat16), v=v.to(torch.bfloat16),
                    meta={"seed": seed, "offset_std": offset_std, "q_offset_std": q_offset_std})


def _static_dynamic_kv(g: torch.Generator, B: int, T: int, H: int, W: int,
                       cube: Tuple[int, int, int], Hkv: int, D: int, offset_std: float,
                       noise_std: float) -> Tuple[torch.Tensor, torch.Tensor]:
    """Video K/V whose first T/2 frames are static and whose last T/2 frames are i.i.d.

    Static half: one base frame (N(0,1); K additionally carries one offset per ch x cw patch
    block) repeated over time plus N(0, noise_std^2) noise per element.  Dynamic half:
    N(0,1) with a per-cube offset on K.
    """
    ct, ch, cw = cube
    Ts = T // 2
    Td = T - Ts
    # static half
    k0 = _randn(g, B, 1, H, W, Hkv, D)
    v0 = _randn(g, B, 1, H, W, Hkv, D)
    off0 = _randn(g, B, 1, H // ch, 1, W // cw, 1, Hkv, D, std=offset_std)
    k0.view(B, 1, H // ch, ch, W // cw, cw, Hkv, D).add_(off0)
    ks = k0.expand(B, Ts, H, W, Hkv, D) + _randn(g, B, Ts, H, W, Hkv, D, std=noise_std)
    vs = v0.expand(B, Ts, H, W, Hkv, D) + _randn(g, B, Ts, H, W, Hkv, D, std=noise_std)
    # dynamic half
    kd = _randn(g, B, Td * H * W, Hkv, D)
    vd = _randn(g, B, Td * H * W, Hkv, D)
    _add_cube_offsets(kd, g, Td, H, W, cube, offset_std)
    k = torch.cat([ks.reshape(B, Ts * H * W, Hkv, D), kd], dim=1)
    v = torch.cat([vs.reshape(B, Ts * H * W, Hkv, D), vd], dim=1)
    return k, v


def make_heterogeneous(name: str, *, seed: int, B: int, T: int, H: int, W: int,
                       cube: Tuple[int, int, int], n_text: int, Hq: int, Hkv: int, D: int,
                       top_p: float, offset_std: float = 1.5, noise_std: float = 0.05,
                       with_q: bool = True, with_decode_token: bool = False,
                       device: str = "cpu") -> Workload:
    """Half-static / half-dynamic video (load-imbalance stress), optional text and decode token."""
    g = _gen(seed, device)
    assert T % 2 == 0 and (T // 2) % cube[0] == 0
    k, v = _static_dynamic_kv(g, B, T, H, W, cube, Hkv, D, offset_std, noise_std)
    if n_text > 0:
        k = torch.cat([k, _randn(g, B, n_text, Hkv, D)], dim=1)
        v = torch.cat([v, _randn(g, B, n_text, Hkv, D)], dim=1)
    q = _randn(g, B, T * H * W + n_text, Hq, D).to(torch.bfloat16) if with_q else None
    wl = Workload(name=name, B=B, T=T, H=H, W=W, cube=cube, n_text=n_text, Hq=Hq, Hkv=Hkv, D=D,
                  top_p=top_p, q=q, k=k.to(torch.bfloat16), v=v.to(torch.bfloat16),
                  meta={"seed": seed, "offset_std": offset_std, "noise_std": noise_std})
    if with_decode_token:
        wl.q_new = _randn(g, B, 1, Hq, D).to(torch.bfloat16)
        wl.k_new = _randn(g, B, 1, Hkv, D).to(torch.bfloat16)
        wl.v_new = _randn(g, B, 1, Hkv, D).to(torch.bfloat16)
    return wl


# --------------------------------------------------------------------------------------
# The five benchmark configurations (seed = 1000 * config + variant) and scaled-down twins.
# --------------------------------------------------------------------------------------

def config1(variant: int = 0) -> Workload:
    """Tiny prefill: 8x8x8 video, cube 2x4x4 (32 tokens, 16 cubes), 32 text, 4/4 heads, D=64."""
    return make_prefill("cfg1_tiny", seed=1000 + variant, B=1, T=8, H=8, W=8, cube=(2, 4, 4),
                        n_text=32, Hq=4, Hkv=4, D=64, top_p=0.9, offset_std=2.0)


def config2(variant: int = 0, top_p: float = 0.9, device: str = "cpu") -> Workload:
    """Qwen2-7B-shaped layer: 64x16x16 video, cube 4x4x4, 128 text, 28/4 heads, D=128."""
    return make_prefill("cfg2_qwen7b_16k", seed=2000 + variant, B=1, T=64, H=16, W=16,
                        cube=(4, 4, 4), n_text=128, Hq=28, Hkv=4, D=128, top_p=top_p,
                        offset_std=1.5, device=device)


def config2_cohesive(variant: int = 0, top_p: float = 0.9, q_offset_std: float = 1.0,
                     q_noise_std: float = 0.25, cube: Tuple[int, int, int] = (4, 4, 4),
                     device: str = "cpu") -> Workload:
    """Config-2 shapes with cohesive queries: the video queries of a cube share an offset of std
    ``q_offset_std`` per query head and an own part of std ``q_noise_std``, so the rows of a query
    tile select overlapping cube sets and the tile's union of selected blocks is far smaller than the
    whole prefix."""
    return make_prefill("cfg2_cohesive_q", seed=2500 + variant, B=1, T=64, H=16, W=16,
                        cube=cube, n_text=128, Hq=28, Hkv=4, D=128, top_p=top_p,
                        offset_std=1.5, device=device, q_offset_std=q_offset_std,
                        q_noise_std=q_noise_std)


def config3(sigma: float = 1.5, top_p: float = 0.9, device: str = "cpu") -> Workload:
    """Sweep: 256x16x16 video (1024 cubes), 256 text; sigma in {0.5,1.5,3.0}; p in {.5,.7,.9,.95,1}."""
    variant = {0.5: 0, 1.5: 1, 3.0: 2}[float(sigma)]
    return make_prefill(f"cfg3_sweep_s{sigma}_p{top_p}", seed=3000 + variant, B=1, T=256, H=16,
                        W=16, cube=(4, 4, 4), n_text=256, Hq=28, Hkv=4, D=128, top_p=top_p,
                        offset_std=float(sigma), device=device)


def config4(variant: int = 0, device: str = "cpu") -> Workload:
    """Heterogeneous complexity: 512x16x16 video (2048 cubes), first half static, no text."""
    return make_heterogeneous("cfg4_hetero_128k", seed=4000 + variant, B=1, T=512, H=16, W=16,
                              cube=(4, 4, 4), n_text=0, Hq=28, Hkv=4, D=128, top_p=0.9,
                              device=device)


def config5(variant: int = 0, B: int = 16, device: str = "cpu") -> Workload:
    """Decode: B sequences, 131072-token video cache (cfg-4 distribution) + 512 text + 1 new token."""
    return make_heterogeneous("cfg5_decode_128k", seed=5000 + variant, B=B, T=512, H=16, W=16,
                              cube=(4, 4, 4), n_text=512, Hq=28, Hkv=4, D=128, top_p=0.9,
                              with_q=False, with_decode_token=True, device=device)


def small_prefill(seed: int = 7, *, B: int = 1, T: int = 8, H: int = 8, W: int = 8,
                  cube: Tuple[int, int, int] = (4, 4, 4), n_text: int = 40, Hq: int = 4,
                  Hkv: int = 2, D: int = 128, top_p: float = 0.9,
                  offset_std: float = 1.5, n_prefix: int = 0) -> Workload:
    """A scaled-down prefill problem for element-by-element parity (several tiles, ragged text)."""
    return make_prefill("small_prefill", seed=seed, B=B, T=T, H=H, W=W, cube=cube, n_text=n_text,
                        Hq=Hq, Hkv=Hkv, D=D, top_p=top_p, offset_std=offset_std, n_prefix=n_prefix)


def small_decode(seed: int = 11, *, B: int = 2, T: int = 16, H: int = 8, W: int = 8,
                 cube: Tuple[int, int, int] = (4, 4, 4), n_text: int = 37, Hq: int = 8,
                 Hkv: int = 2, D: int = 128, top_p: float = 0.9) -> Workload:
    """A scaled-down decode problem (cfg-5 distribution)."""
    return make_heterogeneous("small_decode", seed=seed, B=B, T=T, H=H, W=W, cube=cube,
                              n_text=n_text, Hq=Hq, Hkv=Hkv, D=D, top_p=top_p, with_q=False,
                              with_decode_token=True)
