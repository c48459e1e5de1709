"""Seeded synthetic inputs for the SWAA attention path.

This module only draws random tensors with the shapes, value distributions and
structure of the five benchmark workloads; it holds none of the method's
arithmetic (no masks, no softmax) and is the one piece that both the GPU tests
and the CPU oracle's callers may share.  Everything is bf16, i.i.d. N(0,1),
drawn with a seeded ``torch.Generator`` on the requested device (CPU and CUDA
generators give different bits for the same seed, which is fine: the very same
tensor is handed to both sides of a comparison).

The paper's own timing run used random input data on a 128k-token prompt
(App. D); its accuracy benchmarks use 16k-128k contexts (Sec. 4.1.2).  These
generators stand in for those workloads.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch


@dataclass(frozen=True)
class PrefillConfig:
    name: str
    seqlens: tuple          # per-sequence lengths (packed batch)
    Hq: int
    Hkv: int
    D: int
    window: int
    n_sink: int
    is_full: bool = False
    seed: int = 0
    sink_shift: float = 0.0  # cfg2: K row 0 of each kv-head shifted by this much along a random unit direction

    @property
    def T(self) -> int:
        return int(sum(self.seqlens))

    @property
    def B(self) -> int:
        return len(self.seqlens)


@dataclass(frozen=True)
class DecodeConfig:
    name: str
    B: int
    Lmax: int
    Hq: int
    Hkv: int
    D: int
    window: int
    n_sink: int
    seed: int = 0
    seqlens: tuple = field(default=())  # empty: every sequence is Lmax long


def cfg_tiny() -> PrefillConfig:
    """Workload 1: tiny SWA+sink prefill."""
    return PrefillConfig("cfg1_tiny_swa_sink", (1024,), 4, 2, 64, 128, 4, False, seed=1)


def cfg_long(L: int = 32768, is_full: bool = False, window: int = 2048, n_sink: int = 4) -> PrefillConfig:
    """Workload 2: long-context SWA prefill, K row 0 shifted so the sink draws attention mass."""
    return PrefillConfig("cfg2_long_swa" if not is_full else "cfg2_long_full", (L,), 32, 8, 128, window, n_sink,
                         is_full, seed=2, sink_shift=3.0)


def cfg_stack_layer(layer: int, L: int = 131072) -> PrefillConfig:
    """Workload 3: layer `layer` of the 36-layer interleaved stack (mask policy comes from the schedule)."""
    return PrefillConfig(f"cfg3_layer{layer}", (L,), 32, 8, 128, 4096, 64, False, seed=3000 + layer)


def cfg_decode(B: int = 16, Lmax: int = 65536) -> DecodeConfig:
    """Workload 4: decode, one query token per sequence against a long cache."""
    return DecodeConfig("cfg4_decode", B, Lmax, 32, 8, 128, 4096, 4, seed=4)


def varlen_lengths(n: int = 8, lo: int = 4096, hi: int = 65536, seed: int = 5) -> tuple:
    return tuple(int(x) for x in np.random.default_rng(seed).integers(lo, hi + 1, n))


def cfg_varlen(lengths: tuple | None = None) -> PrefillConfig:
    """Workload 5: packed varlen prefill batch."""
    if lengths is None:
        lengths = varlen_lengths()
    return PrefillConfig("cfg5_varlen", tuple(lengths), 64, 8, 128, 8192, 4, False, seed=5)


def _randn_bf16(shape, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)


def make_prefill_inputs(cfg: PrefillConfig, device="cpu"):
    """Returns (q [T,Hq,D], k [T,Hkv,D], v [T,Hkv,D], cu_seqlens int32 [B+1]) on `device`; draw order Q, K, V."""
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed)
    T = cfg.T
    q = _randn_bf16((T, cfg.Hq, cfg.D), gen, device)
    if cfg.sink_shift != 0.0 and T > 0:
        k32 = torch.randn((T, cfg.Hkv, cfg.D), generator=gen, device=device, dtype=torch.float32)
        u = torch.randn((cfg.Hkv, cfg.D), generator=gen, device=device, dtype=torch.float32)
        u = u / u.norm(dim=-1, keepdim=True)
        starts = np.concatenate([[0], np.cumsum(cfg.seqlens)[:-1]])
        for s, n in zip(starts, cfg.seqlens):
            if n > 0:
                k32[int(s)] += cfg.sink_shift * u
        k = k32.to(torch.bfloat16)
        del k32
    else:
        k = _randn_bf16((T, cfg.Hkv, cfg.D), gen, device)
    v = _randn_bf16((T, cfg.Hkv, cfg.D), gen, device)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(cfg.seqlens)]).astype(np.int32), device=device)
    return q, k, v, cu


def make_decode_inputs(cfg: DecodeConfig, device="cpu"):
    """Returns (q [B,Hq,D], kcache, vcache [B,Lmax,Hkv,D], seqlens int32 [B]) on `device`."""
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed)
    q = _randn_bf16((cfg.B, cfg.Hq, cfg.D), gen, device)
    kc = torch.empty((cfg.B, cfg.Lmax, cfg.Hkv, cfg.D), dtype=torch.bfloat16, device=device)
    vc = torch.empty_like(kc)
    for b in range(cfg.B):  # per-sequence draws keep the fp32 temporary small
        kc[b] = _randn_bf16((cfg.Lmax, cfg.Hkv, cfg.D), gen, device)
    for b in range(cfg.B):
        vc[b] = _randn_bf16((cfg.Lmax, cfg.Hkv, cfg.D), gen, device)
    sl = cfg.seqlens if len(cfg.seqlens) else (cfg.Lmax,) * cfg.B
    seqlens = torch.tensor(sl, dtype=torch.int32, device=device)
    return q, kc, vc, seqlens


def to_f32_numpy(t: torch.Tensor) -> np.ndarray:
    """Exact float32 copy of a bf16 tensor on the host (what the oracle consumes)."""
    return t.detach().to("cpu").to(torch.float32).numpy()
