"""Seeded synthetic inputs shaped like one Swimba layer.

This module only draws random tensors; it contains none of the method's
arithmetic and is the one piece of code that both the CPU oracle's tests and
the CUDA path's tests and benchmark use, so that both sides see identical
arrays.  Everything is generated on the host with a torch CPU generator in a
fixed draw order (u, x, dt, W_r, W_e, A, dt_bias, D, h0).

The paper's own workloads (a 52-layer hybrid language model served on public
evaluation suites) need weights and datasets that are not available; these
tensors take the layer's shapes and the init distributions of Mamba-2 style
layers and stand in for them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    name: str
    dtype: str          # "fp32" or "bf16" (activations + router/expert weights)
    B: int              # sequences
    L: int              # tokens per sequence (1 for decode)
    F: int              # d_model: width of the token features the router/experts read
    H: int              # heads
    P: int              # head dim
    N: int              # state size
    G: int              # B/C groups
    E: int              # experts
    k: int              # active experts per token
    Q: int              # chunk length
    router_std: Optional[float] = None   # std of W_r entries (default 0.02)
    h0_std: float = 0.0                  # std of the initial state (0 -> none)
    steps: int = 1                       # decode steps (decode configs)

    @property
    def S(self) -> int:
        return 2 * self.G * self.N

    @property
    def tokens(self) -> int:
        return self.B * self.L


# The five workloads the benchmark and the parity tests use.
CONFIGS: Dict[str, LayerConfig] = {
    "tiny_fp32": LayerConfig("tiny_fp32", "fp32", 1, 256, 256, 8, 64, 16, 1, 4, 1, 64),
    "small_lm": LayerConfig("small_lm", "bf16", 8, 2048, 768, 24, 64, 128, 1, 8, 2, 256),
    "mid": LayerConfig("mid", "bf16", 4, 8192, 2048, 64, 64, 128, 1, 8, 2, 256,
                       router_std=0.25 / math.sqrt(2048)),
    "long_seq": LayerConfig("long_seq", "bf16", 1, 65536, 1024, 32, 64, 128, 1, 16, 2, 256),
    "decode": LayerConfig("decode", "bf16", 128, 1, 2048, 64, 64, 128, 1, 8, 2, 256,
                          h0_std=0.1, steps=512),
}
CONFIG_ORDER = ["tiny_fp32", "small_lm", "mid", "long_seq", "decode"]


def torch_dtype(name: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def make_weights(cfg: LayerConfig, gen: torch.Generator) -> Dict[str, torch.Tensor]:
    dt_ = torch_dtype(cfg.dtype)
    rstd = cfg.router_std if cfg.router_std is not None else 0.02
    W_r = (torch.randn(cfg.E, cfg.F, generator=gen) * rstd).to(dt_)
    W_e = (torch.randn(cfg.E, cfg.S, cfg.F, generator=gen) * 0.02).to(dt_)
    # A_h = -exp(U(log 1, log 16))
    A = -torch.exp(torch.rand(cfg.H, generator=gen) * math.log(16.0))
    # softplus(dt_bias) ~ logU(1e-3, 1e-1)
    dt0 = torch.exp(torch.rand(cfg.H, generator=gen) * (math.log(1e-1) - math.log(1e-3))
                    + math.log(1e-3))
    dt_bias = dt0 + torch.log(-torch.expm1(-dt0))
    D = 1.0 + 0.1 * torch.randn(cfg.H, generator=gen)
    return dict(W_r=W_r, W_e=W_e, A=A.float(), dt_bias=dt_bias.float(), D=D.float())


def make_inputs(cfg: LayerConfig, seed: int = 0, with_dt: bool = True) -> Dict[str, torch.Tensor]:
    """All tensors of one forward call, on the host, in the config's dtypes."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    dt_ = torch_dtype(cfg.dtype)
    u = torch.randn(cfg.B, cfg.L, cfg.F, generator=gen).to(dt_)
    x = torch.randn(cfg.B, cfg.L, cfg.H, cfg.P, generator=gen).to(dt_)
    dt = 0.5 * torch.randn(cfg.B, cfg.L, cfg.H, generator=gen)
    out = dict(u=u, x=x, dt=dt.float() if with_dt else None)
    out.update(make_weights(cfg, gen))
    if cfg.h0_std > 0:
        out["h0"] = (cfg.h0_std * torch.randn(cfg.B, cfg.H, cfg.P, cfg.N, generator=gen)).float()
    else:
        out["h0"] = None
    return out


def make_decode_step_inputs(cfg: LayerConfig, gen: torch.Generator) -> Dict[str, torch.Tensor]:
    """Fresh per-step token tensors for a decode loop (weights/state made elsewhere)."""
    dt_ = torch_dtype(cfg.dtype)
    u = torch.randn(cfg.B, cfg.F, generator=gen).to(dt_)
    x = torch.randn(cfg.B, cfg.H, cfg.P, generator=gen).to(dt_)
    dt = (0.5 * torch.randn(cfg.B, cfg.H, generator=gen)).float()
    return dict(u=u, x=x, dt=dt)


def f64(t: Optional[torch.Tensor]):
    """Widen a host tensor to a float64 numpy array (exact for fp32 and bf16)."""
    if t is None:
        return None
    return t.detach().to(torch.float64).cpu().numpy()
