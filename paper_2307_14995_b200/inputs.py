"""Seeded synthetic inputs for decayed causal linear attention.

This module only *draws data*: it holds none of the attention arithmetic and is
the one piece shared by the CUDA tests, the benchmark and the CPU oracle's
tests, so that every side sees the same input bits.

Value recipe (stands in for the activations of the paper's private corpus):
  * q, k = SiLU(z), z ~ N(0,1)  -- the token mixer feeds swish-activated
    projections into the attention product (Eq. 4);
  * v, dO ~ N(0,1);
  * the per-head decay follows Eq. 2, lambda_h = exp(-(8 h / H) (1 - l/L)),
    h = 0..H-1, with the layer position l/L given per workload;
  * everything is drawn in fp32 from ``torch.Generator('cpu')`` in the order
    q, k, v, dO and then rounded to the storage dtype (bf16 by
    round-to-nearest-even); consumers widen those rounded values exactly.

Shapes follow the paper's model table (385M / 1B / 7B variants) and its 8192
training length, as fixed by the five benchmark workloads below.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    d: int
    e: int
    in_dtype: torch.dtype
    l_over_L: float
    qk_scale: float = 1.0
    seed: int = 0
    decode_steps: int = 0  # >0: N is the prefill length, then that many recurrent steps

    @property
    def token_heads(self) -> int:
        return self.B * self.H * self.N


WORKLOADS: Dict[str, Workload] = {
    # fp32 reference case: lambda = {1, e^-2}; q,k divided by sqrt(64) in the generator
    "pr1_ref": Workload("pr1_ref", 1, 2, 256, 64, 64, torch.float32, 0.5, qk_scale=1.0 / 8.0),
    "385m": Workload("385m", 4, 16, 2048, 64, 64, torch.bfloat16, 0.25),
    "1b": Workload("1b", 2, 16, 8192, 128, 128, torch.bfloat16, 0.5),
    "7b_long": Workload("7b_long", 1, 32, 65536, 128, 128, torch.bfloat16, 0.9),
    "decode": Workload("decode", 64, 32, 4096, 128, 128, torch.bfloat16, 0.9, decode_steps=256),
}


def decay_rates(H: int, l_over_L: float) -> torch.Tensor:
    """Per-head decay of Eq. 2 as fp32 (the library takes lambda as fp32 data)."""
    h = torch.arange(H, dtype=torch.float64)
    lam = torch.exp(-(8.0 * h / H) * (1.0 - l_over_L))
    return lam.to(torch.float32)


def _silu(z: torch.Tensor) -> torch.Tensor:
    return z * torch.sigmoid(z)


def draw(shape, gen: torch.Generator, kind: str, dtype: torch.dtype, scale: float = 1.0) -> torch.Tensor:
    """One tensor: 'silu' = SiLU(N(0,1))*scale, 'normal' = N(0,1); rounded to dtype."""
    z = torch.randn(shape, generator=gen, dtype=torch.float32)
    if kind == "silu":
        z = _silu(z)
        if scale != 1.0:
            z = z * scale
    elif kind != "normal":
        raise ValueError(kind)
    return z.to(dtype).contiguous()


def make_qkvdo(B: int, H: int, N: int, d: int, e: int, *, dtype=torch.bfloat16, seed: int = 0,
               qk_scale: float = 1.0, with_do: bool = True, gen: Optional[torch.Generator] = None):
    """q,k [B,H,N,d], v,dO [B,H,N,e] on the CPU, drawn in that order from one generator."""
    if gen is None:
        gen = torch.Generator("cpu")
        gen.manual_seed(seed)
    q = draw((B, H, N, d), gen, "silu", dtype, qk_scale)
    k = draw((B, H, N, d), gen, "silu", dtype, qk_scale)
    v = draw((B, H, N, e), gen, "normal", dtype)
    do = draw((B, H, N, e), gen, "normal", dtype) if with_do else None
    return q, k, v, do


def make_state(B: int, H: int, d: int, e: int, *, seed: int = 1, scale: float = 1.0) -> torch.Tensor:
    """A random fp32 [B,H,d,e] tensor (used as kv_in / grad_kv_out in hand-over tests)."""
    gen = torch.Generator("cpu")
    gen.manual_seed(seed)
    return (torch.randn((B, H, d, e), generator=gen, dtype=torch.float32) * scale).contiguous()


def make_theta(H: int, d: int, *, seed: int = 2, base: float = 10000.0, jitter: float = 0.1) -> torch.Tensor:
    """Rotation angles for LRPE-d (Eq. 1), fp32 [H, d]: geometrically spaced frequencies base^(-i/d) (the usual
    initialisation of rotary-style encodings) times a seeded log-normal factor per (head, feature), standing in for
    values a short stretch of training would have moved them to."""
    gen = torch.Generator("cpu")
    gen.manual_seed(seed)
    i = torch.arange(d, dtype=torch.float64)
    freq = torch.pow(torch.tensor(base, dtype=torch.float64), -i / d)
    z = torch.randn((H, d), generator=gen, dtype=torch.float32).double()
    return (freq[None, :] * torch.exp(jitter * z)).float().contiguous()


def make_workload(name: str, *, B: Optional[int] = None, H: Optional[int] = None, N: Optional[int] = None):
    """Inputs of a named workload (optionally with reduced B/H/N for sampled checks).

    Returns a dict with q,k,v,do (CPU tensors in the workload's input dtype),
    lam (fp32 [H]) and the Workload record.  When H is reduced, the decay rates
    are still those of the first H heads of the full schedule.
    """
    w = WORKLOADS[name]
    Bx, Hx, Nx = B or w.B, H or w.H, N or w.N
    lam = decay_rates(w.H, w.l_over_L)[:Hx].contiguous()
    q, k, v, do = make_qkvdo(Bx, Hx, Nx, w.d, w.e, dtype=w.in_dtype, seed=w.seed, qk_scale=w.qk_scale)
    return {"q": q, "k": k, "v": v, "do": do, "lam": lam, "workload": w}


def make_decode_inputs(name: str = "decode", *, B: Optional[int] = None, H: Optional[int] = None,
                       prefill: Optional[int] = None, steps: Optional[int] = None):
    """Prefill q,k,v of length `prefill`, then per-step q,k,v [steps,B,H,d|e] (same generator)."""
    w = WORKLOADS[name]
    Bx, Hx = B or w.B, H or w.H
    P = prefill if prefill is not None else w.N
    S = steps if steps is not None else w.decode_steps
    gen = torch.Generator("cpu")
    gen.manual_seed(w.seed)
    lam = decay_rates(w.H, w.l_over_L)[:Hx].contiguous()
    q, k, v, _ = make_qkvdo(Bx, Hx, P, w.d, w.e, dtype=w.in_dtype, with_do=False, gen=gen)
    qs = draw((S, Bx, Hx, w.d), gen, "silu", w.in_dtype)
    ks = draw((S, Bx, Hx, w.d), gen, "silu", w.in_dtype)
    vs = draw((S, Bx, Hx, w.e), gen, "normal", w.in_dtype)
    return {"q": q, "k": k, "v": v, "qs": qs, "ks": ks, "vs": vs, "lam": lam, "workload": w}


def device_randn_like_workload(name: str, device, *, seed: int = 0):
    """Benchmark-only: the same distributions drawn on the GPU (different bits than
    the CPU generator; the timing legs do not compare values with the oracle)."""
    w = WORKLOADS[name]
    gen = torch.Generator(device)
    gen.manual_seed(seed)

    def silu(shape):
        z = torch.randn(shape, generator=gen, dtype=torch.float32, device=device)
        return (_silu(z) * w.qk_scale).to(w.in_dtype)

    def normal(shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32, device=device).to(w.in_dtype)

    q = silu((w.B, w.H, w.N, w.d))
    k = silu((w.B, w.H, w.N, w.d))
    v = normal((w.B, w.H, w.N, w.e))
    do = normal((w.B, w.H, w.N, w.e))
    return {"q": q, "k": k, "v": v, "do": do, "lam": decay_rates(w.H, w.l_over_L), "workload": w}
