"""Seeded synthetic inputs for the LOT attention forward path.

This module holds no arithmetic of the method: it only draws tensors with the
shapes and value distributions of the five benchmark configurations, on the CPU
with a fixed torch generator, rounds them to the run dtype, and hands the same
rounded values to whoever asks (the CUDA path and the CPU checker alike).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch


@dataclass
class LotInputs:
    q: torch.Tensor          # [B,H,n,d] run dtype (CPU)
    k: torch.Tensor
    v: torch.Tensor
    z: torch.Tensor          # [H,r,d] float32
    beta: torch.Tensor       # [H,r] float32, rows on the simplex
    key_len: Optional[torch.Tensor]  # [B] int32 or None
    eps: float
    iters: int
    name: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def shape(self):
        B, H, n, d = self.q.shape
        return B, H, n, d, self.z.shape[1]

    def f64(self):
        """float64 numpy copies of the (already rounded) values."""
        cv = lambda t: t.to(torch.float64).numpy()
        return dict(q=cv(self.q), k=cv(self.k), v=cv(self.v), z=cv(self.z), beta=cv(self.beta),
                    key_len=None if self.key_len is None else self.key_len.numpy().astype(np.int32))


def _beta(gen, H, r):
    logits = torch.randn(H, r, generator=gen, dtype=torch.float32)
    return torch.softmax(logits, dim=-1).contiguous()


def make(B, H, n, d, r, *, seed, dtype=torch.float32, eps=0.1, iters=10, z_std=1.0,
         qk="normal", key_len_range=None, name=""):
    """Draw one problem.

    qk="normal":  Q,K,V ~ N(0,1) * d^-1/2.
    qk="mixture": Q,K from a 4-component equal-weight Gaussian mixture whose means are
                  N(0,(4/d) I) (shared by Q and K) with within-component std 0.5 d^-1/2;
                  V ~ N(0,1) * d^-1/2.
    Z ~ N(0, z_std^2) per head, float32; beta = softmax of N(0,1) logits, float32.
    key_len_range=(lo,hi): per-sequence valid key length, uniform integer in [lo,hi].
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(seed))
    sc = float(d) ** -0.5
    rn = lambda *s: torch.randn(*s, generator=gen, dtype=torch.float32)
    if qk == "normal":
        q, k = rn(B, H, n, d) * sc, rn(B, H, n, d) * sc
    elif qk == "mixture":
        means = rn(B, H, 4, d) * (2.0 * sc)
        def draw():
            comp = torch.randint(0, 4, (B, H, n), generator=gen)
            mu = torch.gather(means, 2, comp.unsqueeze(-1).expand(B, H, n, d))
            return mu + rn(B, H, n, d) * (0.5 * sc)
        q, k = draw(), draw()
    else:
        raise ValueError(qk)
    v = rn(B, H, n, d) * sc
    z = (rn(H, r, d) * float(z_std)).contiguous()
    beta = _beta(gen, H, r)
    key_len = None
    if key_len_range is not None:
        lo, hi = key_len_range
        key_len = torch.randint(lo, hi + 1, (B,), generator=gen).to(torch.int32)
    cast = lambda t: t.to(dtype).contiguous()
    return LotInputs(cast(q), cast(k), cast(v), z, beta, key_len, float(eps), int(iters), name,
                     dict(B=B, H=H, n=n, d=d, r=r, seed=seed, dtype=str(dtype).replace("torch.", ""), qk=qk))


def config(cfg: int, *, dtype=None, n=None, r=None, iters=None, eps=None, B=None, H=None, variant=0):
    """The five benchmark configurations (seed = 1000*cfg + variant; config 1 uses seed 0)."""
    bf, f32 = torch.bfloat16, torch.float32
    if cfg == 1:
        d = 16
        return make(B or 1, H or 1, n or 64, d, r or 8, seed=0 + variant, dtype=dtype or f32, eps=eps or 0.1,
                    iters=50 if iters is None else iters, z_std=d ** -0.5, name="cfg1-tiny")
    if cfg == 2:
        return make(B or 32, H or 3, n or 197, 64, r or 16, seed=2000 + variant, dtype=dtype or bf,
                    eps=eps or 0.1, iters=10 if iters is None else iters, name="cfg2-deit-tiny")
    if cfg == 3:
        nn = n or 512
        return make(B or 16, H or 12, nn, 64, r or 32, seed=3000 + variant, dtype=dtype or bf,
                    eps=eps or 0.05, iters=20 if iters is None else iters,
                    key_len_range=(nn // 2, nn), name="cfg3-bert-base")
    if cfg == 4:
        nn = n or 16384
        return make(B or 1, H or 16, nn, 64, r or 64, seed=4000 + variant, dtype=dtype or bf,
                    eps=eps or 0.1, iters=10 if iters is None else iters, name=f"cfg4-long-n{nn}")
    if cfg == 5:
        return make(B or 4, H or 8, n or 16384, 128, r or 64, seed=5000 + variant, dtype=dtype or bf,
                    eps=eps or 0.1, iters=20 if iters is None else iters, qk="mixture",
                    name=f"cfg5-stress-r{r or 64}")
    raise ValueError(cfg)


def cotangent(x: "LotInputs", seed: int = 1):
    """A seeded upstream gradient for the backward tests: N(0,1) of out's shape, rounded to the tensor dtype."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(x.meta["seed"]) * 7919 + int(seed))
    return torch.randn(x.q.shape, generator=gen, dtype=torch.float32).to(x.q.dtype).contiguous()
