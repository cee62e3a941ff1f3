"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and casts them: it contains none of the
operator's arithmetic, so the CUDA path's callers and the CPU oracle's callers
can both use it without sharing any of the method between them.

The paper's real workloads are activations of Wan video DiTs (81 frames -> 21
latent frames; 480p gives 21 x 30 x 52 = 32,760 tokens, 720p gives
21 x 45 x 80 = 75,600) and learned feature-map matrices; neither ships with
the paper, so these stand in for them:

  config 1  B=1 H=2  n=1024  d=64  fp32  q,k,v ~ N(0,1)
  config 2  B=1 H=12 n=32760 d=128 bf16  q,k,v ~ N(0,1)/sqrt(d)
  config 3  B=1 H=40 n=32760 d=128 bf16  as 2, and 5% of K's entries replaced by
                                          Student-t(3)/sqrt(d) (heavy tails)
  config 4  B=1 H=40 n=75600 d=128 bf16  as 2
  config 5  B=2 H=12 n=32760 d=128 bf16  as 2, 30 independent layers
  config 6  B=1 H=30 n=17776 d=64  bf16  as 2: the shape of CogVideoX-2B's joint text + video self-attention
                                          (30 heads of 64; 226 text tokens + 13 x 30 x 45 video tokens for 49 frames
                                          of 480 x 720); the paper names the model but prints none of its dimensions

W_q and W_k are drawn per head as N(0,1) / (sqrt(d) * sigma_x), sigma_x being the
standard deviation of the inputs, so that the logits x W have unit variance: phi
is then neither uniform nor one-hot.  Everything is drawn in fp32 from one CPU
generator per (config, layer) in the order q, k, v, W_q, W_k and cast once to
the storage type; both sides of a parity test consume those cast values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

SEED_BASE = 25100831


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    n: int
    d: int
    dtype: str          # "f32" or "bf16"
    unit_inputs: bool   # True: q,k,v ~ N(0,1); False: N(0,1)/sqrt(d)
    heavy_tail_k: bool  # 5% of K from Student-t(3)
    layers: int = 1


CONFIGS = {
    1: Workload("tiny", 1, 2, 1024, 64, "f32", True, False),
    2: Workload("wan1.3b-480p", 1, 12, 32760, 128, "bf16", False, False),
    3: Workload("wan14b-480p-heavytail", 1, 40, 32760, 128, "bf16", False, True),
    4: Workload("wan14b-720p", 1, 40, 75600, 128, "bf16", False, False),
    5: Workload("wan1.3b-cfg-pair-30-layers", 2, 12, 32760, 128, "bf16", False, False, 30),
    6: Workload("cogvideox2b-480x720-49f", 1, 30, 17776, 64, "bf16", False, False),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def make_inputs(config: int, layer: int = 0, *, B=None, H=None, n=None, d=None, dtype=None):
    """CPU tensors {q, k, v: [B,H,n,d]; Wq, Wk: [H,d,d/2]} for one layer of a config.

    Shape arguments override the config's own (same distributions, same seed), which is
    how the parity tests get reduced-size cases of each workload."""
    w = CONFIGS[config]
    B = w.B if B is None else B
    H = w.H if H is None else H
    n = w.n if n is None else n
    d = w.d if d is None else d
    dt = torch_dtype(w.dtype if dtype is None else dtype)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED_BASE + 1000 * config + layer)
    sigma_x = 1.0 if w.unit_inputs else 1.0 / math.sqrt(d)

    def draw(*shape):
        return torch.randn(*shape, generator=gen, dtype=torch.float32)

    q = draw(B, H, n, d) * sigma_x
    k = draw(B, H, n, d) * sigma_x
    v = draw(B, H, n, d) * sigma_x
    Wq = draw(H, d, d // 2) / (math.sqrt(d) * sigma_x)
    Wk = draw(H, d, d // 2) / (math.sqrt(d) * sigma_x)
    if w.heavy_tail_k:
        mask = torch.rand(B, H, n, d, generator=gen) < 0.05
        g0 = draw(B, H, n, d)
        chi = (draw(B, H, n, d) ** 2 + draw(B, H, n, d) ** 2 + draw(B, H, n, d) ** 2) / 3.0
        t3 = g0 / chi.sqrt()
        k = torch.where(mask, t3 * sigma_x, k)
    return {"q": q.to(dt), "k": k.to(dt), "v": v.to(dt), "Wq": Wq.to(dt), "Wk": Wk.to(dt)}
