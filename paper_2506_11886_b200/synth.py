"""Seeded synthetic inputs for the hybrid-KV decode path.

This module holds NO arithmetic of the method (no basis, no projection, no
attention): it only draws index sets, K/V streams, queries and appended tokens
with the value distributions of the benchmark configurations, so that the CUDA
library and the CPU oracle can be fed identical bits.  It is the only module
both sides may import.

Recipe (per layer; every tensor has its own seed derived from ``seed``):
  * index sets: per (KV head, K|V) a seeded random subset of ``n_full`` of the
    ``d`` head dims is kept full, sorted ascending; the rest is compressed;
  * kept dims: i.i.d. N(0, 1) per token;
  * compressed dims, per (batch row, KV head, dim): a sum of 8 sinusoids over
    the absolute token index t,  x_t = sum_i a_i cos(2 pi f_i t / T + psi_i)
    + N(0, 0.05),  a_i ~ U(0.25, 0.75), psi_i ~ U(0, 2 pi), and f_i either an
    integer in [1, k) ("grid", in band) or a real in (0, k) ("offgrid", leaks
    across bins);
  * q: N(0, sigma = d^-1/2), used with softmax_scale = 1 so logits have unit scale;
  * appended tokens continue the same streams at t = L, L + 1, ...
Values are rounded once to the storage dtype; those bits go to both sides.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace

import torch


@dataclass(frozen=True)
class Shape:
    """One benchmark configuration of the path (names follow the paper)."""
    name: str
    B: int
    layers: int
    Hq: int
    Hkv: int
    d: int
    L: int                 # prefill length
    dtype: str             # "f32" | "bf16"  (storage of K/V/q/out)
    n_full_k: int
    n_full_v: int
    M: int                 # 2k real coefficients
    T: int                 # period of the translated window
    L_init: int
    L_local: int
    decode_steps: int = 1
    softmax_scale: float = 1.0
    mid_classes: int = 0   # 0: choose T / k (one residue class per FFT point)

    @property
    def k(self) -> int:
        return self.M // 2

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def with_(self, **kw) -> "Shape":
        return replace(self, **kw)


# The five configurations of the benchmark description.  Window sizes 4 / 1024
# and k = 512 are the paper's (Sec. 4.1); where the description is silent the
# values are the ones listed in the design notes.
CONFIGS = {
    0: Shape("cfg0_toy_f32", B=1, layers=1, Hq=4, Hkv=1, d=128, L=1024, dtype="f32",
             n_full_k=32, n_full_v=32, M=64, T=1024, L_init=0, L_local=0),
    1: Shape("cfg1_llama31_8b_32k", B=1, layers=1, Hq=32, Hkv=8, d=128, L=32768, dtype="bf16",
             n_full_k=32, n_full_v=32, M=1024, T=32768, L_init=4, L_local=1024, decode_steps=1000),
    2: Shape("cfg2_compress_32layers", B=1, layers=32, Hq=32, Hkv=8, d=128, L=32768, dtype="bf16",
             n_full_k=32, n_full_v=32, M=1024, T=32768, L_init=4, L_local=1024),
    3: Shape("cfg3_llama2_7b_mha_b8", B=8, layers=32, Hq=32, Hkv=32, d=128, L=4096, dtype="bf16",
             n_full_k=48, n_full_v=48, M=256, T=4096, L_init=4, L_local=1024, decode_steps=512),
    4: Shape("cfg4_128k_b4", B=4, layers=32, Hq=32, Hkv=8, d=128, L=131072, dtype="bf16",
             n_full_k=32, n_full_v=32, M=2048, T=131072, L_init=4, L_local=2048),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def index_sets(shape: Shape, seed: int, layer: int = 0):
    """(idx_full_k, idx_full_v): int32 [Hkv][n_full], each row sorted ascending."""
    out = []
    for side, n_full in ((0, shape.n_full_k), (1, shape.n_full_v)):
        rows = []
        for h in range(shape.Hkv):
            g = _gen(seed * 1000003 + layer * 7919 + side * 104729 + h * 31 + 17, "cpu")
            perm = torch.randperm(shape.d, generator=g)[:n_full]
            rows.append(torch.sort(perm).values.to(torch.int32))
        out.append(torch.stack(rows) if rows else torch.zeros((0, n_full), dtype=torch.int32))
    return out[0], out[1]


@dataclass
class KVStream:
    """Endless seeded K/V token stream of one layer; ``tokens(t0, t1)`` is
    deterministic in (seed, layer, t0, t1) and in the device it is drawn on."""
    shape: Shape
    seed: int
    layer: int = 0
    device: str = "cpu"
    freq: str = "grid"            # "grid" | "offgrid"
    n_sin: int = 8
    noise_sigma: float = 0.05
    _par: dict = field(default_factory=dict, repr=False)

    def __post_init__(self):
        s = self.shape
        self.idx_full_k, self.idx_full_v = index_sets(s, self.seed, self.layer)
        for side in (0, 1):
            g = _gen(self.seed * 2000003 + self.layer * 6007 + side * 15485863 + 5, "cpu")
            shp = (s.B, s.Hkv, s.d, self.n_sin)
            amp = torch.rand(shp, generator=g, dtype=torch.float64) * 0.5 + 0.25
            psi = torch.rand(shp, generator=g, dtype=torch.float64) * (2.0 * math.pi)
            if self.freq == "grid":
                f = torch.randint(1, max(2, s.k), shp, generator=g).to(torch.float64)
            else:
                f = torch.rand(shp, generator=g, dtype=torch.float64) * s.k
            self._par[side] = (amp.to(self.device), f.to(self.device), psi.to(self.device))

    def _side(self, side: int, t0: int, t1: int, work_dtype) -> torch.Tensor:
        s = self.shape
        n = t1 - t0
        idx_full = (self.idx_full_k if side == 0 else self.idx_full_v).to(torch.int64)
        amp, f, psi = self._par[side]
        g = _gen(self.seed * 3000017 + self.layer * 4241 + side * 86028121 + t0 * 2 + 1, self.device)
        t = torch.arange(t0, t1, device=self.device, dtype=work_dtype).view(1, n, 1, 1)
        x = torch.zeros((s.B, n, s.Hkv, s.d), device=self.device, dtype=work_dtype)
        w = 2.0 * math.pi / s.T
        for i in range(self.n_sin):
            a_i = amp[..., i].to(work_dtype).unsqueeze(1)       # [B][1][Hkv][d]
            f_i = f[..., i].to(work_dtype).unsqueeze(1)
            p_i = psi[..., i].to(work_dtype).unsqueeze(1)
            x += a_i * torch.cos(w * f_i * t + p_i)
        x += self.noise_sigma * torch.randn(x.shape, generator=g, device=self.device, dtype=work_dtype)
        full = torch.randn((s.B, n, s.Hkv, idx_full.shape[1]), generator=g, device=self.device, dtype=work_dtype)
        for h in range(s.Hkv):
            x[:, :, h, idx_full[h].to(self.device)] = full[:, :, h, :]
        return x.to(s.torch_dtype())

    def tokens(self, t0: int, t1: int, work_dtype=torch.float64):
        """K, V of absolute tokens t0..t1-1: [B][t1-t0][Hkv][d] in the storage dtype."""
        return self._side(0, t0, t1, work_dtype), self._side(1, t0, t1, work_dtype)


def queries(shape: Shape, seed: int, step: int = 0, layer: int = 0, device="cpu", peak: float = 1.0) -> torch.Tensor:
    """q: [B][Hq][d], N(0, d^-1/2) times ``peak``, in the storage dtype."""
    g = _gen(seed * 5000011 + layer * 3571 + step * 13 + 3, device)
    q = torch.randn((shape.B, shape.Hq, shape.d), generator=g, device=device, dtype=torch.float32)
    return (q * (peak / math.sqrt(shape.d))).to(shape.torch_dtype())
