"""Seeded synthetic gradient generators for the Sketched-SGD compression step.

This module only produces INPUTS (worker gradients g[W][ld], fp32).  It holds none of the method's
arithmetic -- no hashing, sketching, selection or state update -- so that both the CUDA library's
tests and the CPU oracle's tests can draw the same inputs from it without sharing any code of the
method itself.

The five workload families stand in for the gradients of the models the paper trains (a ~90M
transformer and a ~73M LSTM on WMT14, a ResNet on CIFAR-10; Section 5), whose datasets and weights
are not available: they reproduce the flat-vector sizes, the per-layer scale structure and the
heavy-tailed coordinates that make top-k recovery meaningful.

Seeds: structure (block boundaries, scales, heavy sets) comes from a CPU generator seeded with
`structure_seed(cfg)`, so it does not depend on the device; the values of worker w at step t come
from a generator on the target device seeded with `value_seed(cfg, t, w)`.  CPU and CUDA generators
give different streams: whoever needs the same buffers on both sides copies them.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    kind: str          # "lognormal_planted" | "block_gauss" | "block_laplace" | "embedding_mix"
    base_seed: int
    d: int             # coordinates
    W: int             # workers
    r: int             # sketch rows
    c: int             # sketch columns
    ncand: int         # candidates queried in the second round (the paper's P*k)
    k: int             # final sparsity
    rho: float         # momentum
    steps: int         # consecutive steps with fresh gradients
    sketch_seed: int = 0x5EED

    @property
    def ld(self) -> int:
        """Leading dimension of the [W][ld] buffers: d rounded up to 4 floats (16-byte rows)."""
        return (self.d + 3) // 4 * 4

    def scaled(self, **kw) -> "Workload":
        """Same family and seeds at another size (used for small parity cases)."""
        return dataclasses.replace(self, **kw)


C1 = Workload("C1", "lognormal_planted", 1, 1_048_576, 4, 5, 16_384, 2_000, 1_000, 0.9, 1)
C2 = Workload("C2", "block_gauss", 2, 11_173_962, 16, 5, 262_144, 100_000, 50_000, 0.9, 10)
C3 = Workload("C3", "block_laplace", 3, 20_000_000, 32, 5, 1_048_576, 200_000, 100_000, 0.9, 10)
C4 = Workload("C4", "embedding_mix", 4, 90_000_000, 16, 5, 4_194_304, 200_000, 100_000, 0.9, 5)
C5 = tuple(C2.scaled(name=f"C5_W{w}", base_seed=5, W=w, steps=3) for w in (8, 32, 128, 256))

# The paper's own sketch shapes (Table 1 footnotes; 4 workers, k = 100,000), on the block-structured
# Gaussian gradient model: 40x transformer run (15 x 180,000, P = 16), 20x transformer run (5 x 1,000,000,
# P = 36) and the LSTM run (~73M parameters, 5 x 180,000, P = 26).
P1 = Workload("P1", "block_gauss", 11, 90_000_000, 4, 15, 180_000, 1_600_000, 100_000, 0.9, 3)
P2 = Workload("P2", "block_gauss", 12, 90_000_000, 4, 5, 1_000_000, 3_600_000, 100_000, 0.9, 3)
P3 = Workload("P3", "block_gauss", 13, 73_000_000, 4, 5, 180_000, 2_600_000, 100_000, 0.9, 3)

CONFIGS = {w.name: w for w in (C1, C2, C3, C4) + C5 + (P1, P2, P3)}


def structure_seed(cfg: Workload) -> int:
    return cfg.base_seed * 7_919 + 17


def value_seed(cfg: Workload, step: int, w: int) -> int:
    return cfg.base_seed * 1_000_003 + step * 4_099 + w


def _distinct(n: int, d: int, gen: torch.Generator) -> torch.Tensor:
    """n distinct uniform indices in [0, d), from the CPU generator `gen`."""
    n = max(0, min(n, d))
    if n == 0:
        return torch.zeros(0, dtype=torch.int64)
    if d <= 4 * n or d <= 1 << 20:
        return torch.randperm(d, generator=gen)[:n].clone()
    # sparse draw: oversample with replacement, deduplicate, keep a uniform subset of n
    while True:
        uniq = torch.unique(torch.randint(0, d, (int(n * 1.3) + 16,), generator=gen))
        if uniq.numel() >= n:
            return uniq[torch.randperm(uniq.numel(), generator=gen)[:n]].clone()


class Structure:
    """Per-workload fixed structure: a per-coordinate scale vector and family-specific extras."""

    def __init__(self, cfg: Workload, device):
        self.cfg = cfg
        self.device = torch.device(device)
        gen = torch.Generator().manual_seed(structure_seed(cfg))
        d = cfg.d
        self.scale = None          # fp32 [d] on device, multiplies the unit-variance draw
        self.planted_idx = None    # C1: int64 [n] on device
        self.planted_val = None    # C1: fp32 [n] on device (filled on first use)
        self.planted_sign = None
        self.n_embed = 0           # C4: length of the mostly-zero head
        if cfg.kind == "lognormal_planted":
            n = min(1000, max(1, d // 1024))
            self.planted_idx = _distinct(n, d, gen).to(self.device)
            sign = torch.randint(0, 2, (n,), generator=gen).to(torch.float32) * 2 - 1
            self.planted_sign = sign.to(self.device)
        elif cfg.kind == "block_gauss":
            nb = 62 if d >= 62 * 16 else max(1, d // 16)
            t = torch.rand(nb, generator=gen, dtype=torch.float64)
            wts = torch.exp(t * math.log(5000.0))
            lens = torch.floor(d * wts / wts.sum()).to(torch.int64)
            lens[-1] += d - int(lens.sum())
            sigma = torch.pow(10.0, -4.0 + 3.0 * torch.rand(nb, generator=gen, dtype=torch.float64))
            scale = torch.repeat_interleave(sigma.to(torch.float32), lens)
            heavy = _distinct(d // 1000, d, gen)
            scale[heavy] *= 20.0
            self.scale = scale.to(self.device)
        elif cfg.kind == "block_laplace":
            nb = 8
            lens = torch.full((nb,), d // nb, dtype=torch.int64)
            lens[-1] += d - int(lens.sum())
            sigma = torch.pow(10.0, -5.0 + 3.0 * torch.rand(nb, generator=gen, dtype=torch.float64))
            scale = torch.repeat_interleave(sigma.to(torch.float32), lens)
            heavy = _distinct(d // 200, d, gen)
            scale[heavy] *= 30.0
            self.scale = scale.to(self.device)
        elif cfg.kind == "embedding_mix":
            self.n_embed = d // 3
            scale = torch.empty(d, dtype=torch.float32)
            scale[: self.n_embed] = 0.1                     # N(0, 1e-2): standard deviation 0.1
            scale[self.n_embed:] = math.sqrt(1e-3)          # N(0, 1e-3)
            n_rest = d - self.n_embed
            heavy = _distinct(n_rest // 500, n_rest, gen) + self.n_embed
            scale[heavy] *= 25.0
            self.scale = scale.to(self.device)
        else:
            raise ValueError(f"unknown workload kind {cfg.kind!r}")


def gradients(st: Structure, step: int, out: torch.Tensor | None = None) -> torch.Tensor:
    """The gradients g[W][ld] (fp32, padding columns zero) of every worker at `step`."""
    cfg, dev = st.cfg, st.device
    d, W, ld = cfg.d, cfg.W, cfg.ld
    if out is None:
        out = torch.zeros((W, ld), dtype=torch.float32, device=dev)
    else:
        assert out.shape == (W, ld) and out.dtype == torch.float32 and out.device == dev
        if ld > d:
            out[:, d:].zero_()
    for w in range(W):
        gen = torch.Generator(device=dev).manual_seed(value_seed(cfg, step, w))
        row = out[w, :d]
        if cfg.kind == "lognormal_planted":
            z = torch.randn(d, generator=gen, device=dev, dtype=torch.float32)
            y = torch.randn(d, generator=gen, device=dev, dtype=torch.float32)
            torch.mul(z, torch.exp(1.5 * y), out=row)
            if st.planted_val is None:
                # magnitude: 50 x the median |value| of worker 0's base vector at step 0
                if w == 0 and step == 0:
                    base = row
                else:
                    g0 = torch.Generator(device=dev).manual_seed(value_seed(cfg, 0, 0))
                    z0 = torch.randn(d, generator=g0, device=dev, dtype=torch.float32)
                    y0 = torch.randn(d, generator=g0, device=dev, dtype=torch.float32)
                    base = z0 * torch.exp(1.5 * y0)
                st.planted_val = 50.0 * base.abs().median() * st.planted_sign
            row[st.planted_idx] = st.planted_val
        elif cfg.kind == "block_gauss":
            torch.randn(d, generator=gen, device=dev, dtype=torch.float32, out=row)
            row.mul_(st.scale)
        elif cfg.kind == "block_laplace":
            uu = torch.rand(d, generator=gen, device=dev, dtype=torch.float32) - 0.5
            mag = -torch.log(torch.clamp_min(1.0 - 2.0 * uu.abs(), 2.0 ** -24))
            torch.mul(torch.sign(uu), mag, out=row)          # Laplace(0, 1), finite by the clamp
            row.mul_(st.scale)
        elif cfg.kind == "embedding_mix":
            torch.randn(d, generator=gen, device=dev, dtype=torch.float32, out=row)
            row.mul_(st.scale)
            keep = torch.rand(st.n_embed, generator=gen, device=dev) >= 0.99
            row[: st.n_embed].masked_fill_(~keep, 0.0)       # 99% exact zeros in the head
        else:
            raise ValueError(cfg.kind)
    return out


def zero_state(cfg: Workload, device) -> tuple[torch.Tensor, torch.Tensor]:
    """Zero-initialised momentum u and error accumulation v, [W][ld] fp32 (Algorithm 3 line 1)."""
    u = torch.zeros((cfg.W, cfg.ld), dtype=torch.float32, device=device)
    v = torch.zeros((cfg.W, cfg.ld), dtype=torch.float32, device=device)
    return u, v
