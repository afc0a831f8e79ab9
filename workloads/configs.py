"""Workload table: flat parameter vectors laid out as per-layer segments.

Each config fixes N (parameters), K (simulated workers), the core and
explorer ratios, a seed, and the per-segment value recipe.  The ratios become
integer counts by floor division; the explorer ratio is taken of the non-core
remainder M = N - k_core.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Tuple


@dataclasses.dataclass(frozen=True)
class Segment:
    name: str
    size: int
    sigma: float      # std of the layer's He-normal weights (also scales this segment's gradients)
    kind: str         # "weight" -> N(0, sigma); "zero" -> 0 (biases, BN beta); "one" -> 1 (BN gamma)


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    segments: Tuple[Segment, ...]
    K: int
    core_pct: int
    explore_pct: int
    seed: int
    grad_dist: str            # "normal" | "normal_layer" | "laplace"
    grad_scale: float         # std (normal), multiplier of the layer sigma (normal_layer), b (laplace)
    quantise: bool = False    # snap weights / gradients to 256-value power-of-two grids
    c: float = 1.0            # significance coefficient of Eq. 1

    @property
    def N(self) -> int:
        return sum(s.size for s in self.segments)

    @property
    def k_core(self) -> int:
        return self.N * self.core_pct // 100

    @property
    def M(self) -> int:
        return self.N - self.k_core

    @property
    def k_exp(self) -> int:
        return self.M * self.explore_pct // 100

    @property
    def m(self) -> int:
        return self.k_core + self.k_exp

    @property
    def eta(self) -> float:
        return 1.0 / self.K

    def with_core_pct(self, pct: int) -> "Config":
        return dataclasses.replace(self, core_pct=pct)

    def bounds(self) -> List[Tuple[int, int, Segment]]:
        out, pos = [], 0
        for s in self.segments:
            out.append((pos, pos + s.size, s))
            pos += s.size
        return out


def _he(fan_in: int) -> float:
    return math.sqrt(2.0 / fan_in)


def _conv(name, cin, cout, k, bias=True, bn=False) -> List[Segment]:
    sig = _he(cin * k * k)
    segs = [Segment(f"{name}.weight", cin * cout * k * k, sig, "weight")]
    if bias:
        segs.append(Segment(f"{name}.bias", cout, sig, "zero"))
    if bn:
        segs.append(Segment(f"{name}.bn.gamma", cout, sig, "one"))
        segs.append(Segment(f"{name}.bn.beta", cout, sig, "zero"))
    return segs


def _fc(name, fin, fout) -> List[Segment]:
    sig = _he(fin)
    return [Segment(f"{name}.weight", fin * fout, sig, "weight"),
            Segment(f"{name}.bias", fout, sig, "zero")]


def _flat(n: int, sigma: float) -> Tuple[Segment, ...]:
    return (Segment("flat", n, sigma, "weight"),)


def _googlenet() -> Tuple[Segment, ...]:
    segs: List[Segment] = []
    segs += _conv("conv1", 3, 64, 7)
    segs += _conv("conv2_reduce", 64, 64, 1)
    segs += _conv("conv2", 64, 192, 3)
    # (name, in, 1x1, 3x3 reduce, 3x3, 5x5 reduce, 5x5, pool projection)
    table = [("3a", 192, 64, 96, 128, 16, 32, 32), ("3b", 256, 128, 128, 192, 32, 96, 64),
             ("4a", 480, 192, 96, 208, 16, 48, 64), ("4b", 512, 160, 112, 224, 24, 64, 64),
             ("4c", 512, 128, 128, 256, 24, 64, 64), ("4d", 512, 112, 144, 288, 32, 64, 64),
             ("4e", 528, 256, 160, 320, 32, 128, 128), ("5a", 832, 256, 160, 320, 32, 128, 128),
             ("5b", 832, 384, 192, 384, 48, 128, 128)]
    for n, cin, c1, c3r, c3, c5r, c5, pp in table:
        segs += _conv(f"inc{n}.1x1", cin, c1, 1)
        segs += _conv(f"inc{n}.3x3_reduce", cin, c3r, 1)
        segs += _conv(f"inc{n}.3x3", c3r, c3, 3)
        segs += _conv(f"inc{n}.5x5_reduce", cin, c5r, 1)
        segs += _conv(f"inc{n}.5x5", c5r, c5, 5)
        segs += _conv(f"inc{n}.pool_proj", cin, pp, 1)
    segs += _fc("fc", 1024, 1000)
    return tuple(segs)


def _vgg16() -> Tuple[Segment, ...]:
    chans = [(3, 64), (64, 64), (64, 128), (128, 128), (128, 256), (256, 256), (256, 256),
             (256, 512), (512, 512), (512, 512), (512, 512), (512, 512), (512, 512)]
    segs: List[Segment] = []
    for i, (a, b) in enumerate(chans):
        segs += _conv(f"conv{i}", a, b, 3)
    segs += _fc("fc6", 25088, 4096)
    segs += _fc("fc7", 4096, 4096)
    segs += _fc("fc8", 4096, 1000)
    return tuple(segs)


def _resnet50() -> Tuple[Segment, ...]:
    segs: List[Segment] = []
    segs += _conv("stem", 3, 64, 7, bias=False, bn=True)
    cin = 64
    for stage, (mid, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        cout = mid * 4
        for b in range(blocks):
            p = f"layer{stage + 1}.{b}"
            segs += _conv(f"{p}.conv1", cin, mid, 1, bias=False, bn=True)
            segs += _conv(f"{p}.conv2", mid, mid, 3, bias=False, bn=True)
            segs += _conv(f"{p}.conv3", mid, cout, 1, bias=False, bn=True)
            if b == 0:
                segs += _conv(f"{p}.downsample", cin, cout, 1, bias=False, bn=True)
            cin = cout
    segs += _fc("fc", 2048, 1000)
    return tuple(segs)


CONFIGS = {
    "tiny": Config("tiny", _flat(1_000_000, 0.05), K=4, core_pct=10, explore_pct=5, seed=0,
                   grad_dist="normal", grad_scale=1e-3),
    "googlenet": Config("googlenet", _googlenet(), K=8, core_pct=10, explore_pct=2, seed=1,
                        grad_dist="normal_layer", grad_scale=0.01),
    "vgg16": Config("vgg16", _vgg16(), K=8, core_pct=5, explore_pct=1, seed=2,
                    grad_dist="laplace", grad_scale=1e-4),
    "resnet50_ties": Config("resnet50_ties", _resnet50(), K=16, core_pct=20, explore_pct=5, seed=3,
                            grad_dist="normal_layer", grad_scale=0.01, quantise=True),
    "large": Config("large", _flat(1_000_000_000, 0.02), K=4, core_pct=1, explore_pct=1, seed=4,
                    grad_dist="normal", grad_scale=1e-3),
}

LARGE_CORE_PCTS = (1, 5, 10, 30)


def get_config(name: str) -> Config:
    return CONFIGS[name]


def scaled_config(cfg: Config, n: int) -> Config:
    """The leading n parameters of cfg (same recipe, same random streams):
    a bounded sample of the workload for slow CPU runs."""
    if n >= cfg.N:
        return cfg
    segs, left = [], n
    for s in cfg.segments:
        if left <= 0:
            break
        take = min(left, s.size)
        segs.append(dataclasses.replace(s, size=take))
        left -= take
    return dataclasses.replace(cfg, name=f"{cfg.name}[:{n}]", segments=tuple(segs))
