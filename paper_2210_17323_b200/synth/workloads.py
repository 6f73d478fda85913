"""The five synthetic workloads: layer shapes, calibration sizes and grids.

Shapes are (R, C) = (out features, in features); C is the Hessian size.  Every
layer gets its own seeded W and X (see generator.py for the distributions).
The sets take the shapes of OPT / BLOOM linear layers with 128 x 2048 calibration
tokens (Section 5, Setup); they stand in for trained weights and C4 activations.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

from . import generator as G

BITS_TERNARY = -1

LAYER_KINDS = {"q": 0, "k": 1, "v": 2, "o": 3, "fc1": 4, "fc2": 5}


@dataclass(frozen=True)
class Grid:
    bits: int            # 2, 3, 4, 8 or BITS_TERNARY
    group_size: int      # <= 0: one grid per row
    sym: bool = False


@dataclass(frozen=True)
class Layer:
    config_id: int
    block_idx: int
    kind: str
    R: int
    C: int
    n_tokens: int

    @property
    def name(self) -> str:
        return f"c{self.config_id}.b{self.block_idx}.{self.kind}[{self.R}x{self.C}]"

    def seed(self, tensor_kind: int) -> int:
        return G.stream_seed(self.config_id, self.block_idx, LAYER_KINDS[self.kind], tensor_kind)

    # ---- host-side generation (any subset) ---------------------------------
    def scales(self):
        return G.channel_scales(self.seed(G.TENSOR_SCALES), self.seed(G.TENSOR_OUTLIERS), self.C)

    def x_bits(self, t0=0, t1=None, cols=None, scales=None):
        t1 = self.n_tokens if t1 is None else t1
        s = self.scales() if scales is None else scales
        return G.gen_x_bits(self.seed(G.TENSOR_X), s, self.C, t0, t1, cols)

    def w(self, rows=None):
        return G.gen_w(self.seed(G.TENSOR_W), self.R, self.C, rows)


@dataclass(frozen=True)
class Workload:
    config_id: int
    name: str
    layers: Tuple[Layer, ...]
    grids: Tuple[Grid, ...]
    block: int = 128
    damp: float = 0.01
    block_sweep: Tuple[int, ...] = field(default_factory=tuple)

    @property
    def weights(self) -> int:
        return sum(l.R * l.C for l in self.layers)


def _block_layers(cfg, blk, d_model, d_ffn, n_tokens) -> List[Layer]:
    out = [Layer(cfg, blk, k, d_model, d_model, n_tokens) for k in ("q", "k", "v", "o")]
    out.append(Layer(cfg, blk, "fc1", d_ffn, d_model, n_tokens))
    out.append(Layer(cfg, blk, "fc2", d_model, d_ffn, n_tokens))
    return out


FULL_TOKENS = 128 * 2048


def workload(config_id: int) -> Workload:
    if config_id == 0:
        return Workload(0, "c0-single-768", (Layer(0, 0, "q", 768, 768, 8192),), (Grid(4, 0),))
    if config_id == 1:
        layers = []
        for blk in range(12):
            layers += _block_layers(1, blk, 768, 3072, FULL_TOKENS)
        return Workload(1, "c1-opt125m-set", tuple(layers), (Grid(4, 0), Grid(3, 0)))
    if config_id == 2:
        return Workload(2, "c2-opt6.7b-block", tuple(_block_layers(2, 0, 4096, 16384, FULL_TOKENS)),
                        (Grid(3, 128),))
    if config_id == 3:
        return Workload(3, "c3-opt175b-block", tuple(_block_layers(3, 0, 12288, 49152, FULL_TOKENS)),
                        (Grid(4, 0), Grid(3, 0)))
    if config_id == 4:
        layers = (Layer(4, 0, "q", 14336, 14336, FULL_TOKENS),
                  Layer(4, 0, "fc1", 57344, 14336, FULL_TOKENS),
                  Layer(4, 0, "fc2", 14336, 57344, FULL_TOKENS))
        return Workload(4, "c4-bloom176b-extreme", layers, (Grid(2, 128), Grid(BITS_TERNARY, 128)),
                        block_sweep=(32, 64, 128, 256))
    raise ValueError(f"unknown config {config_id}")
