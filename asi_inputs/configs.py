"""Workload tables: layer shapes of the five benchmark configurations.

Shapes follow the published ResNet-18/34, MobileNetV2 and ViT-Base layer
tables at 224x224 input.  Ranks of the energy-picked configurations are the
numbers in ``energy_ranks.py`` (written by ``oracle/pick_ranks.py`` from the
step-0 tensor of each layer's stream).  Pure data: no method arithmetic here.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

from .generator import LayerStream

SEED_BASE = 20250505


@dataclass(frozen=True)
class LayerSpec:
    name: str
    kind: str                 # "conv" | "linear"
    dims: tuple               # activation shape
    cout: int
    k: int = 1
    stride: int = 1
    pad: int = 0
    groups: int = 1
    ranks: tuple = None
    energy: float = None      # explained-variance threshold the ranks were picked at
    count: int = 1            # how many layers of the network share this shape

    @property
    def out_hw(self):
        H, W = self.dims[2], self.dims[3]
        return ((H + 2 * self.pad - self.k) // self.stride + 1,
                (W + 2 * self.pad - self.k) // self.stride + 1)

    @property
    def dy_shape(self):
        if self.kind == "linear":
            return tuple(self.dims[:-1]) + (self.cout,)
        ho, wo = self.out_hw
        return (self.dims[0], self.cout, ho, wo)

    @property
    def dw_shape(self):
        if self.kind == "linear":
            return (self.cout, self.dims[-1])
        return (self.cout, self.dims[1] // self.groups, self.k, self.k)


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    layers: tuple
    steps: int
    bf16: bool = False
    clip: tuple = None
    rho_rule: str = "0.7"      # "0.7" or "rank-scaled"


def _conv(name, B, C, HW, cout, k, s, p, groups=1, **kw):
    return LayerSpec(name, "conv", (B, C, HW, HW), cout, k, s, p, groups, **kw)


def _with_ranks(cfg_index, layers, energy):
    from .energy_ranks import ENERGY_RANKS
    out = []
    for li, L in enumerate(layers):
        key = (cfg_index, li, energy)
        out.append(replace(L, ranks=tuple(ENERGY_RANKS[key]), energy=energy))
    return tuple(out)


def _config2_layers():
    return (
        _conv("layer4.0.conv1", 64, 256, 14, 512, 3, 2, 1),
        _conv("layer4.0.conv2", 64, 512, 7, 512, 3, 1, 1),
        _conv("layer4.1.conv1", 64, 512, 7, 512, 3, 1, 1),
        _conv("layer4.1.conv2", 64, 512, 7, 512, 3, 1, 1),
    )


def _config3_layers():
    B = 128
    return (
        _conv("block16.project(960->160)", B, 960, 7, 160, 1, 1, 0),
        _conv("block17.expand(160->960)", B, 160, 7, 960, 1, 1, 0),
        _conv("block17.depthwise(960)", B, 960, 7, 960, 3, 1, 1, groups=960),
        _conv("block17.project(960->320)", B, 960, 7, 320, 1, 1, 0),
        _conv("head.conv(320->1280)", B, 320, 7, 1280, 1, 1, 0),
    )


def _config4_layers():
    B = 128
    return (
        _conv("layer1.x(64->64)", B, 64, 56, 64, 3, 1, 1, count=6),
        _conv("layer2.0.conv1(64->128,s2)", B, 64, 56, 128, 3, 2, 1),
        _conv("layer2.0.downsample(1x1,s2)", B, 64, 56, 128, 1, 2, 0),
        _conv("layer2.x(128->128)", B, 128, 28, 128, 3, 1, 1, count=7),
        _conv("layer3.0.conv1(128->256,s2)", B, 128, 28, 256, 3, 2, 1),
        _conv("layer3.0.downsample(1x1,s2)", B, 128, 28, 256, 1, 2, 0),
        _conv("layer3.x(256->256)", B, 256, 14, 256, 3, 1, 1, count=11),
        _conv("layer4.0.conv1(256->512,s2)", B, 256, 14, 512, 3, 2, 1),
        _conv("layer4.0.downsample(1x1,s2)", B, 256, 14, 512, 1, 2, 0),
        _conv("layer4.x(512->512)", B, 512, 7, 512, 3, 1, 1, count=5),
    )


def get_config(index: int, energy: float = None, bf16: bool = None) -> Config:
    """Config ``index`` (0-based, the order of the benchmark description)."""
    if index == 0:
        L = (replace(_conv("conv3x3", 8, 32, 16, 32, 3, 1, 1), ranks=(4, 8, 8, 8)),)
        return Config(0, "single-conv", L, steps=3)
    if index == 1:
        e = 0.9 if energy is None else energy
        return Config(1, "resnet18-last4", _with_ranks(1, _config2_layers(), e), steps=10)
    if index == 2:
        e = 0.8 if energy is None else energy
        return Config(2, "mobilenetv2-last5", _with_ranks(2, _config3_layers(), e), steps=10,
                      clip=(0.0, 6.0))
    if index == 3:
        e = 0.9 if energy is None else energy
        return Config(3, "resnet34-sweep", _with_ranks(3, _config4_layers(), e), steps=20,
                      bf16=bool(bf16))
    if index == 4:
        L = (LayerSpec("mlp.fc1(768->3072)", "linear", (32, 197, 768), 3072, ranks=(8, 32, 64)),
             LayerSpec("mlp.fc2(3072->768)", "linear", (32, 197, 3072), 768, ranks=(8, 32, 64)))
        return Config(4, "vit-base-mlp", L, steps=20, bf16=True if bf16 is None else bool(bf16),
                      rho_rule="rank-scaled")
    if index == 5:
        # LLM-shaped tokens (appendix, TinyLlama experiment: batch 8, up to 512 tokens, 2048-wide, a single
        # rank of 20): the rank-range rule r_m <= a_m clips the batch mode to 8
        L = (LayerSpec("attn.proj(2048->2048)", "linear", (8, 512, 2048), 2048, ranks=(8, 20, 20)),
             LayerSpec("mlp.up(2048->5632)", "linear", (8, 512, 2048), 5632, ranks=(8, 20, 20)),
             LayerSpec("mlp.down(5632->2048)", "linear", (8, 512, 5632), 2048, ranks=(8, 20, 20)))
        return Config(5, "llm-tokens", L, steps=20, bf16=True if bf16 is None else bool(bf16),
                      rho_rule="rank-scaled")
    raise ValueError("config index 0..5")


def layer_seed(cfg_index: int, layer_index: int) -> int:
    # the benchmark description numbers its configurations from 1
    return SEED_BASE + 10000 * (cfg_index + 1) + 100 * layer_index


def make_stream(cfg: Config, layer_index: int, ranks=None) -> LayerStream:
    L = cfg.layers[layer_index]
    r = tuple(ranks if ranks is not None else L.ranks)
    kw = {}
    if cfg.rho_rule == "rank-scaled":
        kw["rho"] = tuple(0.7 ** (8.0 / rm) for rm in r)
        kw["gen_ranks"] = tuple(min(d, 2 * rm) for d, rm in zip(L.dims, r))
    return LayerStream(dims=L.dims, ranks=r, dy_shape=L.dy_shape,
                       seed=layer_seed(cfg.index, layer_index), clip=cfg.clip,
                       bf16=cfg.bf16, **kw)


def untuned_layers(index: int):
    """Layer shapes of an energy-picked configuration before ranks are chosen
    (used by the rank-picking script)."""
    return {1: _config2_layers, 2: _config3_layers, 3: _config4_layers}[index]()


CONFIG_CLIP = {1: None, 2: (0.0, 6.0), 3: None}
