"""Pins the oracle's closed forms to numbers the paper prints (ImageNet table, vanilla rows)
and to hand-expanded instances of the storage / overhead / cost formulas."""
import os

import numpy as np

from oracle import asi_oracle as O

MiB = 1024.0 * 1024.0


def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_table_imagenet.txt")
    out = {}
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def _mem_MB(shapes, B=64):
    return sum(B * c * h * w * 4 for (c, h, w) in shapes) / MiB


def _gmac(layers, B=64):
    """layers: (C, H, W, Cout, k, stride, pad)"""
    tot = 0
    for (C, H, W, Co, k, s, p) in layers:
        Ho, Wo = O.conv_out_size(H, k, s, p), O.conv_out_size(W, k, s, p)
        tot += O.macs_O_vanilla((B, C, H, W), Co, k) + O.macs_C_vanilla((B, C, H, W), Co, Ho, Wo, k)
    return tot / 1e9


L4 = (512, 7, 7, 512, 3, 1, 1)
DS4 = (256, 14, 14, 512, 1, 2, 0)


def test_resnet18_vanilla_rows():
    g = _golden()
    assert abs(_mem_MB([(512, 7, 7)] * 2) - g["resnet18_vanilla_mem_2layers_MB"]) < 0.005
    # module order: ..., layer4.0.conv2, layer4.0.downsample, layer4.1.conv1, layer4.1.conv2
    assert abs(_mem_MB([(512, 7, 7)] * 3 + [(256, 14, 14)]) - g["resnet18_vanilla_mem_4layers_MB"]) < 0.006
    assert abs(_gmac([L4, L4]) - g["resnet18_vanilla_gmac_2layers"]) < 0.01
    assert abs(_gmac([L4, L4, L4, DS4]) - g["resnet18_vanilla_gmac_4layers"]) < 0.01


def test_resnet18_all_layers_memory():
    g = _golden()
    shapes = [(3, 224, 224)] + [(64, 56, 56)] * 6 + [(128, 28, 28)] * 5 + [(256, 14, 14)] * 5 + [(512, 7, 7)] * 3
    assert len(shapes) == 20   # 17 convs + 3 downsample convs
    assert abs(_mem_MB(shapes) - g["resnet18_vanilla_mem_all_MB"]) < 0.005


def test_resnet34_and_mobilenet_rows():
    g = _golden()
    assert abs(_mem_MB([(512, 7, 7)] * 2) - g["resnet34_vanilla_mem_2layers_MB"]) < 0.005
    assert abs(_mem_MB([(512, 7, 7)] * 4) - g["resnet34_vanilla_mem_4layers_MB"]) < 0.005
    assert abs(_gmac([L4] * 2) - g["resnet34_vanilla_gmac_2layers"]) < 0.01
    assert abs(_gmac([L4] * 4) - g["resnet34_vanilla_gmac_4layers"]) < 0.01
    assert abs(_mem_MB([(960, 7, 7), (320, 7, 7)]) - g["mobilenetv2_vanilla_mem_2layers_MB"]) < 0.005
    assert abs(_mem_MB([(960, 7, 7), (320, 7, 7), (960, 7, 7), (160, 7, 7)])
               - g["mobilenetv2_vanilla_mem_4layers_MB"]) < 0.006
    assert abs(_gmac([(960, 7, 7, 320, 1, 1, 0), (320, 7, 7, 1280, 1, 1, 0)])
               - g["mobilenetv2_vanilla_gmac_2layers"]) < 0.01


def test_storage_and_ratio_hand_expanded():
    shape, r = (8, 32, 16, 16), (4, 8, 8, 8)
    assert O.compressed_elems(shape, r) == 4 * 8 * 8 * 8 + 8 * 4 + 32 * 8 + 16 * 8 + 16 * 8
    assert np.isclose(O.ratio_RC(shape, r), 65536 / 2592.0)
    # full rank stores more than the tensor itself
    assert O.compressed_elems((2, 3, 4, 5), (2, 3, 4, 5)) == 120 + 4 + 9 + 16 + 25


def test_overhead_and_cost_hand_expanded():
    shape, r = (8, 32, 16, 16), (4, 8, 8, 8)
    n = 65536
    assert O.macs_O_ASI(shape, r) == 2 * n * (4 + 8 + 8 + 8) + 64 + 3 * 512
    # five terms, one by one
    B, C, H, W = shape
    Co, Ho, Wo, k = 32, 16, 16, 3
    t1 = 4 * B * Co * Ho * Wo
    t2 = 4 * 8 * 8 * 8 * H
    t3 = 4 * 8 * 8 * H * W
    t4 = 4 * 8 * Co * Ho * Wo * 9
    t5 = 8 * Co * C * 9
    assert O.macs_C_ASI(shape, r, Co, Ho, Wo, k) == t1 + t2 + t3 + t4 + t5
    assert O.macs_C_vanilla(shape, Co, Ho, Wo, k) == 9 * C * Co * B * Ho * Wo
