"""Layer-shape tables of the five CNNs the paper evaluates (its experiments section names
ResNet18v1, ResNet50v1, MobileNetv2, SqueezeNet and VGGNet).

Only architecture hyper-parameters live here: for every conv / fc layer the weight shape
``[cout, K]`` with ``K = cin/groups * k * k`` and the output feature-map side.  No trained
weights and no dataset items are involved; values are drawn by ``gen.synth``.

Each layer also carries ``act``, the value distribution its output tensor is drawn from:
  "relu"   ReLU(N(0, s_c))        -- about half the mass exactly zero
  "relu6"  min(ReLU(N(0, s_c)), 6)
  "half"   |N(0, s_c)|            -- half-normal
  "gauss"  N(0, s_c)              -- outputs that feed a residual add, linear bottlenecks, logits
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List


@dataclass(frozen=True)
class LayerShape:
    name: str
    cout: int
    k_elems: int          # weights per output channel: cin/groups * k * k
    out_hw: int           # output feature-map side (1 for fc)
    act: str              # distribution of the layer's output tensor
    kind: str = "conv"    # "conv" | "dw" | "fc"

    @property
    def weight_elems(self) -> int:
        return self.cout * self.k_elems

    @property
    def act_elems_per_image(self) -> int:
        return self.cout * self.out_hw * self.out_hw

    @property
    def macs(self) -> int:
        """Multiply-accumulates of the layer for one image (the MAC(op) of the paper's BOPs
        formula): weight elements times output positions."""
        return self.weight_elems * self.out_hw * self.out_hw


def _conv(name, cout, cin, k, hw, act, groups=1):
    kind = "dw" if groups == cin and groups > 1 else "conv"
    return LayerShape(name, cout, (cin // groups) * k * k, hw, act, kind)


def _fc(name, cout, cin, act="gauss"):
    return LayerShape(name, cout, cin, 1, act, "fc")


def squeezenet_v1_0(act="relu") -> List[LayerShape]:
    layers = [_conv("conv1", 96, 3, 7, 109, act)]

    def fire(idx, cin, s, e, hw):
        return [
            _conv(f"fire{idx}.squeeze", s, cin, 1, hw, act),
            _conv(f"fire{idx}.expand1x1", e, s, 1, hw, act),
            _conv(f"fire{idx}.expand3x3", e, s, 3, hw, act),
        ]

    spec = [(2, 96, 16, 64, 54), (3, 128, 16, 64, 54), (4, 128, 32, 128, 54),
            (5, 256, 32, 128, 27), (6, 256, 48, 192, 27), (7, 384, 48, 192, 27),
            (8, 384, 64, 256, 27), (9, 512, 64, 256, 13)]
    for idx, cin, s, e, hw in spec:
        layers += fire(idx, cin, s, e, hw)
    layers.append(_conv("conv10", 1000, 512, 1, 13, act))
    return layers


def resnet18_v1(post_relu="half") -> List[LayerShape]:
    layers = [_conv("conv1", 64, 3, 7, 112, post_relu)]
    cin = 64
    for stage, (c, hw) in enumerate([(64, 56), (128, 28), (256, 14), (512, 7)], start=1):
        for b in range(2):
            layers.append(_conv(f"layer{stage}.{b}.conv1", c, cin, 3, hw, post_relu))
            layers.append(_conv(f"layer{stage}.{b}.conv2", c, c, 3, hw, "gauss"))
            if b == 0 and cin != c:
                layers.append(_conv(f"layer{stage}.{b}.downsample", c, cin, 1, hw, "gauss"))
            cin = c
    layers.append(_fc("fc", 1000, 512))
    return layers


def resnet50_v1(post_relu="relu") -> List[LayerShape]:
    layers = [_conv("conv1", 64, 3, 7, 112, post_relu)]
    cin = 64
    for stage, (c, hw, n) in enumerate([(64, 56, 3), (128, 28, 4), (256, 14, 6), (512, 7, 3)], 1):
        for b in range(n):
            layers.append(_conv(f"layer{stage}.{b}.conv1", c, cin, 1, hw, post_relu))
            layers.append(_conv(f"layer{stage}.{b}.conv2", c, c, 3, hw, post_relu))
            layers.append(_conv(f"layer{stage}.{b}.conv3", 4 * c, c, 1, hw, "gauss"))
            if b == 0:
                layers.append(_conv(f"layer{stage}.{b}.downsample", 4 * c, cin, 1, hw, "gauss"))
            cin = 4 * c
    layers.append(_fc("fc", 1000, 2048))
    return layers


def mobilenet_v2(with_fc=True) -> List[LayerShape]:
    layers = [_conv("stem", 32, 3, 3, 112, "relu6")]
    cin, hw = 32, 112
    blk = 0
    for t, c, n, s in [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                       (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]:
        for b in range(n):
            stride = s if b == 0 else 1
            hid = cin * t
            if t != 1:
                layers.append(_conv(f"block{blk}.expand", hid, cin, 1, hw, "relu6"))
            hw = hw // stride
            layers.append(_conv(f"block{blk}.depthwise", hid, hid, 3, hw, "relu6", groups=hid))
            layers.append(_conv(f"block{blk}.project", c, hid, 1, hw, "gauss"))
            cin = c
            blk += 1
    layers.append(_conv("last", 1280, 320, 1, 7, "relu6"))
    if with_fc:
        layers.append(_fc("classifier", 1000, 1280))
    return layers


def vgg16(post_relu="half") -> List[LayerShape]:
    layers = []
    cin = 3
    i = 0
    for c, hw, n in [(64, 224, 2), (128, 112, 2), (256, 56, 3), (512, 28, 3), (512, 14, 3)]:
        for _ in range(n):
            i += 1
            layers.append(_conv(f"conv{i}", c, cin, 3, hw, post_relu))
            cin = c
    layers += [_fc("fc6", 4096, 25088, post_relu), _fc("fc7", 4096, 4096, post_relu),
               _fc("fc8", 1000, 4096, "gauss")]
    return layers


SHAPES = {
    "squeezenet": squeezenet_v1_0,
    "resnet18": resnet18_v1,
    "resnet50": resnet50_v1,
    "mobilenetv2": mobilenet_v2,
    "vgg16": vgg16,
}
