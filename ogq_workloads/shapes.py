"""Parameter shapes of the two CNNs whose gradient buckets the benchmark mimics.

The shapes are generated from the architecture rules (Table 1 of the paper
quotes the totals: ResNet-50 25.6 M and VGG-19 143.7 M parameters) and are
checked against the exact totals in the CPU tests.
"""
from __future__ import annotations

from typing import List, Tuple

Shape = Tuple[int, ...]


def numel(shape: Shape) -> int:
    n = 1
    for d in shape:
        n *= int(d)
    return n


def _bn(ch: int) -> List[Tuple[str, Shape]]:
    return [("bn_weight", (ch,)), ("bn_bias", (ch,))]


def resnet50_shapes() -> List[Tuple[str, Shape]]:
    """161 tensors, 25,557,032 elements.

    Stem 7x7 convolution + batch norm; four stages of (3, 4, 6, 3) bottleneck
    blocks with widths 64/128/256/512 and expansion 4 (1x1, 3x3, 1x1
    convolutions, each followed by a batch-norm weight and bias); a 1x1
    down-sampling convolution + batch norm in the first block of every stage;
    a 1000-way fully connected layer with bias.
    """
    out: List[Tuple[str, Shape]] = [("conv", (64, 3, 7, 7))]
    out += _bn(64)
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            out.append(("conv", (planes, inplanes, 1, 1)))
            out += _bn(planes)
            out.append(("conv", (planes, planes, 3, 3)))
            out += _bn(planes)
            out.append(("conv", (planes * 4, planes, 1, 1)))
            out += _bn(planes * 4)
            if b == 0:
                out.append(("conv", (planes * 4, inplanes, 1, 1)))
                out += _bn(planes * 4)
            inplanes = planes * 4
    out.append(("fc_weight", (1000, 2048)))
    out.append(("fc_bias", (1000,)))
    return out


def vgg19_shapes() -> List[Tuple[str, Shape]]:
    """38 tensors, 143,667,240 elements.

    Sixteen 3x3 convolutions (64, 64, 128, 128, 256 x4, 512 x4, 512 x4) with
    biases, then fully connected layers 25088->4096, 4096->4096, 4096->1000
    with biases.
    """
    out: List[Tuple[str, Shape]] = []
    cin = 3
    for cout in (64, 64, 128, 128, 256, 256, 256, 256, 512, 512, 512, 512, 512, 512, 512, 512):
        out.append(("conv", (cout, cin, 3, 3)))
        out.append(("bias", (cout,)))
        cin = cout
    for fin, fout in ((25088, 4096), (4096, 4096), (4096, 1000)):
        out.append(("fc_weight", (fout, fin)))
        out.append(("fc_bias", (fout,)))
    return out
