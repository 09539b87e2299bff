"""Parameter shapes of ResNet-50 (v1.5 layout), regenerated from the architecture rule.

Stem 7x7 conv 3->64 + BN; four stages of (3, 4, 6, 3) bottleneck blocks with
widths (64, 128, 256, 512) and expansion 4, each block 1x1 -> 3x3 -> 1x1 convs
with a BN (weight, bias) after every conv, and a 1x1 downsample conv + BN on the
first block of each stage; a 2048 -> 1000 fully connected layer with bias.
"""
from __future__ import annotations


def parameter_shapes() -> list[tuple[int, ...]]:
    shapes: list[tuple[int, ...]] = []

    def conv_bn(cout: int, cin: int, k: int) -> None:
        shapes.append((cout, cin, k, k))
        shapes.append((cout,))
        shapes.append((cout,))

    conv_bn(64, 3, 7)
    cin = 64
    for width, blocks in zip((64, 128, 256, 512), (3, 4, 6, 3)):
        for b in range(blocks):
            conv_bn(width, cin, 1)
            conv_bn(width, width, 3)
            conv_bn(4 * width, width, 1)
            if b == 0:
                conv_bn(4 * width, cin, 1)
            cin = 4 * width
    shapes.append((1000, 2048))
    shapes.append((1000,))
    return shapes
