"""Parameter-tensor shapes of the architectures the synthetic workloads borrow.

Only the *shapes* are used: the flat parameter vector is the concatenation of
the tensors in definition order, and each tensor is one layer ``j`` in the
sense of the per-layer loop of Algorithm 3 / Algorithm 2.  No weights, no data.
"""
from __future__ import annotations

from math import prod
from typing import List, Tuple

Shape = Tuple[str, Tuple[int, ...]]


def _bn(name: str, c: int) -> List[Shape]:
    return [(f"{name}.weight", (c,)), (f"{name}.bias", (c,))]


def resnet18_shapes(num_classes: int = 1000) -> List[Shape]:
    """ResNet-18, basic blocks [2,2,2,2], widths 64..512 (62 tensors)."""
    out: List[Shape] = [("conv1.weight", (64, 3, 7, 7))] + _bn("bn1", 64)
    cin = 64
    for stage, width in enumerate((64, 128, 256, 512), start=1):
        for block in range(2):
            p = f"layer{stage}.{block}"
            out.append((f"{p}.conv1.weight", (width, cin, 3, 3)))
            out += _bn(f"{p}.bn1", width)
            out.append((f"{p}.conv2.weight", (width, width, 3, 3)))
            out += _bn(f"{p}.bn2", width)
            if block == 0 and stage > 1:
                out.append((f"{p}.downsample.0.weight", (width, cin, 1, 1)))
                out += _bn(f"{p}.downsample.1", width)
            cin = width
    out.append(("fc.weight", (num_classes, 512)))
    out.append(("fc.bias", (num_classes,)))
    return out


def resnet50_shapes(num_classes: int = 1000) -> List[Shape]:
    """ResNet-50, bottleneck blocks [3,4,6,3], expansion 4 (161 tensors)."""
    out: List[Shape] = [("conv1.weight", (64, 3, 7, 7))] + _bn("bn1", 64)
    cin = 64
    for stage, (width, blocks) in enumerate(
            zip((64, 128, 256, 512), (3, 4, 6, 3)), start=1):
        for block in range(blocks):
            p = f"layer{stage}.{block}"
            out.append((f"{p}.conv1.weight", (width, cin, 1, 1)))
            out += _bn(f"{p}.bn1", width)
            out.append((f"{p}.conv2.weight", (width, width, 3, 3)))
            out += _bn(f"{p}.bn2", width)
            out.append((f"{p}.conv3.weight", (4 * width, width, 1, 1)))
            out += _bn(f"{p}.bn3", 4 * width)
            if block == 0:
                out.append((f"{p}.downsample.0.weight", (4 * width, cin, 1, 1)))
                out += _bn(f"{p}.downsample.1", 4 * width)
            cin = 4 * width
    out.append(("fc.weight", (num_classes, 2048)))
    out.append(("fc.bias", (num_classes,)))
    return out


def gpt2_small_shapes(vocab: int = 50257, ctx: int = 1024, d: int = 768,
                      layers: int = 12) -> List[Shape]:
    """GPT-2 small: token + position embeddings, 12 blocks, final LN (148 tensors)."""
    out: List[Shape] = [("wte.weight", (vocab, d)), ("wpe.weight", (ctx, d))]
    for i in range(layers):
        p = f"h.{i}"
        out += _bn(f"{p}.ln_1", d)
        out += [(f"{p}.attn.c_attn.weight", (d, 3 * d)), (f"{p}.attn.c_attn.bias", (3 * d,))]
        out += [(f"{p}.attn.c_proj.weight", (d, d)), (f"{p}.attn.c_proj.bias", (d,))]
        out += _bn(f"{p}.ln_2", d)
        out += [(f"{p}.mlp.c_fc.weight", (d, 4 * d)), (f"{p}.mlp.c_fc.bias", (4 * d,))]
        out += [(f"{p}.mlp.c_proj.weight", (4 * d, d)), (f"{p}.mlp.c_proj.bias", (d,))]
    out += _bn("ln_f", d)
    return out


def sizes(shapes: List[Shape]) -> List[int]:
    return [prod(s) for _, s in shapes]
