"""Segment layouts: how a d-dimensional parameter vector splits into tensors.

Blockwise-SignSGD (Def. 5) and per-tensor top-k (Def. 2 applied tensor by tensor)
act on contiguous blocks of the flattened model.  The layouts below reproduce the
parameter-tensor shapes of three public architectures from their published
descriptions (layer widths, kernel sizes, block counts); only the element counts
matter here, so each tensor is reduced to its size.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import numpy as np


@dataclass(frozen=True)
class Layout:
    name: str
    sizes: tuple  # n_t for every segment t

    @property
    def num_segments(self) -> int:
        return len(self.sizes)

    @property
    def dim(self) -> int:
        return int(sum(self.sizes))

    @property
    def seg_offsets(self) -> np.ndarray:
        off = np.zeros(len(self.sizes) + 1, dtype=np.int64)
        np.cumsum(np.asarray(self.sizes, dtype=np.int64), out=off[1:])
        return off

    def subset(self, segment_ids: Sequence[int], name: str | None = None) -> "Layout":
        """A layout made of the chosen segments only, in the given order."""
        return Layout(name or f"{self.name}[subset]", tuple(self.sizes[t] for t in segment_ids))


def flat_layout(d: int) -> Layout:
    return Layout(f"flat{d}", (int(d),))


def _bn(c: int) -> List[int]:
    return [c, c]  # weight, bias


def resnet18_layout() -> Layout:
    sizes: List[int] = [64 * 3 * 7 * 7] + _bn(64)
    inp = 64
    for stage, width in enumerate((64, 128, 256, 512)):
        for block in range(2):
            sizes += [width * inp * 9] + _bn(width) + [width * width * 9] + _bn(width)
            if block == 0 and stage > 0:
                sizes += [width * inp] + _bn(width)  # 1x1 projection shortcut
            inp = width
    sizes += [512 * 1000, 1000]
    lay = Layout("resnet18", tuple(sizes))
    assert lay.num_segments == 62 and lay.dim == 11_689_512, (lay.num_segments, lay.dim)
    return lay


def resnet50_layout() -> Layout:
    sizes: List[int] = [64 * 3 * 7 * 7] + _bn(64)
    inp = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        out = 4 * width
        for block in range(blocks):
            sizes += [width * inp] + _bn(width)          # 1x1 reduce
            sizes += [width * width * 9] + _bn(width)    # 3x3
            sizes += [out * width] + _bn(out)            # 1x1 expand
            if block == 0:
                sizes += [out * inp] + _bn(out)          # projection shortcut
            inp = out
    sizes += [2048 * 1000, 1000]
    lay = Layout("resnet50", tuple(sizes))
    assert lay.num_segments == 161 and lay.dim == 25_557_032, (lay.num_segments, lay.dim)
    return lay


def gpt2_small_layout() -> Layout:
    h, vocab, ctx, layers = 768, 50257, 1024, 12
    sizes: List[int] = [vocab * h, ctx * h]
    for _ in range(layers):
        sizes += [h, h]                      # ln_1
        sizes += [h * 3 * h, 3 * h]          # attention qkv
        sizes += [h * h, h]                  # attention output projection
        sizes += [h, h]                      # ln_2
        sizes += [h * 4 * h, 4 * h]          # mlp up
        sizes += [4 * h * h, h]              # mlp down
    sizes += [h, h]                          # ln_f
    lay = Layout("gpt2_small", tuple(sizes))
    assert lay.num_segments == 148 and lay.dim == 124_439_808, (lay.num_segments, lay.dim)
    return lay


def scaled_layout(base: Layout, divisor: int, name: str | None = None) -> Layout:
    """Same tensor list with every size divided (rounded up, at least 1).

    Keeps the size spread and the segment count of the architecture while
    shrinking d so that the CPU oracle runs many steps in seconds.
    """
    def shrink(n: int) -> int:
        m = max(1, -(-n // divisor))
        if n % 8 == 0:          # keep the 8-element granularity of the original tensor
            m = -(-m // 8) * 8  # (rows and segments then start 16-byte aligned, as in the full layout)
        return m
    sizes = tuple(shrink(n) for n in base.sizes)
    return Layout(name or f"{base.name}/{divisor}", sizes)


def ragged_layout() -> Layout:
    """Deliberately awkward sizes: 1-element, sub-word, word+1, tile+-1, several tiles + tail."""
    return Layout("ragged", (1, 7, 33, 64, 1000, 8191, 8193, 3 * 8192 + 5, 31, 32, 2 * 8192, 4099))


def equal_blocks_layout(d: int, num_blocks: int, name: str | None = None) -> Layout:
    """d elements cut into num_blocks contiguous blocks of (almost) equal size, the first d % num_blocks
    one element longer: the paper's Blockwise-SignSGD runs split the gradient into 10, 18 or 14 blocks
    without saying how; this is the plain reading."""
    base, extra = divmod(int(d), int(num_blocks))
    assert base >= 1
    return Layout(name or f"blocks{num_blocks}x{d}", tuple(base + (1 if b < extra else 0) for b in range(num_blocks)))


def topk_counts(layout: Layout, num: int, den: int) -> np.ndarray:
    """k_t = max(1, floor(n_t * num / den)) in integer arithmetic."""
    return np.asarray([max(1, (n * num) // den) for n in layout.sizes], dtype=np.int64)
