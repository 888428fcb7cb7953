"""Segments of more than 2048 tiles (16.7 M elements): the tile partials of such a segment are
combined chunk by chunk (2048 tiles, then the chunk sums), a path that the benchmark workloads
take (the 38.6 M-element embedding of the GPT-2 list, every flat vector from 2^25) and that the
small cases never reach.  Everything here is compared with the oracle bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_helpers import Pair, f32, widen
from liec_synth import make_gradients
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu

SIGN = liec.COMP_SCALED_SIGN
BIG = 2049 * 8192 + 5          # 2050 tiles: one full chunk, a second chunk of two tiles, a ragged tail
OFF = [0, BIG, BIG + 1000]


@pytest.mark.parametrize("dist,gdt", [("normal", liec.F32), ("bf16_outliers", liec.BF16)])
def test_sign_step_with_a_segment_of_more_than_2048_tiles(dist, gdt):
    P = Pair(2, OFF, SIGN, SIGN, grad_dtype=gdt)
    for step in range(2):
        G = make_gradients(dist, 0.01, 2, OFF[-1], step, base_seed=61)
        P.step(G, 0.05)


def test_sumsq_on_a_segment_of_more_than_2048_tiles():
    """Squared norms of e, g and x per segment, raw binary64 sums: a wrong order shows in the bits."""
    N, d = 2, OFF[-1]
    G = make_gradients("normal", 1.0, N, d, 0, base_seed=62)
    X = (make_gradients("normal", 3.0, N, d, 1, base_seed=62)).cuda()
    e = make_gradients("normal", 0.5, 1, d, 2, base_seed=62)[0].contiguous().cuda()
    ctx = liec.Context(X, e, OFF, SIGN, SIGN)
    Gd = G.cuda()
    for which, rows, src in ((liec.SUMSQ_ERROR, 1, e.view(1, d)), (liec.SUMSQ_GRADS, N, Gd), (liec.SUMSQ_PARAMS, N, X)):
        out = torch.zeros(rows, 2, dtype=torch.float64, device="cuda")
        ctx.liec_sumsq(which, out, grads=Gd if which == liec.SUMSQ_GRADS else None)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        h = f32(src)
        for r in range(rows):
            for t in range(2):
                want = oracle.tree_sumsq(h[r, OFF[t]:OFF[t + 1]])
                assert got[r, t] == want, (which, r, t, got[r, t], want)
