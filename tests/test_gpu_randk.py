"""Random-k (Def. 3) on the GPU against the oracle: the subsets are drawn once on the host and
given to both sides; messages, v, the global error and the models must agree bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from liec_synth import make_gradients, random_subsets, ragged_layout, resnet50_layout, scaled_layout, topk_counts
from paper_2402_11857_b200 import liec

from gpu_helpers import DEV, Pair

pytestmark = pytest.mark.gpu

IDENT, SIGN, TOPK, RANDK = oracle.IDENTITY, oracle.SIGN, oracle.TOPK, oracle.RANDK


def _steps(P, N, off, k, steps, base_seed, dist="normal", scale=1.0, staged=False, dtype=None):
    K_up = P.up == RANDK
    K_down = P.down == RANDK
    for step in range(steps):
        G = make_gradients(dist, scale, N, int(off[-1]), step, base_seed=base_seed)
        if dtype is not None:
            G = G.to(dtype)
        up = random_subsets(off, k, N, step, base_seed) if K_up else None
        down = random_subsets(off, k, 1, step, base_seed + 1000)[0] if K_down else None
        P.step(G, 0.05, staged=staged, up_sets=up, down_set=down)


def test_randk_both_ways_ragged_segments():
    """Segments of 1 element up to several tiles with ragged tails, N = 3 (not a power of two)."""
    off = np.asarray([0, 1, 6, 8192 + 6, 8192 + 6 + 33, 4 * 8192 + 7, 4 * 8192 + 7 + 20000], np.int64)
    k = np.asarray([1, 2, 700, 33, 911, 150], np.int64)
    P = Pair(3, off, RANDK, RANDK, k=k)
    _steps(P, 3, off, k, 6, base_seed=301)


def test_randk_resnet50_list_shrunk():
    """ResNet-50 tensor list shrunk 32x, N = 16, heavy-tailed gradients, k = 1 % per tensor."""
    lay = scaled_layout(resnet50_layout(), 32)
    k = topk_counts(lay, 1, 100)
    P = Pair(16, lay.seg_offsets, RANDK, RANDK, k=k)
    _steps(P, 16, lay.seg_offsets, k, 3, base_seed=302, dist="student_t3", scale=1e-3)


@pytest.mark.parametrize("up,down", [(RANDK, SIGN), (RANDK, IDENT), (RANDK, TOPK), (SIGN, RANDK), (TOPK, RANDK), (IDENT, RANDK)])
def test_randk_mixed_with_other_operators(up, down):
    off = np.asarray([0, 5000, 5000 + 3 * 8192 + 11, 5000 + 3 * 8192 + 11 + 12345], np.int64)
    k = np.asarray([50, 800, 123], np.int64)
    P = Pair(4, off, up, down, k=k)
    _steps(P, 4, off, k, 4, base_seed=303, staged=True)


def test_randk_bf16_gradients():
    off = np.asarray([0, 3 * 8192 + 8, 3 * 8192 + 8 + 776], np.int64)
    k = np.asarray([500, 77], np.int64)
    P = Pair(5, off, RANDK, RANDK, k=k, grad_dtype=liec.BF16)
    _steps(P, 5, off, k, 3, base_seed=304, dist="bf16_outliers", scale=1e-2)


def test_randk_every_index_kept_is_the_identity_step():
    off = np.asarray([0, 100, 100 + 8192 + 5], np.int64)
    k = np.diff(off)
    full = np.arange(off[-1], dtype=np.uint32)
    P = Pair(2, off, RANDK, RANDK, k=k)
    Q = Pair(2, off, IDENT, IDENT)
    for step in range(3):
        G = make_gradients("normal", 1.0, 2, int(off[-1]), step, base_seed=305)
        P.step(G, 0.05, up_sets=np.tile(full, (2, 1)), down_set=full)
        Q.step(G, 0.05)
        assert torch.equal(P.Xd, Q.Xd) and torch.equal(P.ed, Q.ed)


def test_randk_refused_subsets_are_flagged_and_stay_in_bounds():
    """An index outside its segment, a repeated index and a descending pair: the status word gets
    bit 16, nothing outside the buffers is touched, and the context works again afterwards."""
    off = np.asarray([0, 9000, 9000 + 8192], np.int64)
    k = np.asarray([4, 3], np.int64)
    N, d = 2, int(off[-1])
    G = make_gradients("normal", 1.0, N, d, 0, base_seed=306).to(DEV)
    good = np.asarray([[1, 5, 100, 8999, 9000, 9100, 17191]] * N, np.uint32)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int32)).to(DEV)
    for bad_row in ([1, 5, 100, 9000, 9001, 9100, 17191],     # first segment reaches into the second
                    [1, 5, 5, 8999, 9000, 9100, 17191],        # repeated
                    [5, 1, 100, 8999, 9000, 9100, 17191],      # descending
                    [1, 5, 100, 8999, 9000, 9100, 4000000000]):  # far outside the vector
        ctx = liec.Context(torch.zeros(N, d, device=DEV), torch.zeros(d, device=DEV), off, RANDK, RANDK, k)
        bad = good.copy()
        bad[1] = np.asarray(bad_row, np.uint32)
        ctx.liec_set_subsets(dev(bad), dev(good[0]))
        ctx.liec_step(G, 0.1)
        assert ctx.liec_device_status() & 16
        assert ctx.liec_device_status() & 16       # sticky until cleared
        ctx.liec_clear_status()
        assert ctx.liec_device_status() == 0
        # the same subsets on the downlink
        ctx = liec.Context(torch.zeros(N, d, device=DEV), torch.zeros(d, device=DEV), off, RANDK, RANDK, k)
        ctx.liec_set_subsets(dev(good), dev(bad[1]))
        ctx.liec_step(G, 0.1)
        assert ctx.liec_device_status() & 16
    ctx = liec.Context(torch.zeros(N, d, device=DEV), torch.zeros(d, device=DEV), off, RANDK, RANDK, k)
    with pytest.raises(liec.LiecError):   # no subset given for a random-k side
        ctx.liec_step(G, 0.1)
    ctx = liec.Context(torch.zeros(N, d, device=DEV), torch.zeros(d, device=DEV), off, RANDK, RANDK, k)
    ctx.liec_set_subsets(dev(good), dev(good[0]))
    ctx.liec_step(G, 0.1)
    assert ctx.liec_device_status() == 0
