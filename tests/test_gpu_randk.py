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


# ---------------------------------------------------------------------------------------------
# Seeded draw (liec_draw_subsets): both sides draw the subsets from (seed, epoch), each with its own
# implementation of the generator and of the ranking; the uplink and downlink messages carry the
# index lists, so comparing the messages compares the subsets of all N workers and of the server.
# ---------------------------------------------------------------------------------------------

def _seeded_steps(P, N, off, steps, seed, dist="normal", scale=1.0, staged=False):
    for step in range(steps):
        G = make_gradients(dist, scale, N, int(off[-1]), step, base_seed=seed & 0xffff)
        P.step(G, 0.05, staged=staged, draw=(seed, step))


def test_seeded_draw_ragged_segments():
    """One element up to several tiles with ragged tails, k_t = n_t, k_t = 1, single-tile and multi-tile."""
    off = np.asarray([0, 1, 6, 8192 + 6, 8192 + 6 + 33, 4 * 8192 + 7, 4 * 8192 + 7 + 20000, 4 * 8192 + 7 + 20000 + 8192], np.int64)
    k = np.asarray([1, 2, 700, 33, 911, 1, 8192], np.int64)
    P = Pair(3, off, RANDK, RANDK, k=k)
    _seeded_steps(P, 3, off, 5, seed=0x9e3779b97f4a7c15)


def test_seeded_draw_resnet50_list_shrunk():
    lay = scaled_layout(resnet50_layout(), 16)
    k = topk_counts(lay, 1, 100)
    P = Pair(16, lay.seg_offsets, RANDK, RANDK, k=k)
    _seeded_steps(P, 16, lay.seg_offsets, 3, seed=12345, dist="student_t3", scale=1e-3)


@pytest.mark.parametrize("up,down", [(RANDK, SIGN), (TOPK, RANDK), (RANDK, IDENT)])
def test_seeded_draw_mixed_with_other_operators(up, down):
    off = np.asarray([0, 5000, 5000 + 3 * 8192 + 11, 5000 + 3 * 8192 + 11 + 12345], np.int64)
    k = np.asarray([50, 800, 123], np.int64)
    P = Pair(4, off, up, down, k=k)
    _seeded_steps(P, 4, off, 3, seed=(7 << 32) | 5, staged=True)


def test_seeded_draw_small_fractions_and_large_k():
    """k_t far below n_t / 2048 (the expected-threshold bound is then finer than a first-digit bin),
    k_t = n_t / 2 and k_t = n_t - 1 on multi-tile segments: every route of the selection."""
    n = 40 * 8192 + 123
    off = np.asarray([0, n, 2 * n, 3 * n, 4 * n], np.int64)
    k = np.asarray([1, 37, n // 2, n - 1], np.int64)
    P = Pair(2, off, RANDK, RANDK, k=k)
    _seeded_steps(P, 2, off, 3, seed=2024)
    routes = P.ctx  # (the subsets were compared through the messages above)


def test_seeded_draw_is_a_function_of_seed_epoch_row_segment():
    """Same (seed, epoch): same lists; another epoch or seed: other lists; keeping the lists for several
    iterations is allowed; liec_set_subsets replaces them."""
    off = np.asarray([0, 3 * 8192 + 5, 3 * 8192 + 5 + 900], np.int64)
    k = np.asarray([300, 9], np.int64)
    N = 3
    X = torch.zeros(N, int(off[-1]), device=DEV)
    e = torch.zeros(int(off[-1]), device=DEV)
    ctx = liec.Context(X, e, off, RANDK, RANDK, k)
    G = make_gradients("normal", 1.0, N, int(off[-1]), 0, base_seed=9).to(DEV)

    def lists(seed, epoch, draw=True):
        if draw:
            ctx.liec_draw_subsets(seed, epoch)
        ctx.liec_step(G, 0.1)
        torch.cuda.synchronize()
        m = ctx.liec_get_messages()
        return m["up_idx"].cpu().numpy().copy(), m["down_idx"].cpu().numpy().copy()

    a = lists(1, 0)
    b = lists(1, 0)
    c = lists(1, 0, draw=False)        # kept for another iteration
    d = lists(1, 1)
    f = lists(2, 0)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and np.array_equal(a[0], c[0])
    assert not np.array_equal(a[0], d[0]) and not np.array_equal(a[0], f[0]) and not np.array_equal(a[1], d[1])
    want = oracle.draw_subsets(2, 0, N + 1, off, k)
    assert np.array_equal(f[0].view(np.uint32), want[:N]) and np.array_equal(f[1].view(np.uint32), want[N])
    assert ctx.liec_device_status() == 0
    with pytest.raises(liec.LiecError):      # a configuration without random-k has nothing to draw
        liec.Context(X, e, off, SIGN, SIGN).liec_draw_subsets(1, 0)


def test_seeded_draw_on_a_segment_beyond_the_one_cta_limits():
    """A segment of 1100 tiles whose candidate buffer exceeds 2^17 entries: the selection runs as wide
    launches (candidate histograms, count, scan, write) instead of one CTA per problem."""
    n = 1100 * 8192 + 17
    off = np.asarray([0, n, n + 5000], np.int64)
    k = np.asarray([90000, 50], np.int64)
    N = 1
    X = torch.zeros(N, int(off[-1]), device=DEV)
    e = torch.zeros(int(off[-1]), device=DEV)
    ctx = liec.Context(X, e, off, RANDK, RANDK, k)
    G = make_gradients("normal", 1.0, N, int(off[-1]), 0, base_seed=11).to(DEV)
    for epoch in (0, 1):
        ctx.liec_draw_subsets(77, epoch)
        ctx.liec_step(G, 0.1)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        m = ctx.liec_get_messages()
        want = oracle.draw_subsets(77, epoch, N + 1, off, k)
        assert np.array_equal(m["up_idx"].cpu().numpy().view(np.uint32), want[:N])
        assert np.array_equal(m["down_idx"].cpu().numpy().view(np.uint32), want[N])
