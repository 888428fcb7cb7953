"""Parity at the full benchmark sizes (C2, C3, C4), in the launch configuration bench.py times.

The oracle cannot run a whole C3/C4 step in reasonable time, but every stage of the step is
local to a segment (element-wise work plus per-segment reductions and selections), so the oracle
is run on a sample of whole segments with all N workers, and the library's outputs restricted
to those segments must match it bit for bit.  Properties that hold at any size are checked over
all segments on the device."""
import numpy as np
import pytest
import torch

import oracle
from gpu_helpers import assert_close, f32, u32, widen
from liec_synth import WORKLOADS, make_gradients, random_subsets, topk_counts
from paper_2402_11857_b200 import liec

pytestmark = pytest.mark.gpu


def _sample_segments(lay, budget_elems):
    """A spread of segments by size (largest that fits, median, small ones) within an element budget."""
    order = sorted(range(lay.num_segments), key=lambda t: -lay.sizes[t])
    chosen, total = [], 0
    for t in order[:: max(1, lay.num_segments // 12)] + order[-3:]:
        if t not in chosen and total + lay.sizes[t] <= budget_elems:
            chosen.append(t)
            total += lay.sizes[t]
    return sorted(chosen)


def _pack_negative(x):
    """Sign words by the definition, on the device: bit b of word w is set iff x[32w+b] < 0 (int64 tensor)."""
    n = x.numel()
    neg = torch.zeros(((n + 31) // 32) * 32, dtype=torch.bool, device=x.device)
    neg[:n] = x < 0
    return (neg.view(-1, 32).to(torch.int64) << torch.arange(32, device=x.device)).sum(dim=1)


def _check_whole_segment_sign(ctx, m, G, v_seg, lay, t, woff):
    """One segment too large for an oracle step with all workers (the 38.6 M-element embedding):
    every worker's scale and the server's against the oracle's scale of the same bytes, the words
    against the definition."""
    off = lay.seg_offsets
    lo, hi = int(off[t]), int(off[t + 1])
    for i in range(G.shape[0]):
        want = oracle.scale(widen(G[i, lo:hi]))
        got = f32(m["up_scales"][i, t:t + 1])[0]
        assert np.float32(got).view(np.uint32) == np.float32(want).view(np.uint32), ("up scale", i, got, want)
        words = m["up_words"][i, woff[t]:woff[t + 1]].to(torch.int64) & 0xFFFFFFFF
        assert torch.equal(words, _pack_negative(G[i, lo:hi].float())), ("up words", i)
    want = oracle.scale(f32(v_seg))
    got = f32(m["down_scales"][t:t + 1])[0]
    assert np.float32(got).view(np.uint32) == np.float32(want).view(np.uint32), ("down scale", got, want)
    words = m["down_words"][woff[t]:woff[t + 1]].to(torch.int64) & 0xFFFFFFFF
    assert torch.equal(words, _pack_negative(v_seg)), "down words"


def _run(name, steps, budget_elems, randk=False, whole_segment=None, routes=None):
    w = WORKLOADS[name]
    lay = w.layout()
    N, d, off = w.num_workers, lay.dim, lay.seg_offsets
    comp = liec.COMP_SCALED_SIGN if w.compressor == "sign" else liec.COMP_TOPK
    ocomp = oracle.SIGN if w.compressor == "sign" else oracle.TOPK
    if randk:   # the same tensor list and k_t with random-k (Def. 3) both ways
        comp, ocomp = liec.COMP_RANDK, oracle.RANDK
    k = topk_counts(lay, *w.topk_frac) if w.compressor == "topk" else None
    gdt = liec.BF16 if w.grad_dtype == "bf16" else liec.F32
    X = torch.zeros(N, d, device="cuda")
    e = torch.zeros(d, device="cuda")
    ctx = liec.Context(X, e, off, comp, comp, k, gdt)
    G = torch.empty(N, d, device="cuda", dtype=torch.bfloat16 if gdt == liec.BF16 else torch.float32)

    segs = _sample_segments(lay, budget_elems)
    sub_sizes = [lay.sizes[t] for t in segs]
    sub_off = np.concatenate([[0], np.cumsum(sub_sizes)]).astype(np.int64)
    cols = torch.cat([torch.arange(off[t], off[t + 1], device="cuda") for t in segs])
    Xh = np.zeros((N, int(sub_off[-1])), np.float32)
    eh = np.zeros(int(sub_off[-1]), np.float32)
    ksub = None if k is None else k[segs]
    woff = np.concatenate([[0], np.cumsum((np.diff(off) + 31) // 32)])
    koff = None if k is None else np.concatenate([[0], np.cumsum(k)])

    for step in range(steps):
        make_gradients(w.dist, w.scale, N, d, step, base_seed=77, device="cuda", out=G)
        sub_sets = {}
        if randk:
            sets = random_subsets(off, k, N + 1, step, 78)
            sets_dev = torch.from_numpy(sets.view(np.int32)).cuda()
            ctx.liec_set_subsets(sets_dev[:N].contiguous(), sets_dev[N].contiguous())
            # the sampled segments' part of every subset, re-based to the sample's own offsets
            part = np.concatenate([sets[:, koff[t]:koff[t + 1]].astype(np.int64) - (int(off[t]) - int(sub_off[q]))
                                   for q, t in enumerate(segs)], axis=1).astype(np.uint32)
            sub_sets = dict(up_sets=part[:N], down_set=part[N])
        v_seg = None
        if whole_segment is not None and step == steps - 1:
            # staged, so that v of the large segment can be read before the downlink overwrites it
            ctx.liec_uplink_compress(G)
            ctx.liec_server_aggregate()
            torch.cuda.synchronize()
            v_seg = e[int(off[whole_segment]):int(off[whole_segment + 1])].clone()
            ctx.liec_downlink_compress()
            ctx.liec_worker_update(G, w.lr)
        else:
            ctx.liec_step(G, w.lr)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        m = ctx.liec_get_messages()
        if v_seg is not None:
            _check_whole_segment_sign(ctx, m, G, v_seg, lay, whole_segment, woff)
        if routes is not None:
            routes.append((ctx.liec_topk_route_counts(True), ctx.liec_topk_route_counts(False)))
        r = oracle.step(Xh, eh, widen(G[:, cols]), w.lr, sub_off, ocomp, ocomp, k=ksub, **sub_sets)
        assert_close(f32(X[:, cols]), Xh, f"{name} step {step}: params on sampled segments")
        assert_close(f32(e[cols]), eh, f"{name} step {step}: error on sampled segments")
        if comp == liec.COMP_SCALED_SIGN:
            sub_woff = np.concatenate([[0], np.cumsum((np.diff(sub_off) + 31) // 32)])
            for q, t in enumerate(segs):
                got = u32(m["up_words"][:, woff[t]:woff[t + 1]])
                assert np.array_equal(got, r.up_words[:, sub_woff[q]:sub_woff[q + 1]]), (name, step, t, "up words")
                assert np.array_equal(u32(m["down_words"][woff[t]:woff[t + 1]]), r.down_words[sub_woff[q]:sub_woff[q + 1]])
            assert np.array_equal(f32(m["up_scales"])[:, segs].view(np.uint32), r.up_scales.view(np.uint32))
            assert np.array_equal(f32(m["down_scales"])[segs].view(np.uint32), r.down_scales.view(np.uint32))
            # any size: one bit per negative gradient, over all segments and workers
            neg = (G < 0).sum(dim=1).cpu().numpy()
            pop = np.array([int(np.unpackbits(u32(m["up_words"][i]).view(np.uint8)).sum()) for i in range(0, N, max(1, N // 4))])
            assert np.array_equal(pop, neg[:: max(1, N // 4)])
        else:
            sub_koff = np.concatenate([[0], np.cumsum(ksub)])
            for q, t in enumerate(segs):
                shift = int(off[t]) - int(sub_off[q])
                got = u32(m["up_idx"][:, koff[t]:koff[t + 1]]).astype(np.int64) - shift
                assert np.array_equal(got, r.up_idx[:, sub_koff[q]:sub_koff[q + 1]].astype(np.int64)), (name, step, t, "up idx")
                gotd = u32(m["down_idx"][koff[t]:koff[t + 1]]).astype(np.int64) - shift
                assert np.array_equal(gotd, r.down_idx[sub_koff[q]:sub_koff[q + 1]].astype(np.int64)), (name, step, t, "down idx")
            if randk:
                # any size: the message is the subset itself and the values found there, for every worker
                assert torch.equal(m["up_idx"].view(torch.int32), sets_dev[:N]) and torch.equal(m["down_idx"].view(torch.int32), sets_dev[N])
                assert torch.equal(m["up_val"], torch.gather(G.float(), 1, sets_dev[:N].long()))
                assert bool((e[sets_dev[N].long()] == 0).all())
                continue
            # any size: per segment exactly k_t indices, ascending and inside the segment (worker 0 and N-1)
            for i in (0, N - 1):
                idx = u32(m["up_idx"][i]).astype(np.int64)
                seg_of = np.repeat(np.arange(lay.num_segments), k)
                assert np.all(idx >= off[seg_of]) and np.all(idx < off[seg_of + 1])
                inner = np.ones(len(idx), bool); inner[koff[:-1]] = False
                assert np.all(np.diff(idx)[inner[1:]] > 0)
                # kept magnitudes dominate the dropped ones in the largest segment
                t = int(np.argmax(lay.sizes))
                g = G[i, off[t]:off[t + 1]].float().abs()
                kept = torch.zeros_like(g, dtype=torch.bool)
                kept[torch.from_numpy(idx[koff[t]:koff[t + 1]] - off[t]).cuda()] = True
                assert g[kept].min() >= g[~kept].max()


def test_c2_resnet18_sign_full_size():
    _run("c2", steps=10, budget_elems=4_000_000)


def test_c3_resnet50_topk_full_size():
    """20 iterations on fresh gradients: error feedback has piled v up under the thresholds and the
    uplink runs on the thresholds of the step before."""
    routes = []
    _run("c3", steps=20, budget_elems=3_500_000, routes=routes)
    up, down = routes[-1]
    assert up["problems"] == 16 * 161 and down["problems"] == 161
    # about two thirds of the 161 tensors fit one tile and are selected directly; after the first step nearly all
    # the others finish on the single pass seeded by the previous threshold
    small = sum(1 for n in WORKLOADS["c3"].layout().sizes if n <= 8192)
    large = 161 - small
    assert all(u["direct"] == 16 * small and dn["direct"] == small for u, dn in routes)
    print("c3 routes per step (uplink single-pass of %d, uplink refined, downlink refined):" % (16 * large),
          [(u["single_pass"], u["refined"], dn["refined"]) for u, dn in routes])
    assert all(u["single_pass"] >= 0.9 * 16 * large for u, _ in routes[2:]), [u for u, _ in routes]
    assert all(u["slow"] == 0 and dn["slow"] == 0 for u, dn in routes)


def test_c4_gpt2_sign_bf16_full_size():
    _run("c4", steps=5, budget_elems=4_000_000, whole_segment=0)


def test_c3_resnet50_randk_full_size():
    _run("c3", steps=2, budget_elems=3_500_000, randk=True)


def test_c3_resnet50_seeded_randk_full_size():
    """The seeded draw at full size (N = 16 workers + the server, 161 tensors): the subsets of sampled
    (row, segment) pairs against the oracle's own draw; for all rows and segments, what holds at any
    size (k_t ascending indices inside the segment); then a whole iteration on them."""
    w = WORKLOADS["c3"]
    lay = w.layout()
    N, d, off = w.num_workers, lay.dim, lay.seg_offsets
    k = topk_counts(lay, *w.topk_frac)
    koff = np.concatenate([[0], np.cumsum(k)])
    X = torch.zeros(N, d, device="cuda")
    e = torch.zeros(d, device="cuda")
    ctx = liec.Context(X, e, off, liec.COMP_RANDK, liec.COMP_RANDK, k)
    G = make_gradients(w.dist, w.scale, N, d, 0, base_seed=79, device="cuda")
    seed = 0xC0FFEE1234567
    for epoch in (0, 1):
        ctx.liec_draw_subsets(seed, epoch)
        ctx.liec_step(G, w.lr)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        m = ctx.liec_get_messages()
        lists = np.concatenate([u32(m["up_idx"]), u32(m["down_idx"])[None, :]], axis=0)   # rows 0..N-1, then the server
        seg_of = np.repeat(np.arange(lay.num_segments), k)
        inner = np.ones(lists.shape[1], bool)
        inner[koff[:-1]] = False
        for row in range(N + 1):
            idx = lists[row].astype(np.int64)
            assert np.all(idx >= off[seg_of]) and np.all(idx < off[seg_of + 1]), row
            assert np.all(np.diff(idx)[inner[1:]] > 0), row
        assert len({lists[row].tobytes() for row in range(N + 1)}) == N + 1          # every row has its own subsets
        # sampled (row, segment) pairs: the largest tensor once, a spread of the others over the rows
        segs = _sample_segments(lay, 5_000_000)
        for q, t in enumerate(segs):
            for row in {q % (N + 1), N}:
                n = int(off[t + 1] - off[t])
                want = oracle.subset_from_scores(oracle.subset_scores(seed, epoch, row, t, n), int(k[t])).astype(np.int64) + int(off[t])
                assert np.array_equal(lists[row, koff[t]:koff[t + 1]].astype(np.int64), want), (epoch, row, t)
        # the messages carry the values found at the subsets
        assert torch.equal(m["up_val"], torch.gather(G, 1, m["up_idx"].long()))


def _assert_is_the_topk_set(x, idx, k):
    """idx (ascending int64, device) is THE top-k set of |x| with ties to the lower index: checked from
    the definition with library primitives (k-th largest magnitude by torch.kthvalue)."""
    n = x.numel()
    mag = x.abs()
    assert idx.numel() == k and bool((idx[1:] > idx[:-1]).all()) and int(idx[0]) >= 0 and int(idx[-1]) < n
    thr = torch.kthvalue(mag, n - k + 1).values            # the k-th largest magnitude
    kept = torch.zeros(n, dtype=torch.bool, device=x.device)
    kept[idx] = True
    assert bool((mag[kept] >= thr).all()) and bool((mag[~kept] <= thr).all())
    ties = mag == thr
    kept_ties, dropped_ties = torch.nonzero(ties & kept).flatten(), torch.nonzero(ties & ~kept).flatten()
    assert int((mag > thr).sum()) + kept_ties.numel() == k
    if dropped_ties.numel():
        assert int(kept_ties.max()) < int(dropped_ties.min()) if kept_ties.numel() else True


def test_c5_flat_2p28_topk_one_percent_full_size():
    """The 2^28 point of the bandwidth sweep (N = 8, one flat vector, k = 1 %), as bench.py runs it: far
    beyond what the oracle finishes, so every stage is checked on the device against its definition
    written with torch's elementwise operations, kthvalue and scatter (IEEE binary32, no contraction):
    the top-k sets of two workers and of the server, v = e + (sum in worker order) / N, e' = v off the
    kept set, and x <- x - lr ((p - p^i) + g) for two workers, all bit for bit; two iterations, so that
    the second one runs on a non-zero e and on the single-pass route."""
    n, N, lr = 1 << 28, 8, 0.1
    k = n // 100
    off = np.asarray([0, n], np.int64)
    X = torch.zeros(N, n, device="cuda")
    e = torch.zeros(n, device="cuda")
    ctx = liec.Context(X, e, off, liec.COMP_TOPK, liec.COMP_TOPK, np.asarray([k], np.int64))
    G = torch.empty(N, n, device="cuda")
    for step in range(2):
        make_gradients("normal", 1.0, N, n, step, base_seed=81, device="cuda", out=G)
        e_before = e.clone()
        x_before = {i: X[i].clone() for i in (0, N - 1)}
        ctx.liec_uplink_compress(G)
        ctx.liec_server_aggregate()
        torch.cuda.synchronize()
        v = e.clone()
        m = ctx.liec_get_messages()
        up_idx = m["up_idx"].to(torch.int64) & 0xFFFFFFFF
        for i in (0, N - 1):
            _assert_is_the_topk_set(G[i], up_idx[i], k)
            assert torch.equal(m["up_val"][i], G[i][up_idx[i]])
        acc = torch.zeros(n, device="cuda")
        for i in range(N):                       # worker order; adding an absent entry's +0 changes nothing
            p_i = torch.zeros(n, device="cuda")
            p_i[up_idx[i]] = m["up_val"][i]
            acc = acc + p_i
        want_v = e_before + acc / N
        assert torch.equal(v.view(torch.int32), want_v.view(torch.int32)), f"v, step {step}"
        del acc, want_v, p_i
        ctx.liec_downlink_compress()
        ctx.liec_worker_update(G, lr)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        m = ctx.liec_get_messages()
        down_idx = m["down_idx"].to(torch.int64) & 0xFFFFFFFF
        _assert_is_the_topk_set(v, down_idx, k)
        assert torch.equal(m["down_val"], v[down_idx])
        p = torch.zeros(n, device="cuda")
        p[down_idx] = m["down_val"]
        want_e = v.clone()
        want_e[down_idx] = 0.0
        assert torch.equal(e.view(torch.int32), want_e.view(torch.int32)), f"e', step {step}"
        del want_e
        for i in (0, N - 1):
            p_i = torch.zeros(n, device="cuda")
            p_i[up_idx[i]] = m["up_val"][i]
            u = (p - p_i) + G[i]
            want_x = x_before[i] - u * lr
            assert torch.equal(X[i].view(torch.int32), want_x.view(torch.int32)), f"x^{i}, step {step}"
            del p_i, u, want_x
        routes = ctx.liec_topk_route_counts(True)
        assert routes["problems"] == N and routes["slow"] == 0
        if step == 1:
            assert routes["single_pass"] == N, routes     # the bound under the first step's thresholds held


def test_c5_flat_2p28_sign_full_size():
    """The 2^28 sign point of the sweep: the scales of one worker and of the server against the oracle's
    scale of the same bytes, every sign word against the definition, v and x against the update rules
    written with torch's elementwise operations (bit for bit)."""
    n, N, lr = 1 << 28, 8, 0.1
    off = np.asarray([0, n], np.int64)
    X = torch.zeros(N, n, device="cuda")
    e = torch.zeros(n, device="cuda")
    ctx = liec.Context(X, e, off, liec.COMP_SCALED_SIGN, liec.COMP_SCALED_SIGN)
    G = torch.empty(N, n, device="cuda")
    for step in range(2):
        make_gradients("normal", 1.0, N, n, step, base_seed=82, device="cuda", out=G)
        e_before = e.clone()
        x_before = X[N - 1].clone()
        ctx.liec_uplink_compress(G)
        ctx.liec_server_aggregate()
        torch.cuda.synchronize()
        v = e.clone()
        ctx.liec_downlink_compress()
        ctx.liec_worker_update(G, lr)
        torch.cuda.synchronize()
        assert ctx.liec_device_status() == 0
        m = ctx.liec_get_messages()
        s_up = m["up_scales"][:, 0]
        want = oracle.scale(f32(G[N - 1]))
        assert np.float32(f32(s_up[N - 1:N])[0]).view(np.uint32) == np.float32(want).view(np.uint32)
        for i in range(N):
            assert torch.equal(m["up_words"][i].to(torch.int64) & 0xFFFFFFFF, _pack_negative(G[i])), ("up words", i)
        acc = torch.zeros(n, device="cuda")
        for i in range(N):                       # worker order
            acc = acc + torch.where(G[i] < 0, -s_up[i], s_up[i])
        want_v = e_before + acc / N
        assert torch.equal(v.view(torch.int32), want_v.view(torch.int32)), f"v, step {step}"
        del acc, want_v
        s_down = m["down_scales"][0]
        want = oracle.scale(f32(v))
        assert np.float32(f32(m["down_scales"][0:1])[0]).view(np.uint32) == np.float32(want).view(np.uint32)
        assert torch.equal(m["down_words"].to(torch.int64) & 0xFFFFFFFF, _pack_negative(v)), "down words"
        p = torch.where(v < 0, -s_down, s_down)
        assert torch.equal(e.view(torch.int32), (v - p).view(torch.int32)), f"e', step {step}"
        p_i = torch.where(G[N - 1] < 0, -s_up[N - 1], s_up[N - 1])
        want_x = x_before - ((p - p_i) + G[N - 1]) * lr
        assert torch.equal(X[N - 1].view(torch.int32), want_x.view(torch.int32)), f"x, step {step}"
        del p, p_i, want_x
