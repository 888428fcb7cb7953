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
