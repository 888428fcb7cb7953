"""Runs the CUDA library and the CPU oracle side by side on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2402_11857_b200 import liec

DEV = "cuda:0"


def u32(t):
    """torch int32 tensor -> numpy uint32."""
    return t.detach().cpu().numpy().view(np.uint32)


def f32(t):
    return t.detach().cpu().numpy()


def widen(G: torch.Tensor) -> np.ndarray:
    """Gradient tensor (f32 or bf16, any device) -> float32 numpy via the oracle's exact widening."""
    if G.dtype == torch.bfloat16:
        bits = G.detach().cpu().view(torch.int16).numpy().view(np.uint16)
        return oracle.widen_bf16(bits)
    return G.detach().cpu().numpy()


class Pair:
    """One problem instance held twice: on the GPU (library) and on the host (oracle)."""

    def __init__(self, N, off, up, down, k=None, grad_dtype=liec.F32, x0=None, e0=None):
        self.off = np.asarray(off, dtype=np.int64)
        self.N, self.d = N, int(self.off[-1])
        self.up, self.down, self.k = up, down, (None if k is None else np.asarray(k, np.int64))
        self.Xh = np.zeros((N, self.d), np.float32) if x0 is None else np.tile(np.asarray(x0, np.float32), (N, 1)).copy()
        self.eh = np.zeros(self.d, np.float32) if e0 is None else np.asarray(e0, np.float32).copy()
        self.Xd = torch.from_numpy(self.Xh.copy()).to(DEV)
        self.ed = torch.from_numpy(self.eh.copy()).to(DEV)
        self.ctx = liec.Context(self.Xd, self.ed, self.off, up, down, self.k, grad_dtype)

    def step(self, G: torch.Tensor, lr: float, staged: bool = False, check_messages: bool = True,
             up_sets=None, down_set=None, draw=None):
        """Runs one iteration on both sides and asserts parity of messages and state.
        up_sets [N,K] / down_set [K] (numpy uint32): the subsets of a random-k side; or
        draw = (seed, epoch): both sides draw them from the seed, each with its own code."""
        Gd = G.to(DEV).contiguous()
        if draw is not None:
            sets = oracle.draw_subsets(draw[0], draw[1], self.N + 1, self.off, self.k)
            r = oracle.step(self.Xh, self.eh, widen(G), lr, self.off, self.up, self.down, k=self.k,
                            up_sets=sets[:self.N], down_set=sets[self.N])
            self.ctx.liec_draw_subsets(draw[0], draw[1])
            return self._gpu_step_and_compare(Gd, lr, r, staged, check_messages)
        r = oracle.step(self.Xh, self.eh, widen(G), lr, self.off, self.up, self.down, k=self.k,
                        up_sets=up_sets, down_set=down_set)
        if up_sets is not None or down_set is not None:
            as_dev = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a).view(np.int32)).to(DEV)
            self.ctx.liec_set_subsets(as_dev(up_sets), as_dev(down_set))
        return self._gpu_step_and_compare(Gd, lr, r, staged, check_messages)

    def _gpu_step_and_compare(self, Gd, lr, r, staged, check_messages):
        if staged or check_messages:
            self.ctx.liec_uplink_compress(Gd)
            self.ctx.liec_server_aggregate()
            torch.cuda.synchronize()
            v = f32(self.ed).copy()
            self.ctx.liec_downlink_compress()
            self.ctx.liec_worker_update(Gd, lr)
        else:
            v = None
            self.ctx.liec_step(Gd, lr)
        torch.cuda.synchronize()
        assert self.ctx.liec_device_status() == 0
        m = self.ctx.liec_get_messages()
        if check_messages:
            if self.up == oracle.SIGN:
                assert np.array_equal(u32(m["up_words"]), r.up_words), "uplink sign words"
                assert np.array_equal(f32(m["up_scales"]).view(np.uint32), r.up_scales.view(np.uint32)), "uplink scales"
            if self.up in (oracle.TOPK, oracle.RANDK):
                assert np.array_equal(u32(m["up_idx"]), r.up_idx), "uplink top-k indices"
                assert np.array_equal(f32(m["up_val"]).view(np.uint32), r.up_val.view(np.uint32)), "uplink top-k values"
            if self.down == oracle.SIGN:
                assert np.array_equal(u32(m["down_words"]), r.down_words), "downlink sign words"
                assert np.array_equal(f32(m["down_scales"]).view(np.uint32), r.down_scales.view(np.uint32)), "downlink scales"
            if self.down in (oracle.TOPK, oracle.RANDK):
                assert np.array_equal(u32(m["down_idx"]), r.down_idx), "downlink top-k indices"
                assert np.array_equal(f32(m["down_val"]).view(np.uint32), r.down_val.view(np.uint32)), "downlink top-k values"
        if v is not None:
            assert_close(v, r.v, "v")
        assert_close(f32(self.ed), self.eh, "global error e")
        assert_close(f32(self.Xd), self.Xh, "params X")
        return r


def max_rel_err(a: np.ndarray, b: np.ndarray) -> float:
    """max_j |a_j - b_j| / max(|b_j|, 1e-6 * max|b|): the bar is 1e-5 for binary32 state."""
    a64, b64 = a.astype(np.float64).ravel(), b.astype(np.float64).ravel()
    if a64.size == 0:
        return 0.0
    floor = 1e-6 * max(np.max(np.abs(b64)), 1e-30)
    return float(np.max(np.abs(a64 - b64) / np.maximum(np.abs(b64), floor)))


REL_TOL = 1e-5   # fp32 parameters and errors must agree within this relative error after each step


def assert_close(a, b, what, tol=REL_TOL, exact=True):
    err = max_rel_err(a, b)
    assert err <= tol, f"{what}: max relative error {err:.3e} > {tol}"
    if exact:
        # the arithmetic is fixed operation by operation, so the bits are expected to agree too
        bad = int(np.count_nonzero(a.view(np.uint32) != b.view(np.uint32)))
        assert bad == 0, f"{what}: {bad} of {a.size} values differ in their bits (max rel err {err:.3e})"
