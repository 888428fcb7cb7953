"""ctypes binding of ``include/liec.h``: same names, argument marshalling only.

PyTorch appears here only as the owner of device memory and streams.  There is no
fallback: if ``libliec.so`` is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

COMP_IDENTITY, COMP_SCALED_SIGN, COMP_TOPK, COMP_RANDK = 0, 1, 2, 3
SUMSQ_ERROR, SUMSQ_GRADS, SUMSQ_PARAMS = 0, 1, 2
F32, BF16 = 0, 1

STATUS_NAMES = {0: "LIEC_OK", 1: "LIEC_ERR_INVALID_ARG", 2: "LIEC_ERR_UNSUPPORTED", 3: "LIEC_ERR_WORKSPACE",
                4: "LIEC_ERR_STATE", 5: "LIEC_ERR_CUDA", 6: "LIEC_ERR_DEVICE_CHECK"}

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libliec.so")
_LIB: Optional[C.CDLL] = None


class LiecError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class liec_config(C.Structure):
    _fields_ = [("num_workers", C.c_int32), ("dim", C.c_int64), ("num_segments", C.c_int32),
                ("seg_offsets", C.POINTER(C.c_int64)), ("uplink", C.c_int32), ("downlink", C.c_int32),
                ("topk_k", C.POINTER(C.c_int64)), ("grad_dtype", C.c_int32)]


class liec_messages(C.Structure):
    _fields_ = [("up_words", C.c_void_p), ("up_scales", C.c_void_p), ("up_idx", C.c_void_p),
                ("up_val", C.c_void_p), ("down_words", C.c_void_p), ("down_scales", C.c_void_p),
                ("down_idx", C.c_void_p), ("down_val", C.c_void_p), ("v", C.c_void_p),
                ("num_words", C.c_int64), ("num_topk", C.c_int64)]


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads libliec.so (built in-tree) and declares every entry point of liec.h."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    p = path or _LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2402_11857_b200.build`")
    lib = C.CDLL(p)
    vp, cfgp = C.c_void_p, C.POINTER(liec_config)
    lib.liec_workspace_bytes.argtypes = [cfgp]
    lib.liec_workspace_bytes.restype = C.c_size_t
    lib.liec_wire_bytes.argtypes = [cfgp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.liec_wire_bytes.restype = C.c_int
    lib.liec_down_message_bytes.argtypes = [cfgp]
    lib.liec_down_message_bytes.restype = C.c_size_t
    lib.liec_init.argtypes = [cfgp, vp, vp, vp, C.c_size_t, C.POINTER(vp)]
    lib.liec_init.restype = C.c_int
    lib.liec_uplink_compress.argtypes = [vp, vp, vp]
    lib.liec_uplink_compress.restype = C.c_int
    lib.liec_server_aggregate.argtypes = [vp, vp]
    lib.liec_server_aggregate.restype = C.c_int
    lib.liec_downlink_compress.argtypes = [vp, vp]
    lib.liec_downlink_compress.restype = C.c_int
    lib.liec_worker_update.argtypes = [vp, vp, C.c_float, vp]
    lib.liec_worker_update.restype = C.c_int
    lib.liec_set_subsets.argtypes = [vp, vp, vp]
    lib.liec_set_subsets.restype = C.c_int
    lib.liec_draw_subsets.argtypes = [vp, C.c_uint64, C.c_uint32, vp]
    lib.liec_draw_subsets.restype = C.c_int
    lib.liec_wire_bytes_seeded.argtypes = [cfgp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.liec_wire_bytes_seeded.restype = C.c_int
    lib.liec_step.argtypes = [vp, vp, C.c_float, vp]
    lib.liec_step.restype = C.c_int
    lib.liec_topk_route_counts.argtypes = [vp, vp, C.c_int32, C.POINTER(C.c_int64), vp]
    lib.liec_topk_route_counts.restype = C.c_int
    lib.liec_abort_step.argtypes = [vp]
    lib.liec_abort_step.restype = C.c_int
    lib.liec_set_copy_wait.argtypes = [vp, C.c_uint32, C.c_uint32]
    lib.liec_set_copy_wait.restype = C.c_int
    lib.liec_average_step.argtypes = [vp, vp, C.c_float, vp]
    lib.liec_average_step.restype = C.c_int
    lib.liec_mean_params.argtypes = [vp, vp, vp]
    lib.liec_mean_params.restype = C.c_int
    lib.liec_sumsq.argtypes = [vp, C.c_int32, vp, vp, vp]
    lib.liec_sumsq.restype = C.c_int
    lib.liec_set_telemetry.argtypes = [vp, C.c_int32]
    lib.liec_set_telemetry.restype = C.c_int
    lib.liec_get_telemetry.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.liec_get_telemetry.restype = C.c_int
    lib.liec_step_host.argtypes = [vp, vp, vp, C.c_float, vp, vp]
    lib.liec_step_host.restype = C.c_int
    lib.liec_get_messages.argtypes = [vp, C.POINTER(liec_messages)]
    lib.liec_get_messages.restype = C.c_int
    lib.liec_device_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
    lib.liec_device_status.restype = C.c_int
    lib.liec_clear_status.argtypes = [vp, vp]
    lib.liec_clear_status.restype = C.c_int
    lib.liec_launch_count.argtypes = [vp]
    lib.liec_launch_count.restype = C.c_int64
    lib.liec_last_error.argtypes = [vp]
    lib.liec_last_error.restype = C.c_char_p
    lib.liec_destroy.argtypes = [vp]
    lib.liec_destroy.restype = None
    lib.liec_sign_compress_noalloc.argtypes = [vp, C.c_int32, C.c_int64, vp, vp, vp]
    lib.liec_sign_compress_noalloc.restype = C.c_int
    lib.liec_noalloc_last_error.argtypes = []
    lib.liec_noalloc_last_error.restype = C.c_char_p
    if path is None:
        _LIB = lib
    return lib


def make_config(num_workers: int, seg_offsets: Sequence[int], uplink: int, downlink: int,
                topk_k: Optional[Sequence[int]] = None, grad_dtype: int = F32):
    """Returns (liec_config, keepalive) - keepalive owns the host arrays the struct points to."""
    off = np.ascontiguousarray(seg_offsets, dtype=np.int64)
    k = None if topk_k is None else np.ascontiguousarray(topk_k, dtype=np.int64)
    cfg = liec_config()
    cfg.num_workers = int(num_workers)
    cfg.dim = int(off[-1]) if off.size else 0
    cfg.num_segments = int(off.size - 1)
    cfg.seg_offsets = off.ctypes.data_as(C.POINTER(C.c_int64))
    cfg.uplink, cfg.downlink = int(uplink), int(downlink)
    cfg.topk_k = k.ctypes.data_as(C.POINTER(C.c_int64)) if k is not None else None
    cfg.grad_dtype = int(grad_dtype)
    return cfg, (off, k)


def workspace_bytes(cfg: liec_config) -> int:
    return int(load_library().liec_workspace_bytes(C.byref(cfg)))


def liec_wire_bytes_seeded(cfg: liec_config):
    """As liec_wire_bytes when sender and receiver draw the random-k subsets from a shared seed."""
    return liec_wire_bytes(cfg, _seeded=True)


def liec_wire_bytes(cfg: liec_config, _seeded: bool = False):
    """(uplink, downlink, full-precision) bytes per worker and iteration."""
    lib = load_library()
    up, down, full = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    fn = lib.liec_wire_bytes_seeded if _seeded else lib.liec_wire_bytes
    st = fn(C.byref(cfg), C.byref(up), C.byref(down), C.byref(full))
    if st != 0:
        raise LiecError(st, lib.liec_last_error(None).decode())
    return int(up.value), int(down.value), int(full.value)


def down_message_bytes(cfg: liec_config) -> int:
    return int(load_library().liec_down_message_bytes(C.byref(cfg)))


NOALLOC_MAX_ELEMENTS = 64 * 1024 * 1024


def liec_sign_compress_noalloc(x, words, scale, stream=None):
    """Scaled sign of one CUDA vector into caller-provided `words` (int32, ceil(n/32)) and `scale`
    (float32, 1 element) without any workspace or allocation; see liec.h for who needs this."""
    import torch
    lib = load_library()
    n = x.numel()
    if not (x.is_cuda and x.is_contiguous() and x.dtype in (torch.float32, torch.bfloat16)):
        raise ValueError("x must be a contiguous CUDA tensor of float32 or bfloat16")
    if not (words.is_cuda and words.is_contiguous() and words.dtype in (torch.int32, torch.uint32)
            and words.numel() == (n + 31) // 32 and words.device == x.device):
        raise ValueError("words must be a contiguous CUDA tensor of ceil(n/32) 32-bit integers on x's device")
    if not (scale.is_cuda and scale.dtype == torch.float32 and scale.numel() == 1 and scale.device == x.device):
        raise ValueError("scale must be a one-element float32 CUDA tensor on x's device")
    dtype = BF16 if x.dtype == torch.bfloat16 else F32
    s = (stream if stream is not None else torch.cuda.current_stream(x.device)).cuda_stream
    with torch.cuda.device(x.device):
        st = lib.liec_sign_compress_noalloc(x.data_ptr(), dtype, x.numel(), words.data_ptr(), scale.data_ptr(), s)
    if st != 0:
        raise LiecError(st, lib.liec_noalloc_last_error().decode())


class Context:
    """Owns a ``liec_ctx`` plus the torch tensors it points into (params, error, workspace)."""

    def __init__(self, params, error, seg_offsets, uplink, downlink, topk_k=None, grad_dtype=F32):
        import torch
        self._torch = torch
        self.lib = load_library()
        if not (params.is_cuda and error.is_cuda):
            raise ValueError("params and error must be CUDA tensors (there is no CPU path)")
        assert params.dtype == torch.float32 and error.dtype == torch.float32
        assert params.is_contiguous() and error.is_contiguous() and params.dim() == 2
        self.params, self.error = params, error
        self.N, self.d = params.shape
        self.cfg, self._keep = make_config(self.N, seg_offsets, uplink, downlink, topk_k, grad_dtype)
        if self.cfg.dim != self.d or error.numel() != self.d:
            raise ValueError("seg_offsets[-1], params.shape[1] and error.numel() must agree")
        nbytes = workspace_bytes(self.cfg)
        if nbytes == 0:
            # let liec_init produce the precise message
            nbytes = 256
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=params.device)
        self._ctx = C.c_void_p()
        with torch.cuda.device(params.device):
            st = self.lib.liec_init(C.byref(self.cfg), params.data_ptr(), error.data_ptr(),
                                    self.workspace.data_ptr(), nbytes, C.byref(self._ctx))
        if st != 0:
            raise LiecError(st, self.lib.liec_last_error(None).decode())
        self.grad_dtype = grad_dtype
        self.T = self.cfg.num_segments

    # -- helpers ---------------------------------------------------------------------------
    def _stream(self, stream=None) -> int:
        s = stream if stream is not None else self._torch.cuda.current_stream(self.params.device)
        return s.cuda_stream

    def _check(self, st: int):
        if st != 0:
            raise LiecError(st, self.lib.liec_last_error(self._ctx).decode())

    def _check_grads(self, grads):
        t = self._torch
        want = t.bfloat16 if self.grad_dtype == BF16 else t.float32
        if not grads.is_cuda or grads.dtype != want or grads.shape != (self.N, self.d) or not grads.is_contiguous():
            raise ValueError("grads must be a contiguous CUDA tensor [N, d] of the configured dtype")

    # -- the C ABI, one method per entry point -----------------------------------------------
    def liec_uplink_compress(self, grads, stream=None):
        self._check_grads(grads)
        self._check(self.lib.liec_uplink_compress(self._ctx, grads.data_ptr(), self._stream(stream)))

    def liec_server_aggregate(self, stream=None):
        self._check(self.lib.liec_server_aggregate(self._ctx, self._stream(stream)))

    def liec_downlink_compress(self, stream=None):
        self._check(self.lib.liec_downlink_compress(self._ctx, self._stream(stream)))

    def liec_worker_update(self, grads, lr: float, stream=None):
        self._check_grads(grads)
        self._check(self.lib.liec_worker_update(self._ctx, grads.data_ptr(), float(lr), self._stream(stream)))

    def liec_set_subsets(self, up_sets=None, down_set=None):
        """Random-k: int32/uint32 CUDA tensors [N, K] / [K] of kept flat indices (ascending inside each
        segment).  The tensors are referenced, not copied; this object keeps them alive."""
        t = self._torch
        for name, s, shape in (("up_sets", up_sets, (self.N, -1)), ("down_set", down_set, (-1,))):
            if s is None:
                continue
            if not s.is_cuda or s.dtype not in (t.int32, t.uint32) or not s.is_contiguous() or s.dim() != len(shape):
                raise ValueError(f"{name} must be a contiguous CUDA tensor of 32-bit indices")
        self._subsets = (up_sets, down_set)
        self._check(self.lib.liec_set_subsets(self._ctx, None if up_sets is None else up_sets.data_ptr(),
                                              None if down_set is None else down_set.data_ptr()))

    def liec_draw_subsets(self, seed: int, epoch: int, stream=None):
        """Random-k: draws and installs the subsets of all workers and the server from (seed, epoch)."""
        self._subsets = None
        self._check(self.lib.liec_draw_subsets(self._ctx, int(seed), int(epoch), self._stream(stream)))

    def liec_step(self, grads, lr: float, stream=None):
        self._check_grads(grads)
        self._check(self.lib.liec_step(self._ctx, grads.data_ptr(), float(lr), self._stream(stream)))

    def liec_topk_route_counts(self, uplink: bool, stream=None, per_problem: bool = False) -> dict:
        """Counts of the routes taken by the last iteration's selections; with per_problem also a uint8
        array [rows, T] of flags (1 single pass, 2 second-digit pass, 4 dense one-CTA path, 8 single tile)."""
        out = (C.c_int64 * 5)()
        flags = np.zeros(((self.N if uplink else 1), self.T), np.uint8) if per_problem else None
        self._check(self.lib.liec_topk_route_counts(self._ctx, self._stream(stream), 1 if uplink else 0, out,
                                                    None if flags is None else flags.ctypes.data_as(C.c_void_p)))
        r = {"problems": int(out[0]), "single_pass": int(out[1]), "refined": int(out[2]), "slow": int(out[3]),
             "direct": int(out[4])}
        if flags is not None:
            r["flags"] = flags
        return r

    def liec_abort_step(self):
        self._check(self.lib.liec_abort_step(self._ctx))

    def liec_set_copy_wait(self, poll_limit: int = 0, expect_extra_bytes: int = 0):
        self._check(self.lib.liec_set_copy_wait(self._ctx, int(poll_limit), int(expect_extra_bytes)))

    def liec_average_step(self, grads, lr: float, stream=None):
        self._check_grads(grads)
        self._check(self.lib.liec_average_step(self._ctx, grads.data_ptr(), float(lr), self._stream(stream)))

    def liec_mean_params(self, out, stream=None):
        assert out.is_cuda and out.dtype == self._torch.float32 and out.numel() == self.d and out.is_contiguous()
        self._check(self.lib.liec_mean_params(self._ctx, out.data_ptr(), self._stream(stream)))

    def liec_sumsq(self, which: int, out, grads=None, stream=None):
        """Per-segment squared norms (SUMSQ_ERROR / SUMSQ_GRADS / SUMSQ_PARAMS) into `out` [rows, T] float64."""
        rows = 1 if which == SUMSQ_ERROR else self.N
        assert out.is_cuda and out.dtype == self._torch.float64 and out.numel() == rows * self.T and out.is_contiguous()
        gptr = None
        if which == SUMSQ_GRADS:
            self._check_grads(grads)
            gptr = grads.data_ptr()
        self._check(self.lib.liec_sumsq(self._ctx, int(which), gptr, out.data_ptr(), self._stream(stream)))

    def liec_set_telemetry(self, on: bool):
        self._check(self.lib.liec_set_telemetry(self._ctx, 1 if on else 0))

    def liec_get_telemetry(self, stream=None, kept: bool = True) -> dict:
        """Per-segment squared norms of the last iteration (float64 CUDA tensors, allocated here):
        e_sumsq [T], v_sumsq [T], g_sumsq [N, T] and, for sides with (index, value) messages and
        kept=True, up_kept_sumsq [N, T] / down_kept_sumsq [T]."""
        t = self._torch
        dev, f64 = self.params.device, t.float64
        sparse = (COMP_TOPK, COMP_RANDK)
        out = {"e_sumsq": t.empty(self.T, dtype=f64, device=dev), "v_sumsq": t.empty(self.T, dtype=f64, device=dev),
               "g_sumsq": t.empty(self.N, self.T, dtype=f64, device=dev),
               "up_kept_sumsq": t.empty(self.N, self.T, dtype=f64, device=dev) if kept and self.cfg.uplink in sparse else None,
               "down_kept_sumsq": t.empty(self.T, dtype=f64, device=dev) if kept and self.cfg.downlink in sparse else None}
        ptr = lambda name: None if out[name] is None else out[name].data_ptr()
        self._check(self.lib.liec_get_telemetry(self._ctx, ptr("e_sumsq"), ptr("v_sumsq"), ptr("g_sumsq"),
                                                ptr("up_kept_sumsq"), ptr("down_kept_sumsq"), self._stream(stream)))
        return out

    def liec_step_host(self, grads_host, grads_dev, lr: float, down_msg_host=None, stream=None):
        self._check_grads(grads_dev)
        assert not grads_host.is_cuda and grads_host.shape == grads_dev.shape and grads_host.dtype == grads_dev.dtype
        out_ptr = down_msg_host.data_ptr() if down_msg_host is not None else None
        self._check(self.lib.liec_step_host(self._ctx, grads_host.data_ptr(), grads_dev.data_ptr(), float(lr),
                                            out_ptr, self._stream(stream)))

    def liec_device_status(self, stream=None) -> int:
        out = C.c_int32(0)
        st = self.lib.liec_device_status(self._ctx, self._stream(stream), C.byref(out))
        if st not in (0, 6):
            self._check(st)
        return int(out.value)

    def liec_clear_status(self, stream=None):
        self._check(self.lib.liec_clear_status(self._ctx, self._stream(stream)))

    def liec_launch_count(self) -> int:
        return int(self.lib.liec_launch_count(self._ctx))

    def liec_get_messages(self) -> dict:
        """Device views (torch tensors aliasing the workspace) of the current messages."""
        t = self._torch
        m = liec_messages()
        self._check(self.lib.liec_get_messages(self._ctx, C.byref(m)))
        base = self.workspace.data_ptr()
        W, K, N, T = int(m.num_words), int(m.num_topk), self.N, self.T

        def view(ptr, count, dtype):
            if not ptr or count == 0:
                return None
            esz = 4
            off = ptr - base
            return self.workspace[off:off + count * esz].view(dtype)

        return {
            "up_words": _reshape(view(m.up_words, N * W, t.int32), (N, W)),
            "up_scales": _reshape(view(m.up_scales, N * T, t.float32), (N, T)),
            "up_idx": _reshape(view(m.up_idx, N * K, t.int32), (N, K)),
            "up_val": _reshape(view(m.up_val, N * K, t.float32), (N, K)),
            "down_words": view(m.down_words, W, t.int32),
            "down_scales": view(m.down_scales, T, t.float32),
            "down_idx": view(m.down_idx, K, t.int32),
            "down_val": view(m.down_val, K, t.float32),
            "v": self.error,
            "num_words": W, "num_topk": K,
        }

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self.lib.liec_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _reshape(t, shape):
    return None if t is None else t.view(*shape)
