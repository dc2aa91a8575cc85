"""ctypes binding of libh2o_b200.so: the same calls as include/h2o.h, argument marshalling only.

Every step of the path runs in the CUDA kernels behind the C ABI.  PyTorch is
used here for device memory and streams, nothing else.  There is no fallback:
if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# H2O_B200_LIB names another build of the same library (the checked variant libh2o_b200_bounds.so of build.py)
LIB_PATH = os.environ.get("H2O_B200_LIB") or os.path.join(_PKG, "libh2o_b200.so")

H2O_OK = 0
H2O_ERR_INVALID_ARG = -1
H2O_ERR_UNSUPPORTED = -2
H2O_ERR_WORKSPACE = -3
H2O_ERR_STATE = -4
H2O_ERR_CUDA = -5
H2O_ERR_TIMEOUT = -6
H2O_F32 = 0
H2O_BF16 = 1
H2O_BF16_KV4 = 2  # bf16 inputs, 4-bit group-quantised K/V slots

EXPORTED = (
    "h2o_cache_workspace_bytes",
    "h2o_prefill_scratch_bytes",
    "h2o_cache_create",
    "h2o_prefill_select",
    "h2o_prefill_select_static",
    "h2o_prefill_static_scratch_bytes",
    "h2o_decode_step",
    "h2o_cache_destroy",
    "h2o_cache_reset",
    "h2o_host_staging_bytes",
    "h2o_prefill_select_host",
    "h2o_decode_step_host",
    "h2o_cache_export",
    "h2o_cache_status",
    "h2o_cache_set_decode_shape",
    "h2o_cache_set_prefill_path",
    "h2o_cache_set_decode_path",
    "h2o_cache_get_decode_path",
    "h2o_debug_set_early_prefetch",
    "h2o_prefill_scratch_layout",
    "h2o_strerror",
)


class h2o_config_t(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32),
        ("n_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("heavy_budget", ctypes.POINTER(ctypes.c_int32)),
        ("recent_window", ctypes.POINTER(ctypes.c_int32)),
        ("softmax_scale", ctypes.c_float),
        ("device", ctypes.c_int32),
        ("query_group", ctypes.c_int32),
    ]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libh2o_b200.so is not built (run `python paper_2306_14048_b200/build.py`); there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    c = ctypes
    vp, i32p = c.c_void_p, c.POINTER(c.c_int32)
    cfgp = c.POINTER(h2o_config_t)
    lib.h2o_cache_workspace_bytes.restype = c.c_size_t
    lib.h2o_cache_workspace_bytes.argtypes = [cfgp]
    lib.h2o_prefill_scratch_bytes.restype = c.c_size_t
    lib.h2o_prefill_scratch_bytes.argtypes = [cfgp, c.c_int64]
    lib.h2o_cache_create.restype = c.c_int
    lib.h2o_cache_create.argtypes = [c.POINTER(vp), cfgp, vp, c.c_size_t]
    lib.h2o_prefill_select.restype = c.c_int
    lib.h2o_debug_wait_probe.argtypes = [vp, c.c_int32, vp]
    lib.h2o_debug_wait_probe.restype = c.c_int
    lib.h2o_cache_attach.argtypes = [c.POINTER(vp), cfgp, vp, c.c_size_t]
    lib.h2o_cache_attach.restype = c.c_int
    lib.h2o_prefill_select.argtypes = [vp, vp, vp, vp, i32p, vp, vp, c.c_size_t, vp]
    lib.h2o_prefill_select_static.restype = c.c_int
    lib.h2o_prefill_select_static.argtypes = [vp, vp, vp, vp, i32p, vp, vp]
    lib.h2o_prefill_static_scratch_bytes.restype = c.c_size_t
    lib.h2o_prefill_static_scratch_bytes.argtypes = []
    lib.h2o_decode_step.restype = c.c_int
    lib.h2o_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.h2o_cache_reset.restype = c.c_int
    lib.h2o_decode_chunk.argtypes = [vp, vp, vp, vp, c.c_int32, vp, vp, vp]
    lib.h2o_decode_chunk.restype = c.c_int
    lib.h2o_cache_set_chunk_path.argtypes = [vp, c.c_int32]
    lib.h2o_cache_set_chunk_path.restype = c.c_int
    lib.h2o_cache_set_score_mode.argtypes = [vp, c.c_int32]
    lib.h2o_cache_set_score_mode.restype = c.c_int
    lib.h2o_cache_set_topk.argtypes = [vp, c.c_int32]
    lib.h2o_cache_set_topk.restype = c.c_int
    lib.h2o_cache_set_mask.argtypes = [vp, c.c_int32, c.c_int32, c.c_int32]
    lib.h2o_cache_set_mask.restype = c.c_int
    lib.h2o_cache_fscore.argtypes = [vp, c.c_int32, vp, vp]
    lib.h2o_cache_fscore.restype = c.c_int
    lib.h2o_cache_reset.argtypes = [vp, vp]
    lib.h2o_host_staging_bytes.restype = c.c_size_t
    lib.h2o_host_staging_bytes.argtypes = [cfgp, c.c_int64]
    lib.h2o_prefill_select_host.restype = c.c_int
    lib.h2o_prefill_select_host.argtypes = [vp, vp, vp, vp, i32p, vp, vp, c.c_size_t, vp, c.c_size_t, vp]
    lib.h2o_decode_step_host.restype = c.c_int
    lib.h2o_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, c.c_size_t, vp]
    lib.h2o_cache_destroy.restype = c.c_int
    lib.h2o_cache_destroy.argtypes = [vp]
    lib.h2o_cache_export.restype = c.c_int
    lib.h2o_cache_export.argtypes = [vp, i32p, c.POINTER(c.c_double), i32p, i32p, c.c_int32, vp]
    lib.h2o_cache_status.restype = c.c_int
    lib.h2o_cache_status.argtypes = [vp, vp]
    lib.h2o_cache_set_decode_shape.restype = c.c_int
    lib.h2o_cache_set_decode_shape.argtypes = [vp, c.c_int32, c.c_int32]
    lib.h2o_cache_set_prefill_path.restype = c.c_int
    lib.h2o_cache_set_decode_path.restype = c.c_int
    lib.h2o_cache_get_decode_path.restype = c.c_int
    lib.h2o_cache_get_decode_path.argtypes = [vp]
    lib.h2o_cache_set_decode_path.argtypes = [vp, c.c_int32]
    lib.h2o_cache_set_prefill_path.argtypes = [vp, c.c_int32]
    lib.h2o_prefill_scratch_layout.restype = c.c_int
    lib.h2o_prefill_scratch_layout.argtypes = [cfgp, c.c_int64, c.POINTER(c.c_size_t)]
    lib.h2o_debug_set_early_prefetch.restype = c.c_int
    lib.h2o_debug_set_early_prefetch.argtypes = [c.c_int32]
    lib.h2o_debug_set_prefill_events.restype = c.c_int
    lib.h2o_debug_set_prefill_events.argtypes = [vp, c.POINTER(vp)]
    lib.h2o_debug_bounds_checked.restype = c.c_int
    lib.h2o_debug_bounds_checked.argtypes = []
    lib.h2o_strerror.restype = c.c_char_p
    lib.h2o_strerror.argtypes = [c.c_int]
    return lib


lib = _load()


class H2OError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, lib.h2o_strerror(code).decode(), code))


def _check(code: int, where: str):
    if code != H2O_OK:
        raise H2OError(code, where)


def make_config(batch, n_heads, head_dim, dtype, heavy: Sequence[int], recent: Sequence[int], softmax_scale=0.0, device=0,
                query_group=1):
    """Returns (h2o_config_t, keepalive) — the budget arrays must outlive the struct."""
    hv = (ctypes.c_int32 * len(heavy))(*[int(x) for x in heavy])
    rc = (ctypes.c_int32 * len(recent))(*[int(x) for x in recent])
    code = {torch.float32: H2O_F32, torch.bfloat16: H2O_BF16, "f32": H2O_F32, "bf16": H2O_BF16,
            "bf16_kv4": H2O_BF16_KV4}.get(dtype, dtype)
    cfg = h2o_config_t(int(batch), int(n_heads), int(head_dim), int(code), hv, rc, float(softmax_scale), int(device),
                       int(query_group))
    return cfg, (hv, rc)


def h2o_cache_workspace_bytes(cfg: h2o_config_t) -> int:
    return int(lib.h2o_cache_workspace_bytes(ctypes.byref(cfg)))


def h2o_prefill_scratch_bytes(cfg: h2o_config_t, total_tokens: int) -> int:
    return int(lib.h2o_prefill_scratch_bytes(ctypes.byref(cfg), int(total_tokens)))


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


class H2OCache:
    """A cache handle plus the torch tensors that back its workspace.

    Methods mirror the C calls one to one: ``prefill_select`` -> h2o_prefill_select,
    ``decode_step`` -> h2o_decode_step, ``export`` -> h2o_cache_export,
    ``status`` -> h2o_cache_status, ``close`` -> h2o_cache_destroy.
    """

    def __init__(self, batch, n_heads, head_dim, dtype, heavy, recent, softmax_scale=0.0, device=0, snapshot=None,
                 query_group=1):
        """``snapshot``: bytes of another handle's workspace (``snapshot()``) to resume from (h2o_cache_attach).
        ``query_group`` > 1: grouped-query attention, q / out carry n_heads * query_group heads."""
        self.cfg, self._keep = make_config(batch, n_heads, head_dim, dtype, heavy, recent, softmax_scale, device,
                                           query_group)
        self.batch, self.n_heads, self.head_dim = int(batch), int(n_heads), int(head_dim)
        self.units = self.batch * self.n_heads
        self.max_B = int(max(int(a) + int(b) for a, b in zip(heavy, recent)))
        self.device = torch.device("cuda", int(device))
        nbytes = h2o_cache_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise H2OError(H2O_ERR_INVALID_ARG, "h2o_cache_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        self._ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        self.workspace_bytes = nbytes
        handle = ctypes.c_void_p()
        if snapshot is None:
            _check(lib.h2o_cache_create(ctypes.byref(handle), ctypes.byref(self.cfg), self._ws_ptr, nbytes), "h2o_cache_create")
        else:
            off = self._ws_ptr - self.workspace.data_ptr()
            self.workspace[off:off + nbytes].copy_(snapshot.to(self.device))
            torch.cuda.synchronize(self.device)
            _check(lib.h2o_cache_attach(ctypes.byref(handle), ctypes.byref(self.cfg), self._ws_ptr, nbytes), "h2o_cache_attach")
        self._h = handle
        self._scratch = None

    def snapshot(self):
        """The workspace bytes (a copy): the complete state of the cache.  Synchronises the device first."""
        torch.cuda.synchronize(self.device)
        off = self._ws_ptr - self.workspace.data_ptr()
        return self.workspace[off:off + self.workspace_bytes].clone()

    def prefill_select(self, q, k, v, cu_seqlens, out, stream=None):
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        need = h2o_prefill_scratch_bytes(self.cfg, int(cu[-1]))
        if self._scratch is None or self._scratch.numel() < need + 256:
            self._scratch = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        sp = (self._scratch.data_ptr() + 255) // 256 * 256
        _check(lib.h2o_prefill_select(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                      cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), out.data_ptr(), sp, need,
                                      _stream_ptr(stream)), "h2o_prefill_select")

    def prefill_select_static(self, q, k, v, cu_seqlens, out, stream=None):
        """h2o_prefill_select_static: the scratch is the library's built-in array, nothing is allocated here."""
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        _check(lib.h2o_prefill_select_static(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                             cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), out.data_ptr(),
                                             _stream_ptr(stream)), "h2o_prefill_select_static")

    def decode_step(self, q, k_new, v_new, out, evicted_pos=None, stream=None):
        _check(lib.h2o_decode_step(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
                                   None if evicted_pos is None else evicted_pos.data_ptr(), _stream_ptr(stream)),
               "h2o_decode_step")

    def decode_chunk(self, q, k, v, out, evicted_pos=None, stream=None):
        """h2o_decode_chunk: q, k, v, out are [n_tokens, batch, n_heads, head_dim]; evicted_pos [n_tokens, batch, n_heads]."""
        _check(lib.h2o_decode_chunk(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), int(q.shape[0]), out.data_ptr(),
                                    None if evicted_pos is None else evicted_pos.data_ptr(), _stream_ptr(stream)),
               "h2o_decode_chunk")

    def set_chunk_path(self, path: int):
        _check(lib.h2o_cache_set_chunk_path(self._h, int(path)), "h2o_cache_set_chunk_path")

    def set_score_mode(self, mode: int):
        """0: rank by the accumulated score, 1: by the averaged score (empty cache only)."""
        _check(lib.h2o_cache_set_score_mode(self._h, int(mode)), "h2o_cache_set_score_mode")

    def set_mask(self, kind: int, a: int = 1, b: int = 0):
        """h2o_cache_set_mask: 0 none, 1 strided(stride a, local window b), 2 fixed(block a, b summary columns)."""
        _check(lib.h2o_cache_set_mask(self._h, int(kind), int(a), int(b)), "h2o_cache_set_mask")

    def set_topk(self, m: int):
        """h2o_cache_set_topk: in decode steps a query attends only its m largest logits (0 = off)."""
        _check(lib.h2o_cache_set_topk(self._h, int(m)), "h2o_cache_set_topk")

    def fscore(self, hkind: int = 0, stream=None):
        """F_score per (sequence, head): sum of h(accumulated score); h: 0 identity, 1 sqrt(z+1), 2 log(z+1)."""
        out = torch.empty(self.cfg.batch * self.cfg.n_heads, dtype=torch.float64, device=self.device)
        _check(lib.h2o_cache_fscore(self._h, int(hkind), out.data_ptr(), _stream_ptr(stream)), "h2o_cache_fscore")
        return out.view(self.cfg.batch, self.cfg.n_heads)

    def reset(self, stream=None):
        _check(lib.h2o_cache_reset(self._h, _stream_ptr(stream)), "h2o_cache_reset")

    def _staging(self, tokens: int):
        need = int(lib.h2o_host_staging_bytes(ctypes.byref(self.cfg), int(tokens)))
        st = getattr(self, "_stage", None)
        if st is None or st.numel() < need + 256:
            self._stage = st = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        return (st.data_ptr() + 255) // 256 * 256, need

    def prefill_select_host(self, q, k, v, cu_seqlens, out, stream=None):
        """Host (ideally pinned) tensors in and out; the copies run on the stream inside the C call."""
        cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
        need = h2o_prefill_scratch_bytes(self.cfg, int(cu[-1]))
        if self._scratch is None or self._scratch.numel() < need + 256:
            self._scratch = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
        sp = (self._scratch.data_ptr() + 255) // 256 * 256
        sg, sg_bytes = self._staging(int(cu[-1]))
        _check(lib.h2o_prefill_select_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                           cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), out.data_ptr(), sg, sg_bytes,
                                           sp, need, _stream_ptr(stream)), "h2o_prefill_select_host")

    def decode_step_host(self, q, k_new, v_new, out, evicted_pos=None, stream=None):
        if getattr(self, "_dstage", None) is None:
            need = int(lib.h2o_host_staging_bytes(ctypes.byref(self.cfg), self.batch))
            buf = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
            self._dstage = (buf, (buf.data_ptr() + 255) // 256 * 256, need)
        _, sg, sg_bytes = self._dstage
        _check(lib.h2o_decode_step_host(self._h, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), out.data_ptr(),
                                        None if evicted_pos is None else evicted_pos.data_ptr(), sg, sg_bytes,
                                        _stream_ptr(stream)), "h2o_decode_step_host")

    def export(self, stream=None):
        """(pos [units, max_B] int32 with -1 padding, acc [units, max_B] float64, count [units], t [units])."""
        pitch = self.max_B
        pos = np.empty((self.units, pitch), dtype=np.int32)
        acc = np.empty((self.units, pitch), dtype=np.float64)
        count = np.empty(self.units, dtype=np.int32)
        t = np.empty(self.units, dtype=np.int32)
        i32p = ctypes.POINTER(ctypes.c_int32)
        _check(lib.h2o_cache_export(self._h, pos.ctypes.data_as(i32p), acc.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                                    count.ctypes.data_as(i32p), t.ctypes.data_as(i32p), pitch, _stream_ptr(stream)),
               "h2o_cache_export")
        return pos, acc, count, t

    def set_decode_shape(self, split: int = 0, stages: int = 0):
        _check(lib.h2o_cache_set_decode_shape(self._h, int(split), int(stages)), "h2o_cache_set_decode_shape")

    def set_prefill_events(self, events):
        """h2o_debug_set_prefill_events: four torch.cuda.Event(enable_timing=True), already recorded once (torch
        creates the CUDA handle lazily), for the next prefill_select call."""
        arr = (ctypes.c_void_p * 4)(*[int(e.cuda_event) for e in events])
        _check(lib.h2o_debug_set_prefill_events(self._h, arr), "h2o_debug_set_prefill_events")

    def set_decode_path(self, path: int):
        _check(lib.h2o_cache_set_decode_path(self._h, int(path)), "h2o_cache_set_decode_path")

    def decode_path(self) -> int:
        return int(lib.h2o_cache_get_decode_path(self._h))

    def set_prefill_path(self, path: int):
        _check(lib.h2o_cache_set_prefill_path(self._h, int(path)), "h2o_cache_set_prefill_path")

    def prefill_column_sums(self, total_tokens: int):
        """acc0 of the last prefill_select as a [n_heads, total_tokens] float64 tensor (a view of the scratch)."""
        acc_off = ctypes.c_size_t()
        _check(lib.h2o_prefill_scratch_layout(ctypes.byref(self.cfg), int(total_tokens), ctypes.byref(acc_off)),
               "h2o_prefill_scratch_layout")
        base = (self._scratch.data_ptr() + 255) // 256 * 256 - self._scratch.data_ptr()
        n = self.n_heads * int(total_tokens)
        raw = self._scratch[base + acc_off.value: base + acc_off.value + 8 * n]
        return raw.view(torch.float64).view(self.n_heads, int(total_tokens))

    def status(self, stream=None) -> int:
        return int(lib.h2o_cache_status(self._h, _stream_ptr(stream)))

    def close(self):
        if getattr(self, "_h", None) is not None:
            lib.h2o_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
