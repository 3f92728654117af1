"""Thin ctypes binding of ``libadaspark_attn.so``: the same entry points as
``include/adaspark_attn.h``, argument marshalling only.  Every step of AdaS-Attn runs inside the
library's CUDA kernels; torch is used here for device memory and streams only.

There is no CPU fallback: if the shared library is missing, ``load()`` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libadaspark_attn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NOT_PARTITIONED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, \
    ERR_TIMEOUT = range(7)
STATUS_NAMES = ["OK", "ERR_INVALID_ARG", "ERR_UNSUPPORTED", "ERR_NOT_PARTITIONED",
                "ERR_WORKSPACE_TOO_SMALL", "ERR_CUDA", "ERR_TIMEOUT"]


class Config(ctypes.Structure):
    _fields_ = [("cube_t", ctypes.c_int32), ("cube_h", ctypes.c_int32), ("cube_w", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("top_p", ctypes.c_float),
                ("softmax_scale", ctypes.c_float), ("device", ctypes.c_int32), ("top_k", ctypes.c_int32)]


class Layout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "n_cubes", "cube_tokens", "s_video", "s_cap", "bitmap_words", "k_cube_bytes",
        "v_cube_bytes", "cube_keys_bytes", "forward_workspace_bytes", "decode_workspace_bytes")]


class AdasparkError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < 7 else status}: {message}")
        self.status = status


_lib: Optional[ctypes.CDLL] = None

EXPORTS = ["adaspark_attn_create", "adaspark_attn_partition", "adaspark_attn_get_layout",
           "adaspark_attn_forward", "adaspark_attn_forward_host", "adaspark_attn_forward_prefix", "adaspark_attn_forward_chunk", "adaspark_attn_decode", "adaspark_attn_destroy",
           "adaspark_attn_last_error", "adaspark_attn_last_launch_count",
           "adaspark_attn_set_prefill_kernel", "adaspark_attn_set_gather", "adaspark_attn_enable_stage_timing",
           "adaspark_attn_get_stage_times", "adaspark_attn_get_attention_kernel_ms", "adaspark_attn_decode_static",
           "adaspark_attn_debug_umma_selftest", "adaspark_attn_debug_imma_selftest",
           "adaspark_attn_debug_fastdiv", "adaspark_attn_debug_wait_timeout"]


def load() -> ctypes.CDLL:
    """dlopen the in-tree library; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_08077_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.adaspark_attn_create.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(vp)]
    lib.adaspark_attn_partition.argtypes = [vp, i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
    lib.adaspark_attn_get_layout.argtypes = [vp, ctypes.POINTER(Layout)]
    lib.adaspark_attn_forward.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.adaspark_attn_forward_host.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.adaspark_attn_forward_prefix.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.adaspark_attn_forward_chunk.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.adaspark_attn_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.adaspark_attn_decode_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.adaspark_attn_debug_umma_selftest.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.adaspark_attn_debug_imma_selftest.argtypes = [vp, vp, vp, vp, vp]
    lib.adaspark_attn_debug_wait_timeout.argtypes = [ctypes.c_uint64, vp, vp, vp]
    lib.adaspark_attn_debug_fastdiv.argtypes = [ctypes.c_int32, ctypes.c_int32]
    lib.adaspark_attn_debug_fastdiv.restype = ctypes.c_int32
    lib.adaspark_attn_destroy.argtypes = [vp]
    lib.adaspark_attn_last_error.argtypes = [vp]
    lib.adaspark_attn_last_error.restype = ctypes.c_char_p
    lib.adaspark_attn_last_launch_count.argtypes = [vp]
    lib.adaspark_attn_last_launch_count.restype = ctypes.c_int64
    lib.adaspark_attn_set_prefill_kernel.argtypes = [vp, i32]
    lib.adaspark_attn_set_gather.argtypes = [vp, ctypes.c_float, ctypes.c_uint64]
    lib.adaspark_attn_enable_stage_timing.argtypes = [vp, i32]
    lib.adaspark_attn_get_stage_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.adaspark_attn_get_attention_kernel_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    for name in EXPORTS:
        if name not in ("adaspark_attn_last_error", "adaspark_attn_last_launch_count"):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors crossing the C ABI must be contiguous"
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        if not torch.cuda.is_available():   # host-side argument checks still run without a GPU
            return None
        return torch.cuda.current_stream().cuda_stream or None
    return stream.cuda_stream or None


# ---- the C entry points, one Python function each (raw: pointers are ints or tensors) ----------

def adaspark_attn_create(config: Config) -> int:
    h = ctypes.c_void_p()
    st = load().adaspark_attn_create(ctypes.byref(config), ctypes.byref(h))
    if st != OK:
        raise AdasparkError(st, "adaspark_attn_create rejected the configuration")
    return h.value


def _check(handle: int, st: int):
    if st != OK:
        raise AdasparkError(st, load().adaspark_attn_last_error(handle).decode())


def adaspark_attn_partition(handle: int, batch: int, frames: int, grid_h: int, grid_w: int,
                            n_text_max: int) -> int:
    ws = ctypes.c_size_t(0)
    _check(handle, load().adaspark_attn_partition(handle, batch, frames, grid_h, grid_w, n_text_max,
                                                  ctypes.byref(ws)))
    return ws.value


def adaspark_attn_get_layout(handle: int) -> Layout:
    lay = Layout()
    _check(handle, load().adaspark_attn_get_layout(handle, ctypes.byref(lay)))
    return lay


def adaspark_attn_forward(handle: int, q, k, v, n_text: int, out, k_cube, v_cube, cube_keys,
                          sel_bitmap, sel_count, workspace, workspace_bytes: int, stream=None):
    _check(handle, load().adaspark_attn_forward(
        handle, _ptr(q), _ptr(k), _ptr(v), n_text, _ptr(out), _ptr(k_cube), _ptr(v_cube),
        _ptr(cube_keys), _ptr(sel_bitmap), _ptr(sel_count), _ptr(workspace), workspace_bytes,
        _stream_ptr(stream)))


def adaspark_attn_forward_host(handle: int, q_host, k_host, v_host, n_text: int, out_host, q_dev, k_dev, v_dev,
                               out_dev, k_cube, v_cube, cube_keys, workspace, workspace_bytes: int, stream=None):
    """Prefill from and to host (pinned) tensors: the library issues the copies on the stream."""
    _check(handle, load().adaspark_attn_forward_host(
        handle, _ptr(q_host), _ptr(k_host), _ptr(v_host), n_text, _ptr(out_host), _ptr(q_dev), _ptr(k_dev),
        _ptr(v_dev), _ptr(out_dev), _ptr(k_cube), _ptr(v_cube), _ptr(cube_keys), _ptr(workspace),
        workspace_bytes, _stream_ptr(stream)))


def adaspark_attn_forward_prefix(handle: int, q, k, v, n_prefix: int, n_text: int, out, k_cube, v_cube, cube_keys,
                                 sel_bitmap, sel_count, workspace, workspace_bytes: int, stream=None):
    _check(handle, load().adaspark_attn_forward_prefix(
        handle, _ptr(q), _ptr(k), _ptr(v), n_prefix, n_text, _ptr(out), _ptr(k_cube), _ptr(v_cube),
        _ptr(cube_keys), _ptr(sel_bitmap), _ptr(sel_count), _ptr(workspace), workspace_bytes,
        _stream_ptr(stream)))


def adaspark_attn_forward_chunk(handle: int, q, k, v, frame_begin: int, frame_count: int, n_text: int, out,
                                k_cube, v_cube, cube_keys, sel_bitmap, sel_count, workspace,
                                workspace_bytes: int, stream=None):
    _check(handle, load().adaspark_attn_forward_chunk(
        handle, _ptr(q), _ptr(k), _ptr(v), frame_begin, frame_count, n_text, _ptr(out), _ptr(k_cube),
        _ptr(v_cube), _ptr(cube_keys), _ptr(sel_bitmap), _ptr(sel_count), _ptr(workspace), workspace_bytes,
        _stream_ptr(stream)))


def adaspark_attn_decode(handle: int, q_new, k_new, v_new, k_cube, v_cube, cube_keys, text_len, out,
                         sel_bitmap, workspace, workspace_bytes: int, stream=None):
    _check(handle, load().adaspark_attn_decode(
        handle, _ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cube), _ptr(v_cube), _ptr(cube_keys),
        _ptr(text_len), _ptr(out), _ptr(sel_bitmap), _ptr(workspace), workspace_bytes,
        _stream_ptr(stream)))


STATIC_SCRATCH_BYTES = 8 << 20


def adaspark_attn_decode_static(handle: int, q_new, k_new, v_new, k_cube, v_cube, cube_keys, text_len,
                                out, sel_bitmap, stream=None):
    """Decode step that takes no workspace: for callers that cannot allocate device memory when
    they decode (all memory already owned by their own pool, or no cudaMalloc allowed inside the
    serving loop).  Scratch is the library's built-in 8 MiB array, shared by all calls on a device."""
    _check(handle, load().adaspark_attn_decode_static(
        handle, _ptr(q_new), _ptr(k_new), _ptr(v_new), _ptr(k_cube), _ptr(v_cube), _ptr(cube_keys),
        _ptr(text_len), _ptr(out), _ptr(sel_bitmap), _stream_ptr(stream)))


def adaspark_attn_debug_umma_selftest(a, b, c, d_out, e_out, status, stream=None) -> int:
    """128x128x128 tcgen05 self-test (see include/adaspark_attn_debug.h); returns the status code."""
    return int(load().adaspark_attn_debug_umma_selftest(_ptr(a), _ptr(b), _ptr(c), _ptr(d_out),
                                                       _ptr(e_out), _ptr(status), _stream_ptr(stream)))


def adaspark_attn_debug_imma_selftest(a, b, d_out, status, stream=None) -> int:
    """128x128x128 int8 tcgen05 self-test (see include/adaspark_attn_debug.h); returns the status code."""
    return int(load().adaspark_attn_debug_imma_selftest(_ptr(a), _ptr(b), _ptr(d_out), _ptr(status),
                                                       _stream_ptr(stream)))


def adaspark_attn_debug_wait_timeout(limit_ns: int, status, waited_ns, stream=None) -> int:
    """A bounded device wait that is made to expire (see include/adaspark_attn_debug.h)."""
    return int(load().adaspark_attn_debug_wait_timeout(int(limit_ns), _ptr(status), _ptr(waited_ns),
                                                       _stream_ptr(stream)))


def adaspark_attn_debug_fastdiv(n: int, d: int) -> int:
    """n // d by the kernels' multiply-shift index arithmetic (host only)."""
    return int(load().adaspark_attn_debug_fastdiv(n, d))


def adaspark_attn_destroy(handle: int):
    load().adaspark_attn_destroy(handle)


def adaspark_attn_last_launch_count(handle: int) -> int:
    return int(load().adaspark_attn_last_launch_count(handle))


def adaspark_attn_set_prefill_kernel(handle: int, which: int):
    _check(handle, load().adaspark_attn_set_prefill_kernel(handle, which))


def adaspark_attn_set_gather(handle: int, pairs_per_block: float, budget_bytes: int):
    _check(handle, load().adaspark_attn_set_gather(handle, float(pairs_per_block), int(budget_bytes)))


def adaspark_attn_enable_stage_timing(handle: int, enable: bool):
    _check(handle, load().adaspark_attn_enable_stage_timing(handle, int(enable)))


def adaspark_attn_get_stage_times(handle: int):
    """Milliseconds of the four stages of the last timed call (waits for its last event)."""
    ms = (ctypes.c_float * 4)()
    _check(handle, load().adaspark_attn_get_stage_times(handle, ms))
    return [float(x) for x in ms]


def adaspark_attn_get_attention_kernel_ms(handle: int) -> float:
    """Milliseconds of the union attention kernel of the last timed prefill."""
    ms = (ctypes.c_float * 1)()
    _check(handle, load().adaspark_attn_get_attention_kernel_ms(handle, ms))
    return float(ms[0])


class WorkspaceHeader(ctypes.Structure):
    _fields_ = [("status", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("executed_kv_blocks", ctypes.c_uint64), ("decode_kv_blocks", ctypes.c_uint64),
                ("fallback_rows", ctypes.c_uint32), ("max_tile_kv_blocks", ctypes.c_uint32),
                ("gather_entries", ctypes.c_uint32), ("gather_items", ctypes.c_uint32),
                ("gather_pair_tiles", ctypes.c_uint32), ("reserved2", ctypes.c_uint32)]


# ---- a small convenience owner of the handle and of the caller-side buffers --------------------

class AdaSAttn:
    """Owns a handle plus the torch-allocated caches and workspace for one partition."""

    def __init__(self, *, cube, n_q_heads, n_kv_heads, head_dim, top_p, softmax_scale=0.0,
                 device: int = 0, top_k: int = 0):
        self.cfg = Config(cube[0], cube[1], cube[2], n_q_heads, n_kv_heads, head_dim, float(top_p),
                          float(softmax_scale), device, int(top_k))
        self.handle = adaspark_attn_create(self.cfg)
        self.device = torch.device("cuda", device)
        self.layout: Optional[Layout] = None

    def set_gather(self, pairs_per_block: float, budget_bytes: int = 24 << 30):
        """Threshold and workspace budget of the query-gather path (budget: before partition())."""
        adaspark_attn_set_gather(self.handle, pairs_per_block, budget_bytes)

    def partition(self, batch, frames, grid_h, grid_w, n_text_max):
        self.ws_bytes = adaspark_attn_partition(self.handle, batch, frames, grid_h, grid_w, n_text_max)
        self.layout = lay = adaspark_attn_get_layout(self.handle)
        self.batch = batch
        dev, c = self.device, self.cfg
        self.k_cube = torch.empty(lay.k_cube_bytes // 2, dtype=torch.bfloat16, device=dev).view(
            batch, c.n_kv_heads, lay.s_cap, c.head_dim)
        self.v_cube = torch.empty(lay.v_cube_bytes // 2, dtype=torch.bfloat16, device=dev).view(
            batch, c.n_kv_heads, lay.s_cap // 64, c.head_dim, 64)
        self.cube_keys = torch.empty(batch, c.n_kv_heads, lay.n_cubes, c.head_dim,
                                     dtype=torch.float32, device=dev)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        return self

    def forward(self, q, k, v, n_text, *, out=None, want_selection=False, stream=None, n_prefix=0):
        """q may be None: builds only the caches.  Returns (out, sel_bitmap, sel_count).
        n_prefix > 0: the first n_prefix tokens of the tensors are text that precedes the video."""
        lay = self.layout
        bitmap = count = None
        if q is not None:
            if out is None:
                out = torch.empty_like(q)
            if want_selection:
                B, S, Hq, _ = q.shape
                bitmap = torch.empty(B, Hq, S, lay.bitmap_words, dtype=torch.int32, device=q.device)
                count = torch.empty(B, Hq, S, dtype=torch.int32, device=q.device)
        if n_prefix:
            adaspark_attn_forward_prefix(self.handle, q, k, v, n_prefix, n_text, out, self.k_cube, self.v_cube,
                                         self.cube_keys, bitmap, count, self.workspace, self.ws_bytes, stream)
        else:
            adaspark_attn_forward(self.handle, q, k, v, n_text, out, self.k_cube, self.v_cube,
                                  self.cube_keys, bitmap, count, self.workspace, self.ws_bytes, stream)
        return out, bitmap, count

    def forward_host(self, q_host, k_host, v_host, n_text, out_host, staging, stream=None):
        """Prefill with host tensors; `staging` = (q, k, v, out) device tensors of the same shapes."""
        qd, kd, vd, od = staging
        adaspark_attn_forward_host(self.handle, q_host, k_host, v_host, n_text, out_host, qd, kd, vd, od,
                                   self.k_cube, self.v_cube, self.cube_keys, self.workspace, self.ws_bytes, stream)
        return out_host

    def forward_chunk(self, q, k, v, frame_begin, frame_count, n_text, *, out=None, want_selection=False,
                      stream=None):
        """One chunk of a chunked prefill (n_text < 0: more video follows).  q may be None."""
        lay = self.layout
        bitmap = count = None
        if q is not None:
            if out is None:
                out = torch.empty_like(q)
            if want_selection:
                B, S, Hq, _ = q.shape
                bitmap = torch.empty(B, Hq, S, lay.bitmap_words, dtype=torch.int32, device=q.device)
                count = torch.empty(B, Hq, S, dtype=torch.int32, device=q.device)
        adaspark_attn_forward_chunk(self.handle, q, k, v, frame_begin, frame_count, n_text, out, self.k_cube,
                                    self.v_cube, self.cube_keys, bitmap, count, self.workspace, self.ws_bytes,
                                    stream)
        return out, bitmap, count

    def decode(self, q_new, k_new, v_new, text_len, *, out=None, want_selection=False, stream=None):
        lay = self.layout
        if out is None:
            out = torch.empty_like(q_new)
        bitmap = None
        if want_selection:
            B, _, Hq, _ = q_new.shape
            bitmap = torch.empty(B, Hq, lay.bitmap_words, dtype=torch.int32, device=q_new.device)
        adaspark_attn_decode(self.handle, q_new, k_new, v_new, self.k_cube, self.v_cube,
                             self.cube_keys, text_len, out, bitmap, self.workspace, self.ws_bytes,
                             stream)
        return out, bitmap

    def header(self) -> WorkspaceHeader:
        """Copy of the workspace header of the last call (synchronises the device)."""
        raw = self.workspace[:ctypes.sizeof(WorkspaceHeader)].cpu().numpy().tobytes()
        return WorkspaceHeader.from_buffer_copy(raw)

    def launches(self) -> int:
        return adaspark_attn_last_launch_count(self.handle)

    def close(self):
        if self.handle:
            adaspark_attn_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
