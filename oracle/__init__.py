"""ctypes front end of the AdaS-Attn CPU oracle (``adas_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The product package never imports
it and it never imports the product package's CUDA binding.

The C file holds all of the arithmetic (Sec. 3.1-3.2, Eqs. 1-3 of the paper); this module only
compiles it with gcc, marshals numpy arrays and, for the decode case, appends the new token to
the cached sequence before asking for the last row (a decode step is a text-rule row).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adas_oracle.c")
_LIB = os.path.join(_HERE, "libadas_oracle.so")
_lib = None


class Shape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("W", ctypes.c_int32), ("ct", ctypes.c_int32), ("ch", ctypes.c_int32),
                ("cw", ctypes.c_int32), ("n_text", ctypes.c_int32), ("Hq", ctypes.c_int32),
                ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32), ("top_p", ctypes.c_double),
                ("scale", ctypes.c_double), ("top_k", ctypes.c_int32), ("n_prefix", ctypes.c_int32)]

    @property
    def N(self) -> int:
        return (-(-self.T // self.ct)) * (-(-self.H // self.ch)) * (-(-self.W // self.cw))

    @property
    def C(self) -> int:
        return self.ct * self.ch * self.cw

    @property
    def S_v(self) -> int:
        return self.T * self.H * self.W

    @property
    def S(self) -> int:
        return self.n_prefix + self.S_v + self.n_text

    @property
    def n_positions(self) -> int:
        """Slots of the causal order: prefix, N cubes of C slots (boundary cubes of a grid the window
        does not divide hold fewer tokens than slots), text."""
        return self.n_prefix + self.N * self.C + self.n_text


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, strict fp64: no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.adas_oracle_num_cubes.restype = ctypes.c_int64
        _lib.adas_oracle_num_positions.restype = ctypes.c_int64
        _lib.adas_oracle_position.restype = ctypes.c_int64
        _lib.adas_oracle_position.argtypes = [ctypes.POINTER(Shape), ctypes.c_int64]
        _lib.adas_oracle_select_row.restype = ctypes.c_int64
        _lib.adas_oracle_select_row.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_double,
            ctypes.c_double, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    return _lib


def n_threads() -> int:
    """Host threads the OpenMP loops use (OMP_NUM_THREADS or all cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


def make_shape(*, B, T, H, W, cube, n_text, Hq, Hkv, D, top_p, scale: Optional[float] = None,
               top_k: int = 0, n_prefix: int = 0) -> Shape:
    ct, ch, cw = cube
    return Shape(B, T, H, W, ct, ch, cw, n_text, Hq, Hkv, D, float(top_p),
                 float(scale) if scale else 1.0 / float(np.sqrt(D)), int(top_k), int(n_prefix))


def shape_of(wl, top_p: Optional[float] = None, top_k: Optional[int] = None) -> Shape:
    """Shape of a ``paper_2604_08077_b200.inputs.Workload`` (duck-typed; no import)."""
    return make_shape(B=wl.B, T=wl.T, H=wl.H, W=wl.W, cube=wl.cube, n_text=wl.n_text, Hq=wl.Hq,
                      Hkv=wl.Hkv, D=wl.D, top_p=wl.top_p if top_p is None else top_p,
                      top_k=getattr(wl, "top_k", 0) if top_k is None else top_k,
                      n_prefix=getattr(wl, "n_prefix", 0))


def as_f32(t) -> np.ndarray:
    """torch (bf16/fp32) or numpy tensor -> contiguous float32 numpy (exact for bf16)."""
    if hasattr(t, "detach"):
        t = t.detach().cpu().float().numpy()
    return np.ascontiguousarray(t, dtype=np.float32)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def positions(shape: Shape):
    """(pos_of_raster [S], raster_of_pos [n_positions], -1 where a slot holds no token): the order
    of the tokens and its inverse (O1)."""
    pos = np.empty(shape.S, np.int64)
    inv = np.empty(shape.n_positions, np.int64)
    lib().adas_oracle_positions(ctypes.byref(shape), _p(pos), _p(inv))
    return pos, inv


def mean_keys(shape: Shape, k: np.ndarray) -> np.ndarray:
    """Mean key per (batch, KV head, cube): fp64 [B,Hkv,N,D] (O2)."""
    k = as_f32(k)
    assert k.shape == (shape.B, shape.S, shape.Hkv, shape.D), k.shape
    kbar = np.empty((shape.B, shape.Hkv, shape.N, shape.D), np.float64)
    lib().adas_oracle_mean_keys(ctypes.byref(shape), _p(k), _p(kbar))
    return kbar


def select_row(q: np.ndarray, kbar_g: np.ndarray, n_cand: int, scale: float, top_p: float, top_k: int = 0):
    """One row of O3+O4.  Returns (sel uint8[n_cand], probs float64[n_cand], margin)."""
    q = as_f32(q)
    kbar_g = np.ascontiguousarray(kbar_g, np.float64)
    D = q.shape[0]
    sel = np.zeros(max(n_cand, 1), np.uint8)
    probs = np.zeros(max(n_cand, 1), np.float64)
    margin = ctypes.c_double(0.0)
    lib().adas_oracle_select_row(_p(q), _p(kbar_g), n_cand, D, float(scale), float(top_p), int(top_k),
                                 _p(sel), _p(probs), ctypes.addressof(margin))
    return sel[:n_cand], probs[:n_cand], margin.value


def rows(shape: Shape, q, k, v, row_list: Sequence, *, kbar: Optional[np.ndarray] = None,
         attend: bool = True) -> dict:
    """Evaluate rows (b, query head, raster token).  Returns out/sel/count/margin/n_attended."""
    q, k = as_f32(q), as_f32(k)
    v = as_f32(v) if attend else None
    assert q.shape == (shape.B, shape.S, shape.Hq, shape.D), (q.shape, shape.S)
    assert k.shape == (shape.B, shape.S, shape.Hkv, shape.D)
    if kbar is None:
        kbar = mean_keys(shape, k)
    r = np.ascontiguousarray(np.asarray(row_list, dtype=np.int64).reshape(-1, 3))
    n = r.shape[0]
    out = np.empty((n, shape.D), np.float64) if attend else None
    sel = np.empty((n, shape.N), np.uint8)
    count = np.empty(n, np.int32)
    margin = np.empty(n, np.float64)
    natt = np.empty(n, np.int64)
    lib().adas_oracle_rows(ctypes.byref(shape), _p(q), _p(k), _p(v), _p(kbar),
                           ctypes.c_int64(n), _p(r), _p(out), _p(sel), _p(count), _p(margin),
                           _p(natt))
    return {"out": out, "sel": sel, "count": count, "margin": margin, "n_attended": natt,
            "rows": r, "kbar": kbar}


def attend_given(shape: Shape, q, k, v, row_list: Sequence, sel: np.ndarray) -> np.ndarray:
    """O5 with a caller-supplied selection (0/1 flags [nrows, N])."""
    q, k, v = as_f32(q), as_f32(k), as_f32(v)
    r = np.ascontiguousarray(np.asarray(row_list, dtype=np.int64).reshape(-1, 3))
    sel = np.ascontiguousarray(sel, np.uint8)
    assert sel.shape == (r.shape[0], shape.N)
    out = np.empty((r.shape[0], shape.D), np.float64)
    lib().adas_oracle_attend_given(ctypes.byref(shape), _p(q), _p(k), _p(v),
                                   ctypes.c_int64(r.shape[0]), _p(r), _p(sel), _p(out))
    return out


def all_rows(shape: Shape) -> np.ndarray:
    """Every (b, h, n) row of the problem, as an int64 [B*Hq*S, 3] array."""
    b, h, n = np.meshgrid(np.arange(shape.B), np.arange(shape.Hq), np.arange(shape.S),
                          indexing="ij")
    return np.stack([b.ravel(), h.ravel(), n.ravel()], axis=1).astype(np.int64)


def decode(shape: Shape, k_cache, v_cache, text_len: Sequence[int], q_new, k_new, v_new,
           *, attend: bool = True, batch_index: Optional[Sequence[int]] = None) -> dict:
    """O6: one decode step per sequence.

    ``k_cache``/``v_cache`` are raster [B, S_v + n_text_cap, Hkv, D] holding ``text_len[b]`` valid
    text tokens; the new token's K/V is appended at text slot ``text_len[b]`` and the new query
    is evaluated as a text row there (it attends itself).  Sequences are evaluated one at a
    time, each as a batch-1 problem of ``S_v + text_len[b] + 1`` tokens.
    Returns out [B,Hq,D], sel [B,Hq,N], count [B,Hq], margin [B,Hq].
    """
    k_cache, v_cache = as_f32(k_cache), as_f32(v_cache)
    q_new, k_new, v_new = as_f32(q_new), as_f32(k_new), as_f32(v_new)
    B = k_cache.shape[0]
    idx = list(range(B)) if batch_index is None else list(batch_index)
    outs, sels, counts, margins = [], [], [], []
    for b in idx:
        tl = int(text_len[b])
        s1 = Shape(1, shape.T, shape.H, shape.W, shape.ct, shape.ch, shape.cw, tl + 1, shape.Hq,
                   shape.Hkv, shape.D, shape.top_p, shape.scale, shape.top_k, 0)
        Sv = shape.S_v
        k1 = np.concatenate([k_cache[b, :Sv + tl], k_new[b]], axis=0)[None]
        v1 = np.concatenate([v_cache[b, :Sv + tl], v_new[b]], axis=0)[None]
        q1 = np.zeros((1, Sv + tl + 1, shape.Hq, shape.D), np.float32)
        q1[0, -1] = q_new[b, 0]
        rl = [(0, h, Sv + tl) for h in range(shape.Hq)]
        res = rows(s1, q1, k1, v1, rl, attend=attend)
        outs.append(res["out"])
        sels.append(res["sel"])
        counts.append(res["count"])
        margins.append(res["margin"])
    return {"out": np.stack(outs) if attend else None, "sel": np.stack(sels),
            "count": np.stack(counts), "margin": np.stack(margins)}
