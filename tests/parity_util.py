"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI and compare it
with the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2604_08077_b200 import binding

MAX_ABS_TOL = 2e-2       # bf16 inputs, fp32 accumulation (stated target of the build)
MEAN_REL_TOL = 1e-2      # mean|o - o_ref| / mean|o_ref|
TIE_MARGIN = 1e-6        # rows whose cumulative-probability margin is below this may differ


def make_engine(wl, n_text_max=None, top_p=None, prefill_kernel=None):
    eng = binding.AdaSAttn(cube=wl.cube, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.D,
                           top_p=wl.top_p if top_p is None else top_p, top_k=getattr(wl, "top_k", 0))
    eng.partition(wl.B, wl.T, wl.H, wl.W, wl.n_text if n_text_max is None else n_text_max)
    if prefill_kernel is not None:
        binding.adaspark_attn_set_prefill_kernel(eng.handle, prefill_kernel)
    return eng


def oracle_shape(wl, top_p=None):
    """Oracle shape with p exactly as the C ABI receives it (a float32)."""
    p = wl.top_p if top_p is None else top_p
    return oracle.shape_of(wl, top_p=float(np.float32(p)))


def unpack_bitmap(words: torch.Tensor, n_cubes: int) -> np.ndarray:
    """int32 words [..., W] -> uint8 flags [..., N]."""
    w = words.cpu().numpy().view(np.uint32)
    bits = (w[..., :, None] >> np.arange(32, dtype=np.uint32)) & 1
    return bits.reshape(*w.shape[:-1], -1)[..., :n_cubes].astype(np.uint8)


def run_forward(wl, *, top_p=None, prefill_kernel=None, want_selection=True):
    eng = make_engine(wl, top_p=top_p, prefill_kernel=prefill_kernel)
    q, k, v = wl.q.cuda(), wl.k.cuda(), wl.v.cuda()
    out, bitmap, count = eng.forward(q, k, v, wl.n_text, want_selection=want_selection)
    torch.cuda.synchronize()
    return eng, out, bitmap, count


def compare_rows(wl, rows, gpu_out, gpu_bitmap, gpu_count=None, *, top_p=None, label=""):
    """Oracle vs CUDA on the listed (b, h, raster token) rows.  Returns a report dict.

    Selection must be bit-exact except on rows whose oracle tie margin is < 1e-6 (counted);
    outputs are compared on the rows with identical selection."""
    sh = oracle_shape(wl, top_p)
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 3)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows)
    dev = gpu_out.device
    b, h, n = (torch.from_numpy(np.ascontiguousarray(rows[:, i])).to(dev) for i in range(3))
    words = gpu_bitmap[b, h, n]
    got_sel = unpack_bitmap(words, sh.N)
    same = (got_sel == res["sel"]).all(axis=1)
    exempt = ~same & (res["margin"] < TIE_MARGIN)
    bad = ~same & ~exempt
    assert not bad.any(), (f"{label}: {bad.sum()} rows differ from the oracle selection with margin "
                           f">= {TIE_MARGIN}; first {rows[bad][:5].tolist()} margins {res['margin'][bad][:5]}")
    if gpu_count is not None:
        got_cnt = gpu_count[b, h, n].cpu().numpy()
        assert np.array_equal(got_cnt, got_sel.sum(axis=1)), f"{label}: sel_count != popcount(bitmap)"
    got = gpu_out[b, n, h].float().cpu().numpy()
    ref = res["out"]
    ok = same
    max_abs = float(np.abs(got[ok] - ref[ok]).max()) if ok.any() else 0.0
    mean_rel = float(np.abs(got[ok] - ref[ok]).mean() / np.abs(ref[ok]).mean()) if ok.any() else 0.0
    assert max_abs <= MAX_ABS_TOL, f"{label}: max-abs error {max_abs} > {MAX_ABS_TOL}"
    assert mean_rel <= MEAN_REL_TOL, f"{label}: mean-relative error {mean_rel} > {MEAN_REL_TOL}"
    assert np.isfinite(got).all()
    return {"rows": len(rows), "tie_exempt": int(exempt.sum()),
            "near_tie_rows": int((res["margin"] < TIE_MARGIN).sum()), "max_abs": max_abs,
            "mean_rel": mean_rel, "mean_selected": float(res["count"].mean()),
            "mean_attended": float(res["n_attended"].mean())}


def sample_rows(wl, n_random, seed=0, whole_tiles=()):
    """Random rows plus every row of the given (b, h, tile) query tiles (tile = 128 consecutive
    cube-major positions)."""
    rng = np.random.default_rng(seed)
    sh = oracle.shape_of(wl)
    rows = np.stack([rng.integers(0, wl.B, n_random), rng.integers(0, wl.Hq, n_random),
                     rng.integers(0, wl.S, n_random)], axis=1)
    extra = []
    if whole_tiles:
        _, inv = oracle.positions(sh)
        for (b, h, t) in whole_tiles:
            for pos in range(t * 128, min(t * 128 + 128, wl.S)):
                extra.append((b, h, int(inv[pos])))
    if extra:
        rows = np.concatenate([rows, np.asarray(extra, dtype=np.int64)])
    return rows
