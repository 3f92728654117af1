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


FORCE_GATHER = 1e30   # threshold of the query-gather path that sends every pair with a selected cube through it


def make_engine(wl, n_text_max=None, top_p=None, prefill_kernel=None, gather=None, gather_budget=24 << 30):
    """gather: None = the library's default decision; 0 = union path only; FORCE_GATHER = gather path
    wherever a row selected a cube before its local range."""
    eng = binding.AdaSAttn(cube=wl.cube, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.D,
                           top_p=wl.top_p if top_p is None else top_p, top_k=getattr(wl, "top_k", 0))
    if gather is not None:
        eng.set_gather(gather, gather_budget)
    eng.partition(wl.B, wl.T, wl.H, wl.W, (wl.n_text + getattr(wl, "n_prefix", 0)) if n_text_max is None else n_text_max)
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


def run_forward(wl, *, top_p=None, prefill_kernel=None, want_selection=True, gather=None, gather_budget=24 << 30):
    eng = make_engine(wl, top_p=top_p, prefill_kernel=prefill_kernel, gather=gather, gather_budget=gather_budget)
    q, k, v = wl.q.cuda(), wl.k.cuda(), wl.v.cuda()
    out, bitmap, count = eng.forward(q, k, v, wl.n_text, want_selection=want_selection,
                                     n_prefix=getattr(wl, "n_prefix", 0))
    torch.cuda.synchronize()
    return eng, out, bitmap, count


def check_nucleus_legal(probs, oracle_sel, gpu_sel, top_p, top_k=0, tol=TIE_MARGIN):
    """Is ``gpu_sel`` a legal answer for a row whose oracle answer is ``oracle_sel``?

    A row may differ from the oracle only because of a tie inside ``tol``: the two sets then have
    sizes within one of each other, differ only in cubes whose probability lies within ``tol`` of the
    probability of the oracle's last selected cube, and the GPU set is itself a top-prefix whose mass
    reaches p while dropping its least probable member falls below p (both within ``tol``).  Returns
    None when legal, else a string saying what is wrong."""
    n = len(probs)
    o, g = oracle_sel[:n].astype(bool), gpu_sel[:n].astype(bool)
    if gpu_sel[n:].any():
        return "a cube outside the row's candidates is selected"
    if abs(int(o.sum()) - int(g.sum())) > 1:
        return f"set sizes {int(g.sum())} vs {int(o.sum())}"
    if not o.any() or not g.any():
        return "empty set on one side only"
    p_edge = probs[o].min()
    diff = o ^ g
    if (np.abs(probs[diff] - p_edge) > tol).any():
        return "sets differ in a cube that is not tied with the boundary cube"
    if (~g).any() and probs[g].min() < probs[~g].max() - tol:
        return "not a prefix of the probability order"
    if top_k > 0:
        return None if int(g.sum()) == int(o.sum()) else "Top-K size"
    mass = probs[g].sum()
    if mass < top_p - tol:
        return f"mass {mass} below p"
    if mass - probs[g].min() >= top_p + tol:
        return "not minimal: the set without its least probable cube still reaches p"
    return None


def check_selection(sh, wl, rows, got_sel, res, *, label=""):
    """Selection parity on the listed rows (res = oracle.rows(...) of the same rows).

    Bit-exact sets are required on every row whose oracle tie margin is >= 1e-6.  Rows inside the
    margin may differ, but then (a) the GPU set must still be a legal nucleus (check_nucleus_legal),
    and (b) there may be only few of them: the GPU evaluates Eqs. 1-2 with an absolute error far
    below the margin, so it can flip only a small share of the near-tie rows -- at most
    max(2, 5 %) of them is accepted.  Returns (same mask, counts dict)."""
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 3)
    same = (got_sel == res["sel"]).all(axis=1)
    near = res["margin"] < TIE_MARGIN
    bad = ~same & ~near
    assert not bad.any(), (f"{label}: {bad.sum()} rows differ from the oracle selection with margin "
                           f">= {TIE_MARGIN}; first {rows[bad][:5].tolist()} margins {res['margin'][bad][:5]}")
    differing = np.flatnonzero(~same)
    limit = max(2, int(0.05 * near.sum()))
    assert len(differing) <= limit, (f"{label}: {len(differing)} rows differ from the oracle (all inside "
                                     f"the tie margin) but only {limit} of the {int(near.sum())} near-tie "
                                     f"rows may")
    if len(differing):
        kbar = res["kbar"]
        G = sh.Hq // sh.Hkv
        pos_of, _ = oracle.positions(sh)
        qf = oracle.as_f32(wl.q)
        for i in differing:
            b, h, n = (int(x) for x in rows[i])
            pos = int(pos_of[n])
            P0 = sh.n_prefix
            n_cand = 0 if pos < P0 else ((pos - P0) // sh.C if pos < P0 + sh.N * sh.C else sh.N)
            _, probs, _ = oracle.select_row(qf[b, n, h], kbar[b, h // G], n_cand, sh.scale, sh.top_p, sh.top_k)
            why = check_nucleus_legal(probs, res["sel"][i], got_sel[i], sh.top_p, sh.top_k)
            assert why is None, f"{label}: row {rows[i].tolist()} differs from the oracle illegally: {why}"
    return same, {"rows": int(len(rows)), "differing": int(len(differing)), "near_tie": int(near.sum())}


def compare_rows(wl, rows, gpu_out, gpu_bitmap, gpu_count=None, *, top_p=None, label="", attend=True):
    """Oracle vs CUDA on the listed (b, h, raster token) rows.  Returns a report dict.

    Selection: see check_selection.  Outputs: every row is compared -- rows with the oracle's
    selection against the oracle's output, rows that legally differ against the oracle's attention
    evaluated on the GPU's own set (Eq. 3 with that set)."""
    sh = oracle_shape(wl, top_p)
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 3)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows, attend=attend)
    dev = gpu_bitmap.device
    b, h, n = (torch.from_numpy(np.ascontiguousarray(rows[:, i])).to(dev) for i in range(3))
    words = gpu_bitmap[b, h, n]
    got_sel = unpack_bitmap(words, sh.N)
    same, rep = check_selection(sh, wl, rows, got_sel, res, label=label)
    if gpu_count is not None:
        got_cnt = gpu_count[b, h, n].cpu().numpy()
        assert np.array_equal(got_cnt, got_sel.sum(axis=1)), f"{label}: sel_count != popcount(bitmap)"
    rep.update({"mean_selected": float(res["count"].mean()),
                "mean_attended": float(res["n_attended"].mean())})
    if not attend:
        return rep
    got = gpu_out[b, n, h].float().cpu().numpy()
    ref = res["out"].copy()
    if not same.all():
        ref[~same] = oracle.attend_given(sh, wl.q, wl.k, wl.v, rows[~same], got_sel[~same])
    max_abs = float(np.abs(got - ref).max()) if len(rows) else 0.0
    mean_rel = float(np.abs(got - ref).mean() / np.abs(ref).mean()) if len(rows) else 0.0
    assert max_abs <= MAX_ABS_TOL, f"{label}: max-abs error {max_abs} > {MAX_ABS_TOL}"
    assert mean_rel <= MEAN_REL_TOL, f"{label}: mean-relative error {mean_rel} > {MEAN_REL_TOL}"
    assert np.isfinite(got).all()
    rep.update({"max_abs": max_abs, "mean_rel": mean_rel})
    return rep


def random_rows(wl, n_rows, seed):
    rng = np.random.default_rng(seed)
    return np.stack([rng.integers(0, wl.B, n_rows), rng.integers(0, wl.Hq, n_rows),
                     rng.integers(0, wl.S, n_rows)], axis=1)


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
