"""GPU parity at the full sizes of the long-sequence benchmark configurations (configs 3, 4, 5):
the CUDA path runs the whole problem through the C ABI; the CPU oracle evaluates a seeded sample
of rows one by one (selection on many rows, outputs on fewer rows plus whole query tiles)."""
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import inputs

import parity_util as pu

pytestmark = pytest.mark.gpu


def _selection_sample(wl, bitmap, n_rows, seed, top_p=None):
    """Selection-only parity on n_rows random (head, token) rows."""
    sh = pu.oracle_shape(wl, top_p)
    rng = np.random.default_rng(seed)
    rows = np.stack([np.zeros(n_rows, np.int64), rng.integers(0, wl.Hq, n_rows),
                     rng.integers(0, wl.S, n_rows)], axis=1)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows, attend=False)
    dev = bitmap.device
    got = pu.unpack_bitmap(bitmap[0, torch.from_numpy(rows[:, 1]).to(dev),
                                  torch.from_numpy(rows[:, 2]).to(dev)], wl.N)
    diff = (got != res["sel"]).any(axis=1)
    bad = diff & (res["margin"] >= pu.TIE_MARGIN)
    assert not bad.any(), f"{bad.sum()} rows differ; first {rows[bad][:5].tolist()}"
    return {"rows": n_rows, "tie_exempt": int(diff.sum()),
            "near_tie": int((res["margin"] < pu.TIE_MARGIN).sum()),
            "mean_selected": float(res["count"].mean())}


def _free():
    gc.collect()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("sigma,p", [(1.5, 0.7), (3.0, 0.95), (0.5, 0.5), (1.5, 1.0)])
def test_config3_full_size_sampled_rows(sigma, p):
    """Config 3 (65536 video tokens in 1024 cubes + 256 text) at four corners of its (sigma, p) sweep."""
    wl = inputs.config3(sigma=sigma, top_p=p)
    eng, out, bitmap, count = pu.run_forward(wl)
    n_tiles = (wl.S + 127) // 128
    tiles = [(0, 0, 0), (0, 11, n_tiles // 2), (0, 27, n_tiles - 1)]
    n_random = 300 if p >= 1.0 else 600
    rows = pu.sample_rows(wl, n_random, seed=3, whole_tiles=tiles if p < 1.0 else tiles[:1] + tiles[2:])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label=f"cfg3 s={sigma} p={p}")
    print("cfg3", sigma, p, rep)
    if p < 1.0:
        print("cfg3 selection", _selection_sample(wl, bitmap, 20000, seed=33))
    hdr = eng.header()
    assert hdr.status == 0
    del eng, out, bitmap, count
    _free()


def test_cohesive_queries_256_token_cubes():
    """Config-2 shapes with the paper's default cube size (4x8x8 = 256 tokens), p = 0.7 and queries
    that share an offset inside a cube: the attention kernel then skips most key blocks (the union
    of a tile's selections is sparse), which the dense-union benchmark configs never exercise."""
    wl = inputs.config2_cohesive(top_p=0.7, cube=(4, 8, 8))
    eng, out, bitmap, count = pu.run_forward(wl)
    n_tiles = (wl.S + 127) // 128
    rows = pu.sample_rows(wl, 1500, seed=6, whole_tiles=[(0, 3, 1), (0, 17, n_tiles // 2), (0, 27, n_tiles - 1)])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label="cohesive")
    hdr = eng.header()
    dense_blocks = sum(2 * ((min(p * 256 + 256, wl.S) + 63) // 64) for p in range((wl.S + 255) // 256)) * wl.Hq
    print("cohesive", rep, "executed/dense blocks", hdr.executed_kv_blocks / dense_blocks)
    assert hdr.status == 0 and hdr.executed_kv_blocks < 0.8 * dense_blocks
    del eng, out, bitmap, count
    _free()


def test_maximum_cube_count_and_smallest_cubes():
    """4096 cubes (the partition limit) of 16 tokens (the smallest cube): 65536 video tokens.  Every
    64-key block then holds four cubes, so the attention kernel's per-chunk masks are mixed almost
    everywhere, and the selection runs on the longest rows the library accepts."""
    wl = inputs.make_prefill("n4096_c16", seed=77, B=1, T=256, H=16, W=16, cube=(1, 4, 4), n_text=33,
                             Hq=4, Hkv=2, D=128, top_p=0.8, offset_std=1.5)
    assert wl.N == 4096
    eng, out, bitmap, count = pu.run_forward(wl)
    n_tiles = (wl.S + 127) // 128
    rows = pu.sample_rows(wl, 300, seed=8, whole_tiles=[(0, 0, 3), (0, 3, n_tiles - 1)])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label="n4096")
    print("n4096", rep)
    print("n4096 selection", _selection_sample(wl, bitmap, 6000, seed=88))
    assert eng.header().status == 0
    del eng, out, bitmap, count
    _free()


def test_config4_full_size_sampled_rows():
    """Config 4 (131072 video tokens in 2048 cubes, half of the frames static, no text)."""
    wl = inputs.config4()
    eng, out, bitmap, count = pu.run_forward(wl)
    n_tiles = wl.S // 128
    rows = pu.sample_rows(wl, 500, seed=4,
                          whole_tiles=[(0, 0, 0), (0, 5, n_tiles // 2 - 1), (0, 20, n_tiles - 1)])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label="cfg4")
    print("cfg4", rep)
    print("cfg4 selection", _selection_sample(wl, bitmap, 20000, seed=44))
    assert eng.header().status == 0
    del eng, out, bitmap, count
    _free()


def test_config5_full_batch():
    """Config 5 at its full batch of 16 sequences: the CUDA path decodes all of them; the oracle
    evaluates every head of four of the sequences (first, last, two in between) with different
    cached text lengths."""
    wl = inputs.config5(B=16, device="cuda")
    text_len = [512 - 17 * b for b in range(wl.B)]
    eng = pu.make_engine(wl)
    eng.forward(None, wl.k, wl.v, wl.n_text)
    tl = torch.tensor(text_len, dtype=torch.int32, device="cuda")
    out, bitmap = eng.decode(wl.q_new, wl.k_new, wl.v_new, tl, want_selection=True)
    torch.cuda.synchronize()
    assert eng.header().status == 0
    idx = [0, 5, 10, 15]
    sh = pu.oracle_shape(wl)
    for b in idx:
        kb, vb = wl.k[b:b + 1].cpu(), wl.v[b:b + 1].cpu()
        res = oracle.decode(sh, kb, vb, [text_len[b]], wl.q_new[b:b + 1].cpu(),
                            wl.k_new[b:b + 1].cpu(), wl.v_new[b:b + 1].cpu())
        got_sel = pu.unpack_bitmap(bitmap[b:b + 1], sh.N)
        same = (got_sel == res["sel"]).all(axis=-1)
        bad = ~same & (res["margin"] >= pu.TIE_MARGIN)
        assert not bad.any(), f"sequence {b}: selection differs on heads {np.argwhere(bad).tolist()}"
        got = out[b:b + 1, 0].float().cpu().numpy()
        err = np.abs(got[same] - res["out"][same])
        assert err.max() <= pu.MAX_ABS_TOL
        assert err.mean() / np.abs(res["out"][same]).mean() <= pu.MEAN_REL_TOL
        print("cfg5 seq", b, "tie-exempt", int((~same).sum()), "max_abs", float(err.max()),
              "mean selected", float(res["count"].mean()))
    del eng, out, bitmap, wl
    _free()
