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


def _selection_sample(wl, bitmap, n_rows, seed, top_p=None, label=""):
    """Selection-only parity on n_rows random (head, token) rows (see parity_util.check_selection)."""
    rep = pu.compare_rows(wl, pu.random_rows(wl, n_rows, seed), None, bitmap, top_p=top_p, attend=False,
                          label=label)
    return rep


def _free():
    gc.collect()
    torch.cuda.empty_cache()


_CFG3 = {}


def _config3(sigma):
    """The three config-3 datasets (one per sigma) are drawn once and shared by the five values of p."""
    if sigma not in _CFG3:
        _CFG3.clear()                      # one dataset at a time in host memory
        _CFG3[sigma] = inputs.config3(sigma=sigma)
    return _CFG3[sigma]


CFG3_OUTPUT_POINTS = {(0.5, 0.5), (0.5, 1.0), (3.0, 0.5), (3.0, 1.0), (1.5, 0.9), (0.5, 0.95), (3.0, 0.9), (1.5, 0.5)}
# points whose selections are sparse enough for the library's own decision to send (nearly) every pair of
# query tiles through the query-gather path, and points that must stay on the union path
CFG3_GATHERED = {(3.0, 0.5), (3.0, 0.7), (3.0, 0.9), (1.5, 0.5)}
CFG3_UNION = {(0.5, 0.5), (0.5, 0.7), (0.5, 0.9), (0.5, 0.95), (1.5, 0.9), (1.5, 0.95)}


@pytest.mark.parametrize("p", [0.5, 0.7, 0.9, 0.95, 1.0])
@pytest.mark.parametrize("sigma", [0.5, 1.5, 3.0])
def test_config3_full_size_sweep(sigma, p):
    """Config 3 (65536 video tokens in 1024 cubes + 256 text) at all 15 points of its (sigma, p)
    sweep: selection on 20000 sampled rows everywhere; outputs on sampled rows plus whole query tiles
    (first, middle, last) at the corners of the sweep, at the sharpest point (sigma 3, p 0.5) and at
    interior points, among them points that run through the query-gather path by the library's default rule."""
    wl = _config3(sigma)
    eng, out, bitmap, count = pu.run_forward(wl, top_p=p)
    label = f"cfg3 s={sigma} p={p}"
    if p < 1.0:
        print(label, "selection", _selection_sample(wl, bitmap, 20000, seed=33, top_p=p, label=label))
    if (sigma, p) in CFG3_OUTPUT_POINTS:
        n_tiles = (wl.S + 127) // 128
        tiles = [(0, 0, 0), (0, 11, n_tiles // 2), (0, 27, n_tiles - 1)]
        n_random = 300 if p >= 1.0 else 600
        rows = pu.sample_rows(wl, n_random, seed=3, whole_tiles=tiles if p < 1.0 else tiles[:1] + tiles[2:])
        rep = pu.compare_rows(wl, rows, out, bitmap, count, top_p=p, label=label)
        print(label, rep)
    hdr = eng.header()
    assert hdr.status == 0
    n_pairs = ((wl.S + 255) // 256) * wl.Hq
    print(label, "gathered pairs", hdr.gather_pair_tiles, "of", n_pairs, "entries", hdr.gather_entries)
    if (sigma, p) in CFG3_GATHERED:
        assert hdr.gather_pair_tiles > 0.9 * n_pairs
    if (sigma, p) in CFG3_UNION or p >= 1.0:
        assert hdr.gather_pair_tiles == 0 and hdr.gather_entries == 0
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
    print("n4096 selection", _selection_sample(wl, bitmap, 6000, seed=88, label="n4096"))
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
    print("cfg4 selection", _selection_sample(wl, bitmap, 20000, seed=44, label="cfg4"))
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
    from test_gpu_decode import compare_decode
    cpu = inputs.Workload(name=wl.name, B=wl.B, T=wl.T, H=wl.H, W=wl.W, cube=wl.cube, n_text=wl.n_text,
                          Hq=wl.Hq, Hkv=wl.Hkv, D=wl.D, top_p=wl.top_p,
                          k=wl.k[idx].cpu(), v=wl.v[idx].cpu(), q_new=wl.q_new[idx].cpu(),
                          k_new=wl.k_new[idx].cpu(), v_new=wl.v_new[idx].cpu())
    cpu.B = len(idx)
    rep = compare_decode(cpu, [text_len[b] for b in idx], out[idx], bitmap[idx], label="cfg5 batch 16")
    print("cfg5 batch 16, sequences", idx, rep)
    del eng, out, bitmap, wl
    _free()
