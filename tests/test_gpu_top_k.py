"""GPU parity of the Top-K selection rule (keep the K most probable candidate cubes) against the
CPU oracle, through the C ABI: every row of small problems, a decode step, and sampled rows of the
config-2 shape."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import inputs

import parity_util as pu
from test_gpu_decode import compare_decode, run_decode

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("k", [1, 3, 40])
def test_small_prefill_top_k_every_row(k, kernel):
    wl = dataclasses.replace(inputs.small_prefill(seed=61, T=16, H=8, W=8, n_text=21), top_k=k)
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=kernel)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label=f"top_k={k}")
    sh = oracle.shape_of(wl)
    pos, _ = oracle.positions(sh)
    n_cand = np.where(np.arange(wl.S) < wl.S_v, pos // wl.C, wl.N)
    got = pu.unpack_bitmap(bitmap, wl.N).sum(-1)
    assert np.array_equal(got, np.broadcast_to(np.minimum(n_cand, k), got.shape))
    print(k, kernel, rep)


def test_decode_top_k():
    wl = dataclasses.replace(inputs.small_decode(seed=62, T=32, H=8, W=8, n_text=19), top_k=5)
    text_len = [wl.n_text, wl.n_text - 4]
    eng, out, bitmap = run_decode(wl, text_len)
    rep = compare_decode(wl, text_len, out, bitmap, label="decode top_k")
    assert (pu.unpack_bitmap(bitmap, wl.N).sum(-1) == 5).all()
    print(rep)


def test_config2_shape_top_k_sampled_rows():
    wl = dataclasses.replace(inputs.config2(), top_k=32)
    eng, out, bitmap, count = pu.run_forward(wl)
    rows = pu.sample_rows(wl, 1200, seed=7, whole_tiles=[(0, 2, 0), (0, 9, 77), (0, 27, 128)])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label="cfg2 top_k=32")
    assert eng.header().status == 0
    print("cfg2 top_k", rep)
