"""Chunked prefill through the C ABI: the video is fed in runs of frames that append their cubes to
the caches; every row must equal the one-shot prefill (same selection, outputs within the bf16
tolerance) and the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu


def run_chunked(wl, frame_chunks, text_with_last=True, want_selection=True):
    """frame_chunks: list of (frame_begin, frame_count).  Returns (engine, out, bitmap, count) in the
    layout of a one-shot forward."""
    eng = pu.make_engine(wl)
    q, k, v = wl.q.cuda(), wl.k.cuda(), wl.v.cuda()
    hw = wl.H * wl.W
    outs, bms, cnts = [], [], []
    calls = [(fb, fc, -1) for fb, fc in frame_chunks]
    if text_with_last:
        fb, fc, _ = calls[-1]
        calls[-1] = (fb, fc, wl.n_text)
    else:
        calls.append((wl.T, 0, wl.n_text))
    for fb, fc, nt in calls:
        lo, hi = fb * hw, (fb + fc) * hw + max(nt, 0)
        o, b, c = eng.forward_chunk(q[:, lo:hi].contiguous(), k[:, lo:hi].contiguous(), v[:, lo:hi].contiguous(),
                                    fb, fc, nt, want_selection=want_selection)
        torch.cuda.synchronize()
        assert eng.header().status == 0
        outs.append(o)
        bms.append(b)
        cnts.append(c)
    return eng, torch.cat(outs, 1), torch.cat(bms, 2), torch.cat(cnts, 2)


@pytest.mark.parametrize("kernel", [1, 0])
def test_small_chunked_prefill_every_row(kernel):
    """8 time blocks fed as 2 + 4 + 2 (+ text in a call of its own): caches, selection and outputs
    of every row against the oracle and against the one-shot forward."""
    wl = inputs.small_prefill(seed=91, T=32, H=8, W=8, n_text=23, Hq=4, Hkv=2, D=128, top_p=0.85)
    one, out1, bm1, cnt1 = pu.run_forward(wl, prefill_kernel=kernel)
    eng = pu.make_engine(wl, prefill_kernel=kernel)
    q, k, v = wl.q.cuda(), wl.k.cuda(), wl.v.cuda()
    hw = wl.H * wl.W
    outs, bms = [], []
    for fb, fc, nt in [(0, 8, -1), (8, 16, -1), (24, 8, -1), (32, 0, wl.n_text)]:
        lo, hi = fb * hw, (fb + fc) * hw + max(nt, 0)
        o, b, _ = eng.forward_chunk(q[:, lo:hi].contiguous(), k[:, lo:hi].contiguous(), v[:, lo:hi].contiguous(),
                                    fb, fc, nt, want_selection=True)
        outs.append(o)
        bms.append(b)
    torch.cuda.synchronize()
    out, bm = torch.cat(outs, 1), torch.cat(bms, 2)
    assert torch.equal(eng.k_cube, one.k_cube) and torch.equal(eng.v_cube, one.v_cube)
    assert torch.equal(eng.cube_keys, one.cube_keys)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bm, label="chunked")
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    assert torch.equal(bm, bm1), "chunked and one-shot selections differ"
    # Both results are checked against the oracle above / elsewhere.  Against each other they may differ by the
    # bf16 rounding of the probabilities: a later chunk runs its softmax against the running maximum, the
    # one-shot call against a reference fixed in advance, so the two round different numbers.
    assert (out.float() - out1.float()).abs().max().item() <= pu.MAX_ABS_TOL


def test_config2_in_four_chunks_matches_one_shot():
    """Config 2 (the bench workload) prefilled in 4 chunks of 16 frames, text with the last chunk."""
    wl = inputs.config2()
    one, out1, bm1, _ = pu.run_forward(wl)
    eng, out, bm, cnt = run_chunked(wl, [(0, 16), (16, 16), (32, 16), (48, 16)])
    rows = pu.sample_rows(wl, 1200, seed=12, whole_tiles=[(0, 3, 31), (0, 9, 32), (0, 27, 128)])
    rep = pu.compare_rows(wl, rows, out, bm, cnt, label="cfg2 chunked")
    print("cfg2 chunked", rep)
    differ = (bm != bm1).any(-1)
    assert int(differ.sum()) <= 2, f"{int(differ.sum())} rows select differently from the one-shot prefill"
    same = ~differ
    assert (out.float() - out1.float()).abs().permute(0, 2, 1, 3)[same].max().item() <= pu.MAX_ABS_TOL


def test_chunk_argument_errors():
    wl = inputs.small_prefill(seed=92, T=16, H=8, W=8, n_text=5)
    eng = pu.make_engine(wl)
    x = torch.zeros(1, 512, 4, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 512, 2, 128, dtype=torch.bfloat16, device="cuda")
    for fb, fc, nt, code in [(2, 4, -1, binding.ERR_INVALID_ARG),      # not a whole time block
                             (0, 20, -1, binding.ERR_INVALID_ARG),     # beyond the video
                             (0, 8, 3, binding.ERR_INVALID_ARG),       # text before the video is complete
                             (0, 0, -1, binding.ERR_INVALID_ARG)]:     # empty
        with pytest.raises(binding.AdasparkError) as e:
            eng.forward_chunk(x, kv, kv, fb, fc, nt)
        assert e.value.status == code, (fb, fc, nt)
