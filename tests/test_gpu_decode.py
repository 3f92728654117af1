"""GPU parity of the decode step (append, score+select, split-KV attention, combine) against the
CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import inputs

import parity_util as pu

pytestmark = pytest.mark.gpu


def run_decode(wl, text_len, *, top_p=None, n_text_max=None, append=True):
    eng = pu.make_engine(wl, n_text_max=n_text_max, top_p=top_p)
    k, v = wl.k.cuda(), wl.v.cuda()
    eng.forward(None, k, v, wl.n_text)                    # build the caches only
    tl = torch.tensor(text_len, dtype=torch.int32, device="cuda")
    if append:
        out, bitmap = eng.decode(wl.q_new.cuda(), wl.k_new.cuda(), wl.v_new.cuda(), tl,
                                 want_selection=True)
    else:
        out, bitmap = eng.decode(wl.q_new.cuda(), None, None, tl, want_selection=True)
    torch.cuda.synchronize()
    return eng, out, bitmap


def compare_decode(wl, text_len, out, bitmap, *, top_p=None, batch_index=None, label=""):
    """Decode step vs the oracle, one row per (sequence, head).  Selection: bit-exact outside the
    1e-6 tie margin; a row inside it may differ only as a legal nucleus (few of them, see
    parity_util.check_selection).  Outputs: every row, a legally differing row against the oracle's
    attention on the GPU's own set."""
    sh = pu.oracle_shape(wl, top_p)
    res = oracle.decode(sh, wl.k, wl.v, text_len, wl.q_new, wl.k_new, wl.v_new,
                        batch_index=batch_index)
    idx = list(range(wl.B)) if batch_index is None else list(batch_index)
    got_sel = pu.unpack_bitmap(bitmap, sh.N)[idx]                     # [n_seq, Hq, N]
    got = out[idx, 0].float().cpu().numpy()
    same = (got_sel == res["sel"]).all(axis=-1)
    near = res["margin"] < pu.TIE_MARGIN
    bad = ~same & ~near
    assert not bad.any(), f"{label}: selection differs on rows {np.argwhere(bad)[:5].tolist()}"
    n_diff = int((~same).sum())
    assert n_diff <= max(2, int(0.05 * near.sum())), f"{label}: {n_diff} differing rows of {int(near.sum())} near ties"
    ref = res["out"].copy()
    G = sh.Hq // sh.Hkv
    kf, qf = oracle.as_f32(wl.k), oracle.as_f32(wl.q_new)
    for i, h in np.argwhere(~same):
        b = idx[i]
        tl = int(text_len[b])
        s1 = oracle.Shape(1, sh.T, sh.H, sh.W, sh.ct, sh.ch, sh.cw, tl + 1, sh.Hq, sh.Hkv, sh.D, sh.top_p,
                          sh.scale, sh.top_k)
        k1 = np.concatenate([kf[b, :sh.S_v + tl], oracle.as_f32(wl.k_new)[b]], axis=0)[None]
        v1 = np.concatenate([oracle.as_f32(wl.v)[b, :sh.S_v + tl], oracle.as_f32(wl.v_new)[b]], axis=0)[None]
        q1 = np.zeros((1, sh.S_v + tl + 1, sh.Hq, sh.D), np.float32)
        q1[0, -1] = qf[b, 0]
        kbar = oracle.mean_keys(s1, k1)
        _, probs, _ = oracle.select_row(q1[0, -1, h], kbar[0, h // G], sh.N, sh.scale, sh.top_p, sh.top_k)
        why = pu.check_nucleus_legal(probs, res["sel"][i, h], got_sel[i, h], sh.top_p, sh.top_k)
        assert why is None, f"{label}: sequence {b} head {h} differs illegally: {why}"
        ref[i, h] = oracle.attend_given(s1, q1, k1, v1, [(0, h, sh.S_v + tl)], got_sel[i, h][None])[0]
    max_abs = float(np.abs(got - ref).max())
    mean_rel = float(np.abs(got - ref).mean() / np.abs(ref).mean())
    assert max_abs <= pu.MAX_ABS_TOL and mean_rel <= pu.MEAN_REL_TOL, (label, max_abs, mean_rel)
    return {"rows": int(same.size), "differing": n_diff, "near_tie": int(near.sum()), "max_abs": max_abs,
            "mean_rel": mean_rel, "mean_selected": float(res["count"].mean())}


@pytest.mark.parametrize("case", ["d128_c64", "d64_c32", "c256", "c16_straddle"])
def test_small_decode(case):
    kw = {"d128_c64": dict(),
          "d64_c32": dict(T=8, H=8, W=8, cube=(2, 4, 4), n_text=64, Hq=4, Hkv=4, D=64, top_p=0.7),
          "c256": dict(T=8, H=16, W=16, cube=(4, 8, 8), n_text=10, Hq=16, Hkv=1, D=128),
          "c16_straddle": dict(T=2, H=4, W=12, cube=(1, 4, 4), n_text=70, Hq=6, Hkv=2, D=64)}[case]
    wl = inputs.small_decode(seed=40, **kw)
    text_len = [wl.n_text - 3 * b for b in range(wl.B)]      # different lengths per sequence
    eng, out, bitmap = run_decode(wl, text_len)
    print(case, compare_decode(wl, text_len, out, bitmap, label=case))
    # the appended token landed in the caches
    for b in range(wl.B):
        pos = wl.S_v + text_len[b]
        assert torch.equal(eng.k_cube[b, :, pos].cpu(), wl.k_new[b, 0])
        assert torch.equal(eng.v_cube[b, :, pos // 64, :, pos % 64].cpu(), wl.v_new[b, 0])


def test_decode_largest_gqa_group_and_cube_count():
    """16 query heads per KV head (the largest group the library takes) over 4096 cubes."""
    wl = inputs.small_decode(seed=44, B=2, T=256, H=16, W=16, cube=(1, 4, 4), n_text=9, Hq=16, Hkv=1, D=64,
                             top_p=0.85)
    assert wl.N == 4096
    text_len = [9, 2]
    eng, out, bitmap = run_decode(wl, text_len)
    print(compare_decode(wl, text_len, out, bitmap, label="g16_n4096"))


def test_decode_without_append_uses_the_cached_token():
    wl = inputs.small_decode(seed=41)
    text_len = [wl.n_text, wl.n_text - 1]
    eng, out1, bm1 = run_decode(wl, text_len, n_text_max=wl.n_text + 4)
    tl = torch.tensor(text_len, dtype=torch.int32, device="cuda")
    out2, bm2 = eng.decode(wl.q_new.cuda(), None, None, tl, want_selection=True)
    torch.cuda.synchronize()
    assert torch.equal(out1, out2) and torch.equal(bm1, bm2)


def test_decode_zero_text_and_dense_p():
    wl = inputs.small_decode(seed=42, n_text=0)
    eng, out, bitmap = run_decode(wl, [0, 0], top_p=1.0, n_text_max=8)
    rep = compare_decode(wl, [0, 0], out, bitmap, top_p=1.0, label="p=1")
    assert pu.unpack_bitmap(bitmap, wl.N).all()
    print(rep)


def test_decode_matches_prefill_last_row():
    """A decode step equals the last text row of a prefill over the appended sequence."""
    wl = inputs.small_decode(seed=43, B=1, n_text=21)
    eng, out, bitmap = run_decode(wl, [wl.n_text])
    full = inputs.Workload(name="appended", B=1, T=wl.T, H=wl.H, W=wl.W, cube=wl.cube,
                           n_text=wl.n_text + 1, Hq=wl.Hq, Hkv=wl.Hkv, D=wl.D, top_p=wl.top_p,
                           q=torch.cat([torch.zeros(1, wl.S, wl.Hq, wl.D, dtype=torch.bfloat16), wl.q_new], 1),
                           k=torch.cat([wl.k, wl.k_new], 1), v=torch.cat([wl.v, wl.v_new], 1))
    _, out_p, bitmap_p, _ = pu.run_forward(full)
    assert torch.equal(bitmap_p[0, :, -1], bitmap[0])
    np.testing.assert_allclose(out[0, 0].float().cpu().numpy(), out_p[0, -1].float().cpu().numpy(),
                               atol=1e-2)


def test_config5_shape_reduced_batch():
    """Config-5 geometry (131072-token video cache, 2048 cubes, 512 text) at batch 2; the oracle
    evaluates every (sequence, head) row."""
    wl = inputs.config5(B=2)
    text_len = [512, 300]
    eng, out, bitmap = run_decode(wl, text_len)
    rep = compare_decode(wl, text_len, out, bitmap, label="cfg5")
    print("cfg5", rep)


@pytest.mark.parametrize("append", [True, False])
def test_text_len_outside_the_partition_is_reported(append):
    """text_len[b] < 0 or > n_text_max: header status 1, a zero output row for that sequence, the
    cache untouched -- with and without an appended token; the other sequence is unaffected."""
    wl = inputs.small_decode(seed=45, B=3, n_text=20)
    n_text_max = wl.n_text + 2
    good = wl.n_text
    text_len = [-1, good, n_text_max + 1]
    eng = pu.make_engine(wl, n_text_max=n_text_max)
    eng.forward(None, wl.k.cuda(), wl.v.cuda(), wl.n_text)
    torch.cuda.synchronize()
    k_before = eng.k_cube.clone()
    tl = torch.tensor(text_len, dtype=torch.int32, device="cuda")
    if append:
        out, bitmap = eng.decode(wl.q_new.cuda(), wl.k_new.cuda(), wl.v_new.cuda(), tl, want_selection=True)
    else:
        # store the middle sequence's token by hand, as a caller that keeps its own cache would
        pos = wl.S_v + good
        eng.k_cube[1, :, pos] = wl.k_new[1, 0].cuda()
        eng.v_cube[1, :, pos // 64, :, pos % 64] = wl.v_new[1, 0].cuda()
        k_before = eng.k_cube.clone()
        out, bitmap = eng.decode(wl.q_new.cuda(), None, None, tl, want_selection=True)
    torch.cuda.synchronize()
    assert eng.header().status == 1
    assert (out[0] == 0).all() and (out[2] == 0).all()
    changed = (eng.k_cube != k_before).flatten(2).any(-1).any(-1)        # per sequence
    assert changed.tolist() == [False, append, False]
    rep = compare_decode(wl, text_len, out, bitmap, batch_index=[1], label="valid sequence beside bad ones")
    assert rep["rows"] == wl.Hq
