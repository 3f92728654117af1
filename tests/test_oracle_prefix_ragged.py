"""Pins of the oracle's two extensions of the paper's setting (both readings are listed in the design
notes): video grids the cube window does not divide (boundary cubes hold fewer tokens) and text placed
before the video (always attended in full, never a candidate of Eq. 1).  Every check compares the oracle
with something it does not compute itself: numpy reshapes of a padded grid, an independently written
dense causal attention, one-hot values that expose the attended key set, and the same workload without
the extension."""
import numpy as np
import pytest

import oracle
from paper_2604_08077_b200 import inputs


def dense_causal(q, k, v, order, scale):
    """Textbook causal softmax attention over the tokens listed in `order` (numpy, fp64): token
    order[i] attends order[0..i].  q [S,D], k/v [S,D] of one head.  Returns [S,D] indexed by token."""
    out = np.zeros((len(order), v.shape[1]))
    kk, vv = k[order].astype(np.float64), v[order].astype(np.float64)
    for i, n in enumerate(order):
        s = kk[:i + 1] @ q[n].astype(np.float64) * scale
        w = np.exp(s - s.max())
        out[n] = (w / w.sum()) @ vv[:i + 1]
    return out


def padded_grid_positions(T, H, W, cube):
    """raster token of every (cube, rank) slot from a numpy reshape of the padded index grid (-1 = no token)."""
    ct, ch, cw = cube
    nT, nH, nW = -(-T // ct), -(-H // ch), -(-W // cw)
    grid = np.full((nT * ct, nH * ch, nW * cw), -1, np.int64)
    grid[:T, :H, :W] = np.arange(T * H * W).reshape(T, H, W)
    return grid.reshape(nT, ct, nH, ch, nW, cw).transpose(0, 2, 4, 1, 3, 5).reshape(nT * nH * nW, ct * ch * cw)


RAGGED = dict(T=5, H=6, W=7, cube=(2, 4, 4))          # 3 x 2 x 2 = 12 cubes of 32 slots, 210 tokens


def test_ragged_positions_hand_example_and_numpy_reshape():
    sh = oracle.make_shape(B=1, T=3, H=2, W=3, cube=(2, 2, 2), n_text=2, Hq=1, Hkv=1, D=8, top_p=0.9, n_prefix=3)
    assert sh.N == 4 and sh.C == 8 and sh.S == 3 + 18 + 2 and sh.n_positions == 3 + 32 + 2
    lib = oracle.lib()
    import ctypes
    pos_of = lambda n: lib.adas_oracle_position(ctypes.byref(sh), n)
    assert pos_of(0) == 0 and pos_of(2) == 2                         # prefix keeps its place
    # video token (t=2, y=1, x=2) = raster 2*6 + 1*3 + 2 = 17: cube (1*1 + 0)*2 + 1 = 3, rank (0*2 + 1)*2 + 0 = 2
    assert pos_of(3 + 17) == 3 + 3 * 8 + 2
    assert pos_of(3 + 18) == 3 + 32 and pos_of(3 + 19) == 3 + 33     # text after the N*C slots
    for kw, n_prefix, n_text in [(RAGGED, 0, 0), (RAGGED, 5, 3), (dict(T=4, H=4, W=4, cube=(2, 2, 2)), 2, 1)]:
        sh = oracle.make_shape(B=1, **kw, n_text=n_text, Hq=1, Hkv=1, D=8, top_p=0.9, n_prefix=n_prefix)
        pos, inv = oracle.positions(sh)
        slots = padded_grid_positions(kw["T"], kw["H"], kw["W"], kw["cube"]).reshape(-1)
        expect = np.concatenate([np.arange(n_prefix), np.where(slots >= 0, slots + n_prefix, -1),
                                 n_prefix + sh.S_v + np.arange(n_text)])
        assert np.array_equal(inv, expect)
        assert np.array_equal(inv[pos], np.arange(sh.S))             # a bijection onto the filled slots


def test_ragged_mean_keys_equal_numpy_masked_mean():
    wl = inputs.make_prefill("r", seed=5, B=2, **RAGGED, n_text=4, Hq=2, Hkv=2, D=16, top_p=0.9, offset_std=1.0, n_prefix=3)
    sh = oracle.shape_of(wl)
    kbar = oracle.mean_keys(sh, wl.k)
    slots = padded_grid_positions(wl.T, wl.H, wl.W, wl.cube)                       # [N, C]
    kv = wl.k[:, wl.n_prefix:wl.n_prefix + wl.S_v].double().numpy()                 # [B, S_v, Hkv, D]
    for c in range(sh.N):
        held = slots[c][slots[c] >= 0]
        assert 0 < len(held) <= sh.C
        np.testing.assert_allclose(kbar[:, :, c], kv[:, held].mean(axis=1), rtol=0, atol=1e-15)
    assert (np.array([np.sum(s_ >= 0) for s_ in slots]) < sh.C).any()              # some cube really is cut


@pytest.mark.parametrize("n_prefix,ragged", [(0, True), (7, False), (5, True)])
def test_p1_is_dense_causal_attention_in_position_order(n_prefix, ragged):
    kw = RAGGED if ragged else dict(T=4, H=4, W=8, cube=(2, 4, 4))
    wl = inputs.make_prefill("d", seed=6, B=1, **kw, n_text=6, Hq=2, Hkv=1, D=16, top_p=1.0, offset_std=1.5, n_prefix=n_prefix)
    sh = oracle.shape_of(wl)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, oracle.all_rows(sh))
    pos, _ = oracle.positions(sh)
    order = np.argsort(pos)
    q, k, v = (oracle.as_f32(t)[0] for t in (wl.q, wl.k, wl.v))
    for h in range(wl.Hq):
        ref = dense_causal(q[:, h], k[:, 0], v[:, 0], order, sh.scale)
        np.testing.assert_allclose(res["out"].reshape(wl.Hq, wl.S, wl.D)[h], ref, rtol=0, atol=1e-12)
    assert np.array_equal(res["n_attended"].reshape(wl.Hq, wl.S)[0], np.argsort(order) + 1)


def test_one_hot_values_expose_the_attended_tokens():
    """V = one-hot of the token index: the output row is the attention weight per token, so its support is
    the attended set.  Video row: the whole prefix, the tokens its selected cubes hold (not their empty
    slots), its own cube up to itself.  Text row: prefix, selected cubes, text up to itself.  Prefix row:
    the prefix up to itself."""
    wl = inputs.make_prefill("h", seed=7, B=1, **RAGGED, n_text=5, Hq=1, Hkv=1, D=16, top_p=0.6, offset_std=2.0, n_prefix=4)
    sh0 = oracle.shape_of(wl)
    S = wl.S
    sh = oracle.make_shape(B=1, T=wl.T, H=wl.H, W=wl.W, cube=wl.cube, n_text=wl.n_text, Hq=1, Hkv=1, D=S, top_p=0.6,
                           scale=sh0.scale, n_prefix=wl.n_prefix)
    # selection from the real q, k (D = 16); attention weights with one-hot values need D = S: evaluate Eq. 3
    # with the planted selection on tensors whose q.k products equal the real ones
    base = oracle.rows(sh0, wl.q, wl.k, wl.v, oracle.all_rows(sh0))
    qf, kf = oracle.as_f32(wl.q), oracle.as_f32(wl.k)
    pad = lambda a: np.concatenate([a, np.zeros(a.shape[:-1] + (S - 16,), np.float32)], axis=-1)
    v1 = np.eye(S, dtype=np.float32)[None, :, None, :]
    w = oracle.attend_given(sh, pad(qf), pad(kf), v1, oracle.all_rows(sh), base["sel"])      # [S, S] weights
    pos, inv = oracle.positions(sh0)
    slots = padded_grid_positions(wl.T, wl.H, wl.W, wl.cube)
    P0, Sv = wl.n_prefix, wl.S_v
    saw_cut_cube = False
    for n in range(S):
        expect = set()
        if n < P0:
            expect = set(range(n + 1))
        else:
            expect |= set(range(P0))
            for c in np.flatnonzero(base["sel"][n]):
                held = slots[c][slots[c] >= 0]
                saw_cut_cube |= len(held) < sh0.C
                expect |= set((held + P0).tolist())
            if n < P0 + Sv:
                c_own = (pos[n] - P0) // sh0.C
                own = slots[c_own]
                expect |= set(int(t) + P0 for t in own[own >= 0] if pos[t + P0] <= pos[n])
            else:
                expect |= set(range(P0 + Sv, n + 1))
        assert set(np.flatnonzero(w[n] > 0).tolist()) == expect, n
        np.testing.assert_allclose(w[n].sum(), 1.0, atol=1e-12)
        assert base["n_attended"][n] == len(expect)
    assert saw_cut_cube


def test_prefix_is_outside_the_cube_softmax():
    """Adding a prefix changes no selection: the video and text part of the workload is the same tensor
    with and without it (the generator draws the prefix last), and Eq. 1 runs over cubes only."""
    kw = dict(seed=8, B=1, T=8, H=8, W=8, cube=(2, 4, 4), n_text=9, Hq=2, Hkv=1, D=32, top_p=0.7, offset_std=1.5)
    a = inputs.make_prefill("a", **kw)
    b = inputs.make_prefill("b", **kw, n_prefix=11)
    assert np.array_equal(oracle.as_f32(a.k), oracle.as_f32(b.k)[:, 11:])
    ra = oracle.rows(oracle.shape_of(a), a.q, a.k, a.v, oracle.all_rows(oracle.shape_of(a)), attend=False)
    rb = oracle.rows(oracle.shape_of(b), b.q, b.k, b.v, oracle.all_rows(oracle.shape_of(b)), attend=False)
    selb = rb["sel"].reshape(2, b.S, -1)
    assert not selb[:, :11].any()                                     # prefix rows have no candidates
    assert np.array_equal(selb[:, 11:].reshape(-1, selb.shape[-1]), ra["sel"])
    assert np.array_equal(rb["n_attended"].reshape(2, b.S)[:, 11:].reshape(-1), ra["n_attended"] + 11)
