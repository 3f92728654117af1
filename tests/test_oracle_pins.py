"""Pins for the CPU oracle: everything here is checked against something other than the oracle
itself (closed forms, numpy reshapes, brute force, an independently written dense attention,
torch's fp64 SDPA).  CPU only."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ O1: cube partition
def ref_raster_of_pos(T, H, W, cube, n_text):
    """Cube-major order by reshaping the raster grid (no index formula)."""
    ct, ch, cw = cube
    grid = np.arange(T * H * W).reshape(T // ct, ct, H // ch, ch, W // cw, cw)
    video = grid.transpose(0, 2, 4, 1, 3, 5).reshape(-1)
    return np.concatenate([video, T * H * W + np.arange(n_text)])


def test_partition_hand_example():
    # 2 frames of 2x4 patches, cube 1x2x2: frame 0 = cubes 0,1; frame 1 = cubes 2,3.
    # raster (t,y,x): token 0..7 frame 0 (row 0: 0-3, row 1: 4-7); token 8..15 frame 1.
    sh = oracle.make_shape(B=1, T=2, H=2, W=4, cube=(1, 2, 2), n_text=2, Hq=1, Hkv=1, D=4,
                           top_p=0.9)
    pos, inv = oracle.positions(sh)
    assert sh.N == 4 and sh.C == 4
    # cube 0 = tokens {0,1,4,5}, cube 1 = {2,3,6,7}, cube 2 = {8,9,12,13}, cube 3 = {10,11,14,15}
    assert inv.tolist() == [0, 1, 4, 5, 2, 3, 6, 7, 8, 9, 12, 13, 10, 11, 14, 15, 16, 17]
    assert pos.tolist() == [0, 1, 4, 5, 2, 3, 6, 7, 8, 9, 12, 13, 10, 11, 14, 15, 16, 17]


@pytest.mark.parametrize("T,H,W,cube,n_text,N", [
    (8, 8, 8, (2, 4, 4), 32, 16), (64, 16, 16, (4, 4, 4), 128, 256),
    (256, 16, 16, (4, 4, 4), 256, 1024), (512, 16, 16, (4, 4, 4), 0, 2048),
    (4, 8, 16, (4, 8, 8), 3, 2), (6, 4, 6, (3, 2, 1), 0, 24)])
def test_partition_matches_reshape_and_counts(T, H, W, cube, n_text, N):
    sh = oracle.make_shape(B=1, T=T, H=H, W=W, cube=cube, n_text=n_text, Hq=1, Hkv=1, D=4,
                           top_p=0.9)
    assert sh.N == N
    pos, inv = oracle.positions(sh)
    ref_inv = ref_raster_of_pos(T, H, W, cube, n_text)
    assert np.array_equal(inv, ref_inv)
    assert np.array_equal(np.sort(pos), np.arange(T * H * W + n_text))  # bijection
    assert np.array_equal(inv[pos], np.arange(T * H * W + n_text))      # round trip


# ------------------------------------------------------------------ O2: mean keys
def test_mean_keys_match_numpy_reshape_mean():
    wl = inputs.make_prefill("t", seed=3, B=2, T=4, H=4, W=8, cube=(2, 2, 4), n_text=5, Hq=4,
                             Hkv=2, D=16, top_p=0.9, offset_std=1.5)
    sh = oracle.shape_of(wl)
    kbar = oracle.mean_keys(sh, wl.k)
    k = wl.k.double().numpy()[:, :wl.S_v].reshape(2, 2, 2, 2, 2, 2, 4, 2, 16)
    ref = k.mean(axis=(2, 4, 6)).reshape(2, sh.N, 2, 16).transpose(0, 2, 1, 3)
    assert kbar.shape == (2, 2, sh.N, 16)
    np.testing.assert_allclose(kbar, ref, rtol=0, atol=1e-14)
    # sum of <= 64 bf16 values and a power-of-two divide are exact in fp64
    assert np.array_equal(kbar, ref)


# ------------------------------------------------------------------ O3 + O4: selection
def load_closed_form_cases():
    cases = []
    with open(os.path.join(GOLDEN, "topp_closed_form.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w, p, exp = [x.strip() for x in line.split("|")]
            cases.append(([float(x) for x in w.split(",")], float(p),
                          [int(x) for x in exp.split(",")]))
    return cases


@pytest.mark.parametrize("w,p,expected", load_closed_form_cases())
def test_selection_closed_form(w, p, expected):
    q = np.array([2, 0, 0, 0], np.float32)
    kbar = np.zeros((len(w), 4))
    kbar[:, 0] = np.log(w)
    sel, probs, _ = oracle.select_row(q, kbar, len(w), 0.5, p)
    np.testing.assert_allclose(probs, np.array(w) / np.sum(w), rtol=1e-14)
    assert np.flatnonzero(sel).tolist() == expected


def brute_force_nucleus(probs, p):
    """All subsets: the least size reaching mass p and, at that size, the largest mass."""
    n = len(probs)
    best_size, best_mass = None, None
    for size in range(1, n + 1):
        masses = [sum(probs[list(c)]) for c in itertools.combinations(range(n), size)]
        if max(masses) >= p:
            best_size, best_mass = size, max(masses)
            break
    return best_size, best_mass


def test_selection_brute_force_all_subsets_config1():
    """Config 1 (<= 16 candidate cubes): no smaller subset reaches p and none of the same size
    has more mass, over an exhaustive enumeration of subsets."""
    wl = inputs.config1()
    sh = oracle.shape_of(wl)
    pos, inv = oracle.positions(sh)
    rng = np.random.default_rng(0)
    # rows spread over the sequence: every cube once for small candidate counts + text rows
    rows = [(0, int(rng.integers(wl.Hq)), int(inv[c * wl.C + int(rng.integers(wl.C))]))
            for c in range(1, 13)]
    rows += [(0, h, wl.S_v + 5 * h) for h in range(2)]          # text rows: 16 candidates
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows, attend=False)
    kbar = res["kbar"]
    q = wl.q.float().numpy()
    for i, (b, h, n) in enumerate(rows):
        n_cand = pos[n] // wl.C if n < wl.S_v else sh.N
        _, probs, _ = oracle.select_row(q[b, n, h], kbar[b, h * wl.Hkv // wl.Hq], n_cand,
                                        sh.scale, wl.top_p)
        size, mass = brute_force_nucleus(probs, wl.top_p)
        sel = res["sel"][i]
        assert sel[n_cand:].sum() == 0
        assert sel.sum() == size == res["count"][i]
        assert abs(probs[sel[:n_cand] > 0].sum() - mass) < 1e-12


def numpy_probs(q, kbar, scale):
    s = (kbar @ q.astype(np.float64)) * scale
    e = np.exp(s - s.max())
    return e / e.sum()


def test_selection_properties_random_rows():
    """softmax sums to one; minimality; mass >= p; p->0 keeps the argmax; p=1 keeps all;
    shifting every logit and permuting cubes act as they must."""
    rng = np.random.default_rng(1)
    D, scale = 32, 1 / np.sqrt(32)
    for trial in range(60):
        n = int(rng.integers(1, 200))
        q = rng.standard_normal(D).astype(np.float32)
        kbar = rng.standard_normal((n, D)) * rng.choice([0.3, 1.0, 3.0])
        p = float(rng.choice([0.3, 0.5, 0.7, 0.9, 0.95, 0.999]))
        sel, probs, margin = oracle.select_row(q, kbar, n, scale, p)
        ref = numpy_probs(q, kbar, scale)
        np.testing.assert_allclose(probs, ref, rtol=1e-12, atol=1e-300)
        assert abs(probs.sum() - 1) < 1e-12
        chosen = np.flatnonzero(sel)
        assert len(chosen) >= 1
        mass = probs[chosen].sum()
        assert mass >= p - 1e-15
        assert mass - probs[chosen].min() < p                      # dropping its smallest fails
        assert probs[chosen].min() >= np.delete(probs, chosen).max(initial=0.0)  # a top prefix
        # independent: sort + cumsum in numpy
        order = np.lexsort((np.arange(n), -probs))
        kstar = int(np.searchsorted(np.cumsum(probs[order]), p, side="left")) + 1
        if margin > 1e-12:
            assert sorted(order[:kstar].tolist()) == chosen.tolist()
        # p -> 0+ and p = 1
        s0, _, _ = oracle.select_row(q, kbar, n, scale, 1e-12)
        assert np.flatnonzero(s0).tolist() == [int(np.argmax(probs))]
        s1, _, m1 = oracle.select_row(q, kbar, n, scale, 1.0)
        assert s1.all() and np.isinf(m1)
        # logit shift (add a common vector u to every key => every logit moves by <q,u>*scale)
        u = rng.standard_normal(D)
        s_shift, _, _ = oracle.select_row(q, kbar + u, n, scale, p)
        if margin > 1e-9:
            assert np.array_equal(s_shift, sel)
        # permuting the cubes permutes the selection
        perm = rng.permutation(n)
        s_perm, _, _ = oracle.select_row(q, kbar[perm], n, scale, p)
        if margin > 1e-9:
            assert np.array_equal(s_perm, sel[perm])
    # no candidates: empty selection
    sel, _, m = oracle.select_row(np.ones(4, np.float32), np.zeros((1, 4)), 0, 0.5, 0.9)
    assert len(sel) == 0 and np.isinf(m)


def test_margin_definition():
    """Tie margin = min(|c_k* - p|, |c_(k*-1) - p|, gap across the cut) on a closed-form row."""
    q = np.array([2, 0, 0, 0], np.float32)
    kbar = np.zeros((4, 4))
    kbar[:, 0] = np.log([8, 4, 2, 2])          # P = .5 .25 .125 .125
    _, _, m = oracle.select_row(q, kbar, 4, 0.5, 0.7)   # cum .5, .75 -> k*=2
    assert abs(m - 0.05) < 1e-12               # |.75-.7| = .05 < |.5-.7| = .2 ; gap .125
    _, _, m = oracle.select_row(q, kbar, 4, 0.5, 0.8)   # cum .875 -> k*=3; gap to next = 0
    assert abs(m) < 1e-15


# ------------------------------------------------------------------ O5: attention
def dense_causal_cube_major(q, k, v, inv, G, scale):
    """Textbook causal softmax attention over the cube-major sequence, written with numpy
    matrices (independent of the oracle's gather loops).  q [S,Hq,D], k/v [S,Hkv,D] raster."""
    S, Hq, D = q.shape
    out = np.zeros((S, Hq, D))
    qp, kp, vp = q[inv].astype(np.float64), k[inv].astype(np.float64), v[inv].astype(np.float64)
    mask = np.tril(np.ones((S, S), bool))
    for h in range(Hq):
        s = (qp[:, h] @ kp[:, h // G].T) * scale
        s[~mask] = -np.inf
        w = np.exp(s - s.max(axis=1, keepdims=True))
        w /= w.sum(axis=1, keepdims=True)
        out[inv, h] = w @ vp[:, h // G]
    return out


def test_p_equal_one_is_dense_causal_attention():
    wl = inputs.make_prefill("t", seed=5, B=1, T=4, H=4, W=4, cube=(2, 2, 2), n_text=9, Hq=4,
                             Hkv=2, D=16, top_p=1.0, offset_std=1.0)
    sh = oracle.shape_of(wl)
    rows = oracle.all_rows(sh)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows)
    _, inv = oracle.positions(sh)
    ref = dense_causal_cube_major(wl.q[0].float().numpy(), wl.k[0].float().numpy(),
                                  wl.v[0].float().numpy(), inv, wl.Hq // wl.Hkv, sh.scale)
    got = res["out"].reshape(wl.Hq, wl.S, wl.D).transpose(1, 0, 2)
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-13)
    # the same through a library routine: torch SDPA in fp64 on the permuted sequence
    inv_t = torch.from_numpy(inv)
    qp = wl.q[0].double()[inv_t].permute(1, 0, 2)[None]
    kp = wl.k[0].double()[inv_t].permute(1, 0, 2).repeat_interleave(wl.Hq // wl.Hkv, 0)[None]
    vp = wl.v[0].double()[inv_t].permute(1, 0, 2).repeat_interleave(wl.Hq // wl.Hkv, 0)[None]
    o = torch.nn.functional.scaled_dot_product_attention(qp, kp, vp, is_causal=True)[0]
    ref2 = np.zeros_like(ref)
    ref2[inv] = o.permute(1, 0, 2).numpy()
    np.testing.assert_allclose(got, ref2, rtol=1e-10, atol=1e-12)


def test_attended_key_set_via_one_hot_values():
    """V[n] = e_n turns the output into the attention weights per raster token: their support
    must be exactly {tokens of selected cubes} + {own-cube prefix | text prefix} and their
    values the softmax of the scaled logits over that set (Eq. 3)."""
    T, H, W, cube, n_text, D = 2, 4, 4, (1, 2, 2), 8, 64
    wl = inputs.make_prefill("t", seed=9, B=1, T=T, H=H, W=W, cube=cube, n_text=n_text, Hq=2,
                             Hkv=1, D=D, top_p=0.6, offset_std=2.0)
    S = wl.S
    assert S <= D
    v = torch.zeros(1, S, 1, D)
    v[0, torch.arange(S), 0, torch.arange(S)] = 1.0
    sh = oracle.shape_of(wl)
    res = oracle.rows(sh, wl.q, wl.k, v, oracle.all_rows(sh))
    inv = ref_raster_of_pos(T, H, W, cube, n_text)
    pos = np.argsort(inv)
    q, k = wl.q[0].double().numpy(), wl.k[0, :, 0].double().numpy()
    saw_sparse = False
    for i, (b, h, n) in enumerate(res["rows"]):
        sel = res["sel"][i]
        attended_pos = [j * wl.C + r for j in np.flatnonzero(sel) for r in range(wl.C)]
        if n < wl.S_v:
            c = pos[n] // wl.C
            assert sel[c:].sum() == 0                      # only preceding cubes are candidates
            attended_pos += list(range(c * wl.C, pos[n] + 1))
            saw_sparse |= 0 < sel.sum() < c
        else:
            attended_pos += list(range(wl.S_v, pos[n] + 1))
        tokens = inv[np.array(attended_pos)]
        assert len(set(tokens.tolist())) == len(tokens) == res["n_attended"][i]
        logits = (k[tokens] @ q[n, h]) * sh.scale
        w = np.exp(logits - logits.max())
        w /= w.sum()
        expect = np.zeros(D)
        expect[tokens] = w
        np.testing.assert_allclose(res["out"][i], expect, rtol=1e-11, atol=1e-15)
    assert saw_sparse


def test_first_cube_is_plain_causal_attention_within_the_cube():
    wl = inputs.config1()
    sh = oracle.shape_of(wl)
    _, inv = oracle.positions(sh)
    rows = [(0, 1, int(inv[r])) for r in range(wl.C)]
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows)
    assert res["count"].sum() == 0 and res["sel"].sum() == 0
    q, k, v = wl.q[0].double().numpy(), wl.k[0].double().numpy(), wl.v[0].double().numpy()
    for r in range(wl.C):
        toks = inv[: r + 1]
        s = (k[toks, 1] @ q[inv[r], 1]) * sh.scale
        w = np.exp(s - s.max())
        w /= w.sum()
        np.testing.assert_allclose(res["out"][r], w @ v[toks, 1], rtol=1e-12, atol=1e-14)


def test_value_linearity_and_given_selection_entry():
    wl = inputs.small_prefill(seed=13, T=4, H=4, W=4, cube=(2, 2, 2), n_text=6, Hq=2, Hkv=1, D=16)
    sh = oracle.shape_of(wl)
    rows = oracle.all_rows(sh)[::7]
    r1 = oracle.rows(sh, wl.q, wl.k, wl.v, rows)
    r2 = oracle.rows(sh, wl.q, wl.k, wl.v * 2, rows)     # exact in bf16
    np.testing.assert_allclose(r2["out"], 2 * r1["out"], rtol=1e-14)
    assert np.array_equal(r1["sel"], r2["sel"])
    given = oracle.attend_given(sh, wl.q, wl.k, wl.v, rows, r1["sel"])
    assert np.array_equal(given, r1["out"])


def test_equal_keys_error_bound():
    """If every key of a cube equals the cube's mean key, the cube softmax is the dense mass per
    cube, so dropping <= 1-p of it moves the output by at most 2(1-p) max|v| (from Eqs. 1, 3)."""
    wl = inputs.make_prefill("t", seed=21, B=1, T=4, H=4, W=8, cube=(2, 2, 2), n_text=0, Hq=2,
                             Hkv=1, D=16, top_p=0.8, offset_std=2.0)
    k = wl.k.float().view(1, 2, 2, 2, 2, 4, 2, 1, 16)
    k = k[:, :, :1, :, :1, :, :1].expand_as(k).reshape(1, wl.S, 1, 16).contiguous()
    sh = oracle.shape_of(wl)
    rows = oracle.all_rows(sh)
    sparse = oracle.rows(sh, wl.q, k, wl.v, rows)["out"]
    dense = oracle.rows(oracle.shape_of(wl, top_p=1.0), wl.q, k, wl.v, rows)["out"]
    bound = 2 * (1 - 0.8) * float(wl.v.float().abs().max())
    assert np.abs(sparse - dense).max() <= bound
    assert np.abs(sparse - dense).max() > 0      # and the selection did drop something


# ------------------------------------------------------------------ O6: decode
def test_decode_is_a_text_row_of_the_appended_sequence():
    wl = inputs.small_decode(seed=4, B=2, T=4, H=4, W=4, cube=(2, 2, 2), n_text=5, Hq=4, Hkv=2,
                             D=16)
    sh = oracle.shape_of(wl)
    cap = 8
    pad = torch.zeros(wl.B, cap - wl.n_text, wl.Hkv, wl.D)
    kc = torch.cat([wl.k.float(), pad], 1)
    vc = torch.cat([wl.v.float(), pad], 1)
    text_len = [5, 3]
    res = oracle.decode(sh, kc, vc, text_len, wl.q_new, wl.k_new, wl.v_new)
    assert res["out"].shape == (2, 4, 16)
    # independent numpy evaluation from the returned selection
    _, inv = oracle.positions(sh)
    for b in range(2):
        ks = torch.cat([wl.k[b, :wl.S_v + text_len[b]].float(), wl.k_new[b].float()]).double().numpy()
        vs = torch.cat([wl.v[b, :wl.S_v + text_len[b]].float(), wl.v_new[b].float()]).double().numpy()
        kbar = oracle.mean_keys(sh, wl.k)[b]
        for h in range(4):
            g = h // 2
            q = wl.q_new[b, 0, h].double().numpy()
            probs = numpy_probs(q, kbar[g], sh.scale)
            order = np.lexsort((np.arange(sh.N), -probs))
            kstar = int(np.searchsorted(np.cumsum(probs[order]), wl.top_p, side="left")) + 1
            chosen = sorted(order[:kstar].tolist())
            assert np.flatnonzero(res["sel"][b, h]).tolist() == chosen
            toks = [int(inv[j * wl.C + r]) for j in chosen for r in range(wl.C)]
            toks += list(range(wl.S_v, wl.S_v + text_len[b] + 1))
            s = (ks[toks, g] @ q) * sh.scale
            w = np.exp(s - s.max())
            w /= w.sum()
            np.testing.assert_allclose(res["out"][b, h], w @ vs[toks, g], rtol=1e-11, atol=1e-14)


# ------------------------------------------------------------------ O4k: Top-K rule
@pytest.mark.parametrize("w,k,expected", [
    ([1, 5, 3, 2], 1, [1]),                 # K = 1 is the argmax cube
    ([1, 5, 3, 2], 2, [1, 2]),
    ([1, 5, 3, 2], 3, [1, 2, 3]),
    ([1, 5, 3, 2], 4, [0, 1, 2, 3]),
    ([1, 5, 3, 2], 9, [0, 1, 2, 3]),        # K beyond the candidate count keeps every candidate
    ([2, 2, 2, 1], 2, [0, 1]),              # equal probabilities: lower cube index first
    ([1, 2, 2, 2], 2, [1, 2]),
])
def test_top_k_closed_form(w, k, expected):
    q = np.array([2, 0, 0, 0], np.float32)
    kbar = np.zeros((len(w), 4))
    kbar[:, 0] = np.log(w)
    sel, probs, _ = oracle.select_row(q, kbar, len(w), 0.5, 0.9, top_k=k)
    np.testing.assert_allclose(probs, np.array(w) / np.sum(w), rtol=1e-14)
    assert np.flatnonzero(sel).tolist() == expected


def test_top_k_brute_force_and_margin():
    """On random rows the Top-K set is the subset of size min(K, n) with the largest total mass
    (checked against every subset of that size), and the margin is the gap to the next cube."""
    rng = np.random.default_rng(3)
    for trial in range(40):
        n, D = int(rng.integers(1, 11)), 8
        k = int(rng.integers(1, 13))
        q = rng.standard_normal(D).astype(np.float32)
        kbar = rng.standard_normal((n, D)) * 2.0
        sel, probs, margin = oracle.select_row(q, kbar, n, 1.0 / np.sqrt(D), 0.9, top_k=k)
        size = min(k, n)
        assert sel.sum() == size
        best = max(sum(probs[list(c)]) for c in itertools.combinations(range(n), size))
        assert abs(probs[sel.astype(bool)].sum() - best) < 1e-15
        srt = np.sort(probs)[::-1]
        if size < n:
            assert abs(margin - (srt[size - 1] - srt[size])) < 1e-15
        else:
            assert np.isinf(margin)


def test_top_k_rows_use_the_rule_inside_the_full_path():
    """oracle.rows with top_k set: every row keeps min(K, candidates) cubes, and the attention over
    them equals attend_given with that selection."""
    wl = inputs.small_prefill(seed=51, T=8, H=8, W=8, n_text=6)
    sh = oracle.shape_of(wl, top_k=3)
    rows = oracle.all_rows(sh)[::7]
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows)
    pos, _ = oracle.positions(sh)
    n_cand = np.where(rows[:, 2] < wl.S_v, pos[rows[:, 2]] // wl.C, wl.N)
    assert np.array_equal(res["count"], np.minimum(n_cand, 3))
    out2 = oracle.attend_given(sh, wl.q, wl.k, wl.v, rows, res["sel"])
    np.testing.assert_allclose(res["out"], out2, rtol=0, atol=1e-15)


def test_chunked_prefill_rows_equal_one_shot_rows():
    """A later chunk never changes an earlier row (Eq. 1: a video query sees only preceding cubes; the
    text follows the video): evaluating the rows of frames [0, T') on the truncated problem gives the
    same selection, bit for bit, and the same outputs as evaluating them on the whole sequence."""
    from paper_2604_08077_b200 import inputs
    wl = inputs.small_prefill(seed=93, T=16, H=8, W=8, n_text=9, Hq=2, Hkv=1, D=64, top_p=0.8)
    full = oracle.shape_of(wl)
    for t_cut in (4, 12):
        s_cut = t_cut * wl.H * wl.W
        part = oracle.make_shape(B=wl.B, T=t_cut, H=wl.H, W=wl.W, cube=wl.cube, n_text=0, Hq=wl.Hq, Hkv=wl.Hkv,
                                 D=wl.D, top_p=wl.top_p)
        rows = [(0, h, n) for h in range(wl.Hq) for n in range(0, s_cut, 7)]
        a = oracle.rows(full, wl.q, wl.k, wl.v, rows)
        b = oracle.rows(part, wl.q[:, :s_cut], wl.k[:, :s_cut], wl.v[:, :s_cut], rows)
        n_part = part.N
        assert np.array_equal(a["sel"][:, :n_part], b["sel"]) and not a["sel"][:, n_part:].any()
        assert np.array_equal(a["count"], b["count"])
        np.testing.assert_allclose(a["out"], b["out"], rtol=0, atol=1e-12)
