"""GPU parity of the query-gather path of the prefill (Eq. 3 over the selected cubes alone: per key block the
rows that selected it are gathered, partial results are merged with the result of the row's local range).
The path is forced for every pair of query tiles, then every row is compared with the CPU oracle exactly as
for the union path; the decision rule, the capacity fallback and the agreement of the two paths are tested
apart."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import binding, inputs

import parity_util as pu
from test_gpu_prefill import SMALL_CASES
from test_gpu_prefix_ragged import CASES as OPEN_CASES

pytestmark = pytest.mark.gpu


def expected_entries(wl, bitmap):
    """(row, 64-key block) entries the path must produce when forced: for every row the key blocks before
    the local range of its 256-row pair that hold a cube it selected.  Pure index arithmetic on the
    selection the library reported (which the caller compares with the oracle)."""
    sh = oracle.shape_of(wl)
    pos_of, _ = oracle.positions(sh)                        # oracle position of every token
    C, N, P0 = sh.C, sh.N, sh.n_prefix
    S_v = N * C
    sel = pu.unpack_bitmap(bitmap, N)                       # [B, Hq, S, N]
    total = 0
    for s in range(wl.S):
        p = int(pos_of[s])
        # cube-major position in the caches: video slots first, then prefix, then text
        if P0 <= p < P0 + S_v:
            cpos = p - P0
        elif p < P0:
            cpos = S_v + p
        else:
            cpos = p
        pair_pos0 = cpos // 256 * 256
        local_start = (pair_pos0 // C) * C if pair_pos0 < S_v else S_v
        first_local_blk = local_start // 64
        cube_lim = first_local_blk * 64 // C
        rows = sel[:, :, s, :cube_lim]                      # [B, Hq, cube_lim]
        if C >= 64:
            total += int(rows.sum()) * (C // 64)
        else:
            per = 64 // C
            pad = (-cube_lim) % per
            r = np.pad(rows, ((0, 0), (0, 0), (0, pad)))
            total += int(r.reshape(*r.shape[:2], -1, per).any(-1).sum())
    return total


@pytest.mark.parametrize("case", sorted(SMALL_CASES))
def test_forced_gather_every_row(case):
    """Every row of the small problems with all selected cubes before the local range on the gather path."""
    wl = SMALL_CASES[case]()
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    hdr = eng.header()
    assert hdr.status == 0
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label=case)
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    assert hdr.gather_entries == expected_entries(wl, bitmap)
    print(case, rep, "entries", hdr.gather_entries, "items", hdr.gather_items, "pairs", hdr.gather_pair_tiles)


@pytest.mark.parametrize("case", sorted(OPEN_CASES))
def test_forced_gather_prefix_and_ragged(case):
    """Text prefix (attended by the union kernel's local part) and ragged grids (empty slots masked in the
    gathered blocks)."""
    wl = OPEN_CASES[case]()
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    hdr = eng.header()
    assert hdr.status == 0
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label=case)
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    assert hdr.gather_entries == expected_entries(wl, bitmap)
    print(case, rep, "entries", hdr.gather_entries)


def test_paths_agree_and_off_switch():
    """Threshold 0 switches the path off (no entries); both paths select the same cubes bit for bit and their
    outputs differ by bf16 rounding of the partial results only."""
    wl = inputs.small_prefill(seed=31, T=24, H=8, W=8, n_text=50, Hq=4, Hkv=2, top_p=0.6, offset_std=3.0)
    e0, out0, bm0, cnt0 = pu.run_forward(wl, prefill_kernel=1, gather=0.0)
    e1, out1, bm1, cnt1 = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    assert e0.header().gather_entries == 0 and e0.header().gather_pair_tiles == 0
    assert e1.header().gather_entries > 0
    assert torch.equal(bm0, bm1) and torch.equal(cnt0, cnt1)
    diff = (out0.float() - out1.float()).abs().max().item()
    assert diff < 2e-2, diff
    # executed work: the gather path computes one 128 x 64 product per item, the union path two per visited
    # block of a pair; with 4-5 cubes kept per row the former must be far below the latter
    assert e1.header().executed_kv_blocks < e0.header().executed_kv_blocks


def test_capacity_fallback():
    """A byte budget too small for the entries sends every pair back to the union path in that call; the
    result is still the oracle's."""
    wl = inputs.small_prefill(seed=32, T=16, H=8, W=8, n_text=20, top_p=0.8)
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER, gather_budget=64 * 280)
    hdr = eng.header()
    assert hdr.status == 0 and hdr.gather_entries == 0 and hdr.gather_pair_tiles == 0
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label="capacity")
    assert rep["rows"] == wl.B * wl.Hq * wl.S


def test_partial_capacity_keeps_the_sparsest_pairs():
    """When the qualifying pairs need more workspace than the budget gives, part of them is gathered -- units of
    (ratio class, row window), sparsest class first -- and the rest take the union path; the result is the
    oracle's either way."""
    wl = inputs.small_prefill(seed=37, T=64, H=8, W=8, n_text=40, Hq=4, Hkv=2, top_p=0.8, offset_std=2.5)
    full, out_f, bm_f, cnt_f = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    n_all, pairs_all = full.header().gather_entries, full.header().gather_pair_tiles
    assert n_all > 0
    # FORCE puts every pair into one class; a finite threshold above the break-even estimate still forces the
    # path and spreads the pairs over the ratio classes.  Which threshold splits this workload is found by trying.
    found = None
    for thr in (50.0, 70.0, 100.0, 140.0, 200.0, 280.0, 400.0):
        ref, _, _, _ = pu.run_forward(wl, prefill_kernel=1, gather=thr)
        n_thr, pairs_thr = ref.header().gather_entries, ref.header().gather_pair_tiles
        if n_thr == 0:
            continue
        part, out_p, bm_p, cnt_p = pu.run_forward(wl, prefill_kernel=1, gather=thr,
                                                  gather_budget=(n_thr * 3 // 4) * (2 * wl.D + 24))
        hp = part.header()
        assert hp.status == 0 and hp.gather_entries <= n_thr * 3 // 4
        if 0 < hp.gather_entries and 0 < hp.gather_pair_tiles < pairs_thr:
            found = (thr, n_thr, pairs_thr, hp.gather_entries, hp.gather_pair_tiles)
            rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out_p, bm_p, cnt_p, label="partial capacity")
            assert rep["rows"] == wl.B * wl.Hq * wl.S
            break
    assert found is not None, "no threshold split the pairs of this workload over several classes"
    print("partial capacity (threshold, entries, pairs, kept entries, kept pairs)", found)


def test_decision_rule_per_pair():
    """With a finite threshold only the pairs whose rows' entries are at most threshold x union blocks take the
    path: a sharp selection (few cubes per row, different per row) qualifies, a flat one does not."""
    sharp = inputs.small_prefill(seed=33, T=256, H=8, W=8, n_text=0, Hq=4, Hkv=2, top_p=0.3, offset_std=4.0)
    flat = inputs.small_prefill(seed=34, T=256, H=8, W=8, n_text=0, Hq=4, Hkv=2, top_p=0.95, offset_std=0.3)
    for wl, expect_on in ((sharp, True), (flat, False)):
        eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=20.0)
        hdr = eng.header()
        assert hdr.status == 0
        assert (hdr.gather_pair_tiles > 0) == expect_on, (hdr.gather_pair_tiles, hdr.gather_entries)
        rep = pu.compare_rows(wl, pu.random_rows(wl, 1500, seed=5), out, bitmap, count, label="rule")
        print("sharp" if expect_on else "flat", rep, hdr.gather_pair_tiles, hdr.gather_entries)


def test_small_gains_stay_on_the_union_path():
    """The same sharp selection on a problem so small that gathering cannot repay its fixed cost: with a threshold
    inside the library's break-even estimate nothing is gathered; forcing (a threshold above it) still gathers."""
    wl = inputs.small_prefill(seed=33, T=32, H=8, W=8, n_text=0, Hq=2, Hkv=1, top_p=0.3, offset_std=4.0)
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=20.0)
    assert eng.header().status == 0 and eng.header().gather_entries == 0
    pu.compare_rows(wl, pu.random_rows(wl, 500, seed=6), out, bitmap, count, label="small gain")
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    assert eng.header().status == 0 and eng.header().gather_entries > 0


def test_set_gather_arguments():
    wl = inputs.small_prefill(seed=35)
    eng = pu.make_engine(wl, gather=20.0, gather_budget=1 << 30)
    with pytest.raises(binding.AdasparkError):
        binding.adaspark_attn_set_gather(eng.handle, -1.0, 1 << 30)
    with pytest.raises(binding.AdasparkError):           # the budget sizes the workspace: not after partition
        binding.adaspark_attn_set_gather(eng.handle, 20.0, 2 << 30)
    binding.adaspark_attn_set_gather(eng.handle, 5.0, 1 << 30)   # the threshold alone may change


def test_forced_gather_chunked_prefill():
    """Chunks of a chunked prefill gather from the caches the earlier chunks built."""
    wl = inputs.small_prefill(seed=36, T=32, H=8, W=8, n_text=23, Hq=4, Hkv=2, D=128, top_p=0.7, offset_std=2.5)
    eng = pu.make_engine(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    q, k, v = wl.q.cuda(), wl.k.cuda(), wl.v.cuda()
    hw = wl.H * wl.W
    outs, bms, cnts, entries = [], [], [], 0
    for fb, fc, nt in [(0, 8, -1), (8, 16, -1), (24, 8, wl.n_text)]:
        lo, hi = fb * hw, (fb + fc) * hw + max(nt, 0)
        o, b, c = eng.forward_chunk(q[:, lo:hi].contiguous(), k[:, lo:hi].contiguous(), v[:, lo:hi].contiguous(),
                                    fb, fc, nt, want_selection=True)
        torch.cuda.synchronize()
        assert eng.header().status == 0
        entries += eng.header().gather_entries
        outs.append(o); bms.append(b); cnts.append(c)
    out, bm, cnt = torch.cat(outs, 1), torch.cat(bms, 2), torch.cat(cnts, 2)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bm, cnt, label="chunked")
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    assert entries == expected_entries(wl, bm)


def test_default_rule_head_dim_64_two_row_windows():
    """A 32768-token video with head_dim 64, batch 2 and a sharp selection: the library's own rule sends it
    through the path (several row windows, 16-token cubes: four cubes per key block), sampled rows and two
    whole query tiles against the oracle."""
    wl = inputs.make_prefill("gather_d64", seed=41, B=2, T=128, H=16, W=16, cube=(1, 4, 4), n_text=70, Hq=8,
                             Hkv=2, D=64, top_p=0.4, offset_std=3.0)
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1)
    hdr = eng.header()
    n_pairs = wl.B * wl.Hq * ((wl.S + 255) // 256)
    assert hdr.status == 0 and hdr.gather_pair_tiles > 0.5 * n_pairs, (hdr.gather_pair_tiles, n_pairs)
    n_tiles = (wl.S + 127) // 128
    rows = pu.sample_rows(wl, 1200, seed=9, whole_tiles=[(1, 5, n_tiles // 2), (0, 2, n_tiles - 1)])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label="gather d64")
    print("gather d64", rep, hdr.gather_pair_tiles, "of", n_pairs, "pairs,", hdr.gather_entries, "entries")


def test_forced_gather_top_k_tiny_p_and_wide_gqa_group():
    """The path only consumes the selection masks: the Top-K rule, p -> 0 (the argmax cube alone) and a GQA
    group of 16 query heads (the widest the library takes: 4 bits of head index in an entry) go through it
    unchanged."""
    wl = inputs.small_prefill(seed=42, T=16, H=8, W=8, n_text=19, Hq=4, Hkv=2, top_p=0.9, offset_std=2.0)
    wl.top_k = 3
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    assert eng.header().status == 0 and eng.header().gather_entries == expected_entries(wl, bitmap)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label="top-k gather")
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    wl = inputs.small_prefill(seed=43, T=16, H=8, W=8, n_text=19, Hq=4, Hkv=2, top_p=1e-6)
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    assert eng.header().status == 0 and eng.header().gather_entries == expected_entries(wl, bitmap)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label="argmax gather")
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    wl = inputs.small_prefill(seed=44, T=16, H=8, W=8, n_text=9, Hq=16, Hkv=1, D=64, top_p=0.7, offset_std=2.5)
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=1, gather=pu.FORCE_GATHER)
    assert eng.header().status == 0 and eng.header().gather_entries == expected_entries(wl, bitmap)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label="gqa16 gather")
    assert rep["rows"] == wl.B * wl.Hq * wl.S
