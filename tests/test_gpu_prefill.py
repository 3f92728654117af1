"""GPU parity of the prefill path (re-layout, pooling, scoring, selection, attention) against
the CPU oracle, through the C ABI, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu


def check_caches(wl, eng):
    """k_cube / v_cube / cube_keys against the oracle's permutation and mean keys (bit-exact)."""
    sh = oracle.shape_of(wl)
    _, inv = oracle.positions(sh)
    inv_t = torch.from_numpy(inv)
    S, s_cap = wl.S, eng.layout.s_cap
    k_ref = wl.k[:, inv_t].permute(0, 2, 1, 3)                         # [B,Hkv,S,D]
    v_ref = wl.v[:, inv_t].permute(0, 2, 1, 3)
    k_got = eng.k_cube.cpu()
    assert torch.equal(k_got[:, :, :S], k_ref)
    assert (k_got[:, :, S:] == 0).all()
    v_got = eng.v_cube.cpu().permute(0, 1, 2, 4, 3).reshape(wl.B, wl.Hkv, s_cap, wl.D)
    assert torch.equal(v_got[:, :, :S], v_ref)
    assert (v_got[:, :, S:] == 0).all()
    kbar = oracle.mean_keys(sh, wl.k).astype(np.float32)                # one rounding to fp32
    assert np.array_equal(eng.cube_keys.cpu().numpy(), kbar)


SMALL_CASES = {
    "cfg1": lambda: inputs.config1(),
    "d128_c64_ragged_text": lambda: inputs.small_prefill(seed=7),
    "d64_c32_no_text": lambda: inputs.small_prefill(seed=8, T=4, H=8, W=8, cube=(2, 4, 4), n_text=0,
                                                    Hq=2, Hkv=2, D=64, top_p=0.7),
    "c256_gqa4": lambda: inputs.small_prefill(seed=9, T=8, H=16, W=8, cube=(4, 8, 8), n_text=5,
                                              Hq=4, Hkv=1, D=128, top_p=0.8),
    "c16_batch2_odd_cubes": lambda: inputs.small_prefill(seed=10, B=2, T=3, H=4, W=12, cube=(1, 4, 4),
                                                         n_text=130, Hq=2, Hkv=1, D=64, top_p=0.9),
    "single_cube": lambda: inputs.small_prefill(seed=11, T=4, H=4, W=4, cube=(4, 4, 4), n_text=3,
                                                Hq=1, Hkv=1, D=128, top_p=0.9),
    # the paper's cube-size ablation runs from 64 to 1024 tokens per cube; 1x1x64 and 8x8x1 are its
    # temporal-only and spatial-only shapes
    "c1024": lambda: inputs.small_prefill(seed=15, T=16, H=16, W=16, cube=(4, 16, 16), n_text=11, Hq=2,
                                          Hkv=1, D=128, top_p=0.7),
    "c64_temporal_only": lambda: inputs.small_prefill(seed=16, T=128, H=2, W=4, cube=(64, 1, 1), n_text=7,
                                                      Hq=2, Hkv=2, D=64, top_p=0.8),
    "c64_spatial_only": lambda: inputs.small_prefill(seed=17, T=6, H=16, W=8, cube=(1, 8, 8), n_text=0,
                                                     Hq=2, Hkv=1, D=128, top_p=0.9),
    "sharp_scores": lambda: inputs.small_prefill(seed=12, T=16, H=8, W=8, n_text=17, top_p=0.5,
                                                 offset_std=3.0),
    # nucleus boundaries far down the tail of a sharp distribution (many octaves below the maximum)
    "deep_tail": lambda: inputs.small_prefill(seed=13, T=32, H=8, W=8, n_text=9, Hq=2, Hkv=1,
                                              top_p=0.999999, offset_std=4.0),
    "flat_scores": lambda: inputs.small_prefill(seed=14, T=32, H=8, W=8, n_text=9, Hq=2, Hkv=1,
                                                top_p=0.6, offset_std=0.0),
}


@pytest.mark.parametrize("case", sorted(SMALL_CASES))
@pytest.mark.parametrize("kernel", [0, 1])
def test_small_prefill_every_row(case, kernel):
    """Element-by-element parity on every row: caches, selection bitmaps, counts, outputs."""
    wl = SMALL_CASES[case]()
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=kernel)
    check_caches(wl, eng)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label=case)
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    print(case, rep)


@pytest.mark.parametrize("p", [1.0, 1e-6])
def test_degenerate_p(p):
    """p = 1 is dense causal attention over the cube-major order; p -> 0 keeps the argmax cube."""
    wl = inputs.small_prefill(seed=21, T=8, H=8, W=8, n_text=20)
    eng, out, bitmap, count = pu.run_forward(wl, top_p=p)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, top_p=p,
                          label=f"p={p}")
    sel = pu.unpack_bitmap(bitmap, wl.N)
    sh = oracle.shape_of(wl)
    pos, _ = oracle.positions(sh)
    n_cand = np.where(np.arange(wl.S) < wl.S_v, pos // wl.C, wl.N)
    if p >= 1.0:
        assert np.array_equal(sel.sum(-1), np.broadcast_to(n_cand, sel.shape[:-1]))
    else:
        assert np.array_equal(sel.sum(-1), np.broadcast_to(np.minimum(n_cand, 1), sel.shape[:-1]))
    print(rep)


@pytest.mark.parametrize("case", ["cfg1", "d128_c64_ragged_text", "deep_tail"])
def test_tcgen05_attention_with_fp64_scoring(case):
    """Kernel option 2: the tcgen05 attention kernel fed by the fp64 (mma.m8n8k4.f64) scoring kernel."""
    wl = SMALL_CASES[case]()
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=2)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label=case)
    assert rep["rows"] == wl.B * wl.Hq * wl.S


def test_cache_only_forward_builds_the_caches():
    wl = inputs.small_prefill(seed=31)
    eng = pu.make_engine(wl)
    eng.forward(None, wl.k.cuda(), wl.v.cuda(), wl.n_text)
    torch.cuda.synchronize()
    check_caches(wl, eng)


def test_selection_only_outputs_are_optional_and_repeatable():
    wl = inputs.small_prefill(seed=32)
    eng, out1, bitmap, count = pu.run_forward(wl)
    out2, b2, c2 = eng.forward(wl.q.cuda(), wl.k.cuda(), wl.v.cuda(), wl.n_text, want_selection=False)
    torch.cuda.synchronize()
    assert b2 is None and c2 is None
    assert torch.equal(out1, out2)
    assert eng.launches() >= 4


def test_config2_full_size_sampled_rows():
    """Config 2 at full size (the bench workload): selection on a large row sample, outputs on
    a sample that includes whole query tiles (first, middle, text)."""
    wl = inputs.config2()
    eng, out, bitmap, count = pu.run_forward(wl)
    rows = pu.sample_rows(wl, 1500, seed=2, whole_tiles=[(0, 0, 0), (0, 13, 64), (0, 27, 128)])
    rep = pu.compare_rows(wl, rows, out, bitmap, count, label="cfg2")
    print("cfg2", rep)
    # selection only, many more rows
    rep = pu.compare_rows(wl, pu.random_rows(wl, 40000, seed=5), None, bitmap, attend=False, label="cfg2 selection")
    print("cfg2 selection", rep)


def test_two_handles_on_two_streams_do_not_interfere():
    """Two engines with different shapes run interleaved on their own streams (each handle also owns
    a private side stream): the results equal those of running them one after the other."""
    wa = inputs.small_prefill(seed=71, T=16, H=8, W=8, n_text=13)
    wb = inputs.small_prefill(seed=72, T=8, H=16, W=8, cube=(2, 4, 4), n_text=40, Hq=6, Hkv=2, D=64, top_p=0.7)
    ea, oa, _, _ = pu.run_forward(wa)
    eb, ob, _, _ = pu.run_forward(wb)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    qa, ka, va = wa.q.cuda(), wa.k.cuda(), wa.v.cuda()
    qb, kb, vb = wb.q.cuda(), wb.k.cuda(), wb.v.cuda()
    torch.cuda.synchronize()
    outs = []
    for _ in range(3):
        xa, _, _ = ea.forward(qa, ka, va, wa.n_text, stream=sa)
        xb, _, _ = eb.forward(qb, kb, vb, wb.n_text, stream=sb)
        outs.append((xa, xb))
    torch.cuda.synchronize()
    for xa, xb in outs:
        assert torch.equal(xa, oa) and torch.equal(xb, ob)
    assert ea.header().status == 0 and eb.header().status == 0


@pytest.mark.parametrize("scale_q,scale_k,compensate", [(16.0, 1.0, True), (1.0 / 64, 1.0 / 32, True),
                                                        (4.0, 4.0, False), (2.0, 16.0, False)])
def test_inputs_far_from_unit_scale(scale_q, scale_k, compensate):
    """Queries and keys scaled by powers of two far from the N(0,1) scale of the benchmark inputs.  The
    tensor-core selection kernel works in fixed point relative to the largest exponents of a query row and
    of a head's mean keys, so a common factor that the logit scale compensates changes nothing; without
    the compensation the logits grow, the fixed-point error in logit units grows with them, and the rows
    leave the range the kernel was validated for: they are handed to the fp64 kernel (header counter
    fallback_rows), so the selection stays exact."""
    hdr = _scaled_inputs_every_row(scale_q, scale_k, compensate)
    if compensate:
        assert hdr.fallback_rows == 0
    else:
        assert hdr.fallback_rows > 0, "rows with large logits should have gone to the fp64 kernel"


@pytest.mark.parametrize("scale_q", [1.125, 1.25, 1.5, 2.0])
def test_softmax_reference_fixed_in_advance_or_running(scale_q):
    """The attention kernel fixes a row's softmax reference in advance when |q| max|k| scale bounds its scores
    by 2^48, and keeps a running maximum otherwise, warp by warp.  Queries scaled so that the bound (27 to 42
    in log2 units at unit scale for these shapes) lies below, around and above that limit: every row against
    the oracle on both sides of the switch and in warps where the rows disagree."""
    _scaled_inputs_every_row(scale_q, 1.0, False)


def _scaled_inputs_every_row(scale_q, scale_k, compensate):
    import dataclasses
    base = inputs.small_prefill(seed=33, T=16, H=8, W=8, n_text=19)
    wl = dataclasses.replace(base, q=(base.q.float() * scale_q).to(torch.bfloat16),
                             k=(base.k.float() * scale_k).to(torch.bfloat16))
    softmax_scale = 1.0 / (np.sqrt(wl.D) * (scale_q * scale_k if compensate else 1.0))
    eng = binding.AdaSAttn(cube=wl.cube, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.D, top_p=wl.top_p,
                           softmax_scale=softmax_scale)
    eng.partition(wl.B, wl.T, wl.H, wl.W, wl.n_text)
    out, bitmap, count = eng.forward(wl.q.cuda(), wl.k.cuda(), wl.v.cuda(), wl.n_text, want_selection=True)
    torch.cuda.synchronize()
    hdr = eng.header()
    assert hdr.status == 0
    sh = oracle.make_shape(B=wl.B, T=wl.T, H=wl.H, W=wl.W, cube=wl.cube, n_text=wl.n_text, Hq=wl.Hq, Hkv=wl.Hkv,
                           D=wl.D, top_p=float(np.float32(wl.top_p)), scale=float(np.float32(softmax_scale)))
    rows = oracle.all_rows(sh)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows)
    got_sel = pu.unpack_bitmap(bitmap, sh.N).reshape(-1, sh.N)
    same, rep = pu.check_selection(sh, wl, rows, got_sel, res, label=f"scale {scale_q} x {scale_k}")
    got = out.float().cpu().numpy().transpose(0, 2, 1, 3).reshape(-1, wl.D)
    assert np.abs(got[same] - res["out"][same]).max() <= pu.MAX_ABS_TOL
    print(scale_q, scale_k, compensate, rep, "fallback rows", hdr.fallback_rows)
    return hdr


def test_forward_from_host_buffers_equals_forward():
    """adaspark_attn_forward_host copies q, k, v from pinned host memory, runs the prefill and copies the
    output back on the caller's stream: same bytes as the device-buffer call."""
    wl = inputs.small_prefill(seed=34, T=16, H=8, W=8, n_text=27)
    eng, out_ref, _, _ = pu.run_forward(wl, want_selection=False)
    q_h, k_h, v_h = wl.q.pin_memory(), wl.k.pin_memory(), wl.v.pin_memory()
    out_h = torch.empty_like(q_h).pin_memory()
    staging = tuple(torch.empty_like(t, device="cuda") for t in (wl.q, wl.k, wl.v, wl.q))
    s = torch.cuda.Stream()
    eng.forward_host(q_h, k_h, v_h, wl.n_text, out_h, staging, stream=s)
    s.synchronize()
    assert torch.equal(out_h, out_ref.cpu())
    assert eng.header().status == 0
