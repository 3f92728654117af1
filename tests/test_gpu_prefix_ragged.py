"""GPU parity for the two settings the paper leaves open: text placed before the video (a prompt prefix,
always attended in full) and video grids the cube window does not divide (boundary cubes hold fewer
tokens).  Every row of small problems against the CPU oracle: caches, mean keys, selection, outputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu


def check_caches(wl, eng):
    """k_cube / v_cube / cube_keys against the oracle's order: video slots first (empty slots of boundary
    cubes zero), then the prefix, then the text; zero beyond the sequence."""
    sh = oracle.shape_of(wl)
    _, inv = oracle.positions(sh)                                   # token at every oracle position (-1: none)
    P0, nvid = sh.n_prefix, sh.N * sh.C
    order = np.concatenate([inv[P0:P0 + nvid], inv[:P0], inv[P0 + nvid:]])    # the caches' order
    held = torch.from_numpy(order >= 0)
    idx = torch.from_numpy(np.where(order >= 0, order, 0))
    n_slots, s_cap = len(order), eng.layout.s_cap
    k_ref = wl.k[:, idx].permute(0, 2, 1, 3) * held[None, None, :, None]
    v_ref = wl.v[:, idx].permute(0, 2, 1, 3) * held[None, None, :, None]
    k_got = eng.k_cube.cpu()
    assert torch.equal(k_got[:, :, :n_slots], k_ref.to(torch.bfloat16))
    assert (k_got[:, :, n_slots:] == 0).all()
    v_got = eng.v_cube.cpu().permute(0, 1, 2, 4, 3).reshape(wl.B, wl.Hkv, s_cap, wl.D)
    assert torch.equal(v_got[:, :, :n_slots], v_ref.to(torch.bfloat16))
    assert (v_got[:, :, n_slots:] == 0).all()
    kbar = oracle.mean_keys(sh, wl.k).astype(np.float32)
    assert np.array_equal(eng.cube_keys.cpu().numpy(), kbar)


CASES = {
    "prefix_37": lambda: inputs.small_prefill(seed=101, T=8, H=8, W=8, n_text=21, n_prefix=37),
    "prefix_200_no_text": lambda: inputs.small_prefill(seed=102, T=8, H=8, W=8, n_text=0, n_prefix=200, Hq=2, Hkv=1, D=64),
    "prefix_c16_straddle": lambda: inputs.small_prefill(seed=103, T=3, H=4, W=12, cube=(1, 4, 4), n_text=70, n_prefix=13,
                                                         Hq=2, Hkv=1, D=64, top_p=0.8),
    "prefix_c256": lambda: inputs.small_prefill(seed=104, T=8, H=16, W=8, cube=(4, 8, 8), n_text=5, n_prefix=70, Hq=4, Hkv=1),
    "ragged_thw": lambda: inputs.small_prefill(seed=105, T=10, H=7, W=9, cube=(4, 4, 4), n_text=9, Hq=4, Hkv=2, top_p=0.85),
    "ragged_t_only": lambda: inputs.small_prefill(seed=106, T=11, H=8, W=8, cube=(4, 4, 4), n_text=30, Hq=2, Hkv=2, D=64),
    "ragged_c16": lambda: inputs.small_prefill(seed=107, T=5, H=6, W=13, cube=(1, 4, 4), n_text=3, Hq=2, Hkv=1, D=64, top_p=0.7),
    "ragged_c256": lambda: inputs.small_prefill(seed=108, T=9, H=12, W=20, cube=(4, 8, 8), n_text=12, Hq=2, Hkv=1, top_p=0.8),
    "ragged_with_prefix": lambda: inputs.small_prefill(seed=109, T=9, H=10, W=6, cube=(2, 4, 4), n_text=17, n_prefix=29,
                                                        Hq=4, Hkv=2, D=64, top_p=0.9),
}


@pytest.mark.parametrize("case", sorted(CASES))
@pytest.mark.parametrize("kernel", [1, 0])
def test_every_row(case, kernel):
    wl = CASES[case]()
    eng, out, bitmap, count = pu.run_forward(wl, prefill_kernel=kernel)
    assert eng.header().status == 0
    check_caches(wl, eng)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, label=case)
    assert rep["rows"] == wl.B * wl.Hq * wl.S
    print(case, kernel, rep)


def test_p1_with_prefix_and_ragged_grid_is_dense_attention():
    wl = CASES["ragged_with_prefix"]()
    eng, out, bitmap, count = pu.run_forward(wl, top_p=1.0)
    rep = pu.compare_rows(wl, oracle.all_rows(oracle.shape_of(wl)), out, bitmap, count, top_p=1.0, label="p=1")
    print(rep)


def test_decode_after_a_prefix_prefill_and_on_a_ragged_grid():
    """A decode step on caches built with a prefix (text_len counts prefix + text) and on a ragged grid
    (empty slots of selected boundary cubes are not attended) equals the oracle's appended row."""
    for wl in (inputs.small_prefill(seed=110, T=8, H=8, W=8, n_text=11, n_prefix=19, Hq=4, Hkv=2),
               inputs.small_prefill(seed=111, T=7, H=6, W=10, n_text=11, Hq=4, Hkv=2, top_p=0.95)):
        eng = pu.make_engine(wl, n_text_max=wl.n_text + wl.n_prefix + 4)
        eng.forward(None, wl.k.cuda(), wl.v.cuda(), wl.n_text, n_prefix=wl.n_prefix)
        g = torch.Generator().manual_seed(5)
        q_new = torch.randn(wl.B, 1, wl.Hq, wl.D, generator=g).to(torch.bfloat16)
        k_new = torch.randn(wl.B, 1, wl.Hkv, wl.D, generator=g).to(torch.bfloat16)
        v_new = torch.randn(wl.B, 1, wl.Hkv, wl.D, generator=g).to(torch.bfloat16)
        tl = torch.full((wl.B,), wl.n_prefix + wl.n_text, dtype=torch.int32, device="cuda")
        out, bitmap = eng.decode(q_new.cuda(), k_new.cuda(), v_new.cuda(), tl, want_selection=True)
        torch.cuda.synchronize()
        assert eng.header().status == 0
        # the oracle's view: the same sequence with one more text token, last row
        full = inputs.Workload(name="appended", B=wl.B, T=wl.T, H=wl.H, W=wl.W, cube=wl.cube, n_text=wl.n_text + 1,
                               Hq=wl.Hq, Hkv=wl.Hkv, D=wl.D, top_p=wl.top_p, n_prefix=wl.n_prefix,
                               q=torch.cat([torch.zeros_like(wl.q), q_new], 1), k=torch.cat([wl.k, k_new], 1),
                               v=torch.cat([wl.v, v_new], 1))
        sh = pu.oracle_shape(full)
        rows = [(b, h, full.S - 1) for b in range(wl.B) for h in range(wl.Hq)]
        res = oracle.rows(sh, full.q, full.k, full.v, rows)
        got_sel = pu.unpack_bitmap(bitmap, sh.N).reshape(-1, sh.N)
        assert ((got_sel == res["sel"]).all(axis=1) | (res["margin"] < pu.TIE_MARGIN)).all()
        err = np.abs(out[:, 0].float().cpu().numpy().reshape(-1, wl.D) - res["out"]).max()
        assert err <= pu.MAX_ABS_TOL, err


def test_what_is_still_refused():
    eng = binding.AdaSAttn(cube=(4, 4, 4), n_q_heads=4, n_kv_heads=2, head_dim=128, top_p=0.9)
    eng.partition(1, 10, 8, 8, 16)                                  # ragged in time
    x = torch.zeros(1, 256, 4, 128, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, 256, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.AdasparkError) as e:                  # chunks need a grid the window divides
        eng.forward_chunk(x, kv, kv, 0, 4, -1)
    assert e.value.status == binding.ERR_UNSUPPORTED
    eng2 = binding.AdaSAttn(cube=(4, 4, 4), n_q_heads=4, n_kv_heads=2, head_dim=128, top_p=0.9)
    eng2.partition(1, 8, 8, 8, 16)
    with pytest.raises(binding.AdasparkError) as e:                  # prefix + text beyond the text capacity
        eng2.forward(x, kv, kv, 10, n_prefix=7)
    assert e.value.status == binding.ERR_INVALID_ARG
