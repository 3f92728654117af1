"""The workspace-free decode entry point, called through the C ABI.

Some callers cannot allocate device memory when they decode (their own pool owns the whole GPU,
or their serving loop must not call cudaMalloc), so `adaspark_attn_decode_static` keeps its
scratch in an 8 MiB array inside the library.  This file checks that it returns what the regular
`adaspark_attn_decode` returns, twice in a row (the array keeps the previous call's contents), that
its output also agrees with the CPU oracle, that the calls allocate no device memory, that a second
handle with another shape can use the same array in between, and that a partition too large for
the array is refused with a clear error.  It is named to be
collected last, so a failure here cannot hide another test's result in a stop-at-first-failure run.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_08077_b200 import binding, inputs

import parity_util as pu

pytestmark = pytest.mark.gpu


def test_static_decode_matches_workspace_decode_twice():
    wl = inputs.small_decode(seed=77, B=2, T=16, H=8, W=8, n_text=37, Hq=8, Hkv=2, D=128)
    eng = pu.make_engine(wl, n_text_max=wl.n_text + 2)
    eng.forward(None, wl.k.cuda(), wl.v.cuda(), wl.n_text)
    assert eng.layout.decode_workspace_bytes <= binding.STATIC_SCRATCH_BYTES
    q_new, k_new, v_new = wl.q_new.cuda(), wl.k_new.cuda(), wl.v_new.cuda()
    for step, text_len in enumerate([[37, 30], [38, 31]]):      # two calls in a row
        tl = torch.tensor(text_len, dtype=torch.int32, device="cuda")
        q_step = (q_new.float() * (1.0 + step)).to(torch.bfloat16)   # a different query each call
        ref, ref_bitmap = eng.decode(q_step, k_new, v_new, tl, want_selection=True)
        out = torch.full_like(ref, float("nan"))
        bitmap = torch.zeros_like(ref_bitmap)
        binding.adaspark_attn_decode_static(eng.handle, q_step, k_new, v_new, eng.k_cube, eng.v_cube,
                                            eng.cube_keys, tl, out, bitmap)
        torch.cuda.synchronize()
        assert torch.equal(bitmap, ref_bitmap)
        err = (out.float() - ref.float()).abs().max().item()
        assert err <= pu.MAX_ABS_TOL, f"call {step}: static decode differs by {err}"
        assert torch.isfinite(out.float()).all()
        if step == 0:                                             # and against the CPU oracle
            res = oracle.decode(pu.oracle_shape(wl), wl.k, wl.v, text_len, q_step.cpu(), wl.k_new, wl.v_new)
            same = (pu.unpack_bitmap(bitmap, wl.N) == res["sel"]).all(axis=-1)
            assert (same | (res["margin"] < pu.TIE_MARGIN)).all()
            err = np.abs(out[:, 0].float().cpu().numpy() - res["out"])[same].max()
            assert err <= pu.MAX_ABS_TOL, f"static decode differs from the oracle by {err}"


def test_static_decode_allocates_nothing_and_tolerates_another_handle():
    """No device memory is taken by the calls (free memory and torch's own allocator are unchanged
    across them), and a second handle of a different shape may use the shared array between two
    calls of the first: whatever it leaves behind does not change the first handle's result."""
    wa = inputs.small_decode(seed=78, B=2, T=16, H=8, W=8, n_text=12, Hq=8, Hkv=2, D=128)
    wb = inputs.small_decode(seed=79, B=1, T=8, H=8, W=8, cube=(2, 4, 4), n_text=40, Hq=4, Hkv=4, D=64, top_p=0.7)
    engs, args = [], []
    for wl in (wa, wb):
        eng = pu.make_engine(wl, n_text_max=wl.n_text + 1)
        eng.forward(None, wl.k.cuda(), wl.v.cuda(), wl.n_text)
        tl = torch.full((wl.B,), wl.n_text, dtype=torch.int32, device="cuda")
        q, k, v = wl.q_new.cuda(), wl.k_new.cuda(), wl.v_new.cuda()
        ref, _ = eng.decode(q, k, v, tl)
        engs.append(eng)
        args.append((q, k, v, tl, ref, torch.empty_like(ref)))

    def call(i):
        q, k, v, tl, _, out = args[i]
        e = engs[i]
        binding.adaspark_attn_decode_static(e.handle, q, k, v, e.k_cube, e.v_cube, e.cube_keys, tl, out, None)

    call(0)                                                        # first call: symbol look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for i in (0, 1, 0, 1, 0):
        call(i)
        torch.cuda.synchronize()                                   # serialised: the handles share the array
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "device memory was allocated or freed by the static decode calls"
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    for q, k, v, tl, ref, out in args:
        assert (out.float() - ref.float()).abs().max().item() <= pu.MAX_ABS_TOL


def test_static_decode_rejects_partitions_beyond_its_scratch():
    eng = binding.AdaSAttn(cube=(4, 4, 4), n_q_heads=28, n_kv_heads=4, head_dim=128, top_p=0.9)
    ws = binding.adaspark_attn_partition(eng.handle, 64, 512, 16, 16, 512)   # batch 64: > 8 MiB
    lay = binding.adaspark_attn_get_layout(eng.handle)
    assert lay.decode_workspace_bytes > binding.STATIC_SCRATCH_BYTES and ws > 0
    fake = 0x1000    # never dereferenced: the size check comes first
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_decode_static(eng.handle, fake, fake, fake, fake, fake, fake, fake, fake,
                                            None)
    assert e.value.status == binding.ERR_WORKSPACE_TOO_SMALL
    assert "built-in scratch" in str(e.value)
