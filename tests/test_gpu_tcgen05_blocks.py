"""tcgen05 / TMA / TMEM building blocks checked in isolation on one 128x128x128 product."""
import pytest
import torch

from paper_2604_08077_b200 import binding

pytestmark = pytest.mark.gpu


def test_umma_selftest_matches_matmul():
    g = torch.Generator(device="cpu").manual_seed(3)
    a, b, c = (torch.randn(128, 128, generator=g).to(torch.bfloat16).cuda() for _ in range(3))
    d = torch.full((128, 128), float("nan"), device="cuda")
    e = torch.full((128, 128), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = binding.adaspark_attn_debug_umma_selftest(a, b, c, d, e, status)
    torch.cuda.synchronize()
    assert rc == binding.OK and int(status.item()) == 0
    d_ref = a.double() @ b.double().T
    assert torch.allclose(d.double(), d_ref, atol=1e-3, rtol=1e-4), (d.double() - d_ref).abs().max()
    p = (d / 64).to(torch.bfloat16)
    e_ref = p.double() @ c.double().T
    assert torch.allclose(e.double(), e_ref, atol=1e-3, rtol=1e-4), (e.double() - e_ref).abs().max()


def test_imma_selftest_is_an_exact_signed_product():
    g = torch.Generator(device="cpu").manual_seed(4)
    for lo, hi in [(-128, 128), (-128, -100), (100, 128)]:
        a = torch.randint(lo, hi, (128, 128), generator=g, dtype=torch.int32).to(torch.int8)
        b = torch.randint(-128, 128, (128, 128), generator=g, dtype=torch.int32).to(torch.int8)
        d = torch.full((128, 128), -1, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        rc = binding.adaspark_attn_debug_imma_selftest(a.cuda(), b.cuda(), d, status)
        torch.cuda.synchronize()
        assert rc == binding.OK and int(status.item()) == 0
        ref = a.to(torch.int64) @ b.to(torch.int64).T
        assert torch.equal(d.cpu().to(torch.int64), ref)


def test_bounded_wait_expires_and_the_context_survives():
    """A wait on a barrier nobody arrives at gives up after its limit (1 ms here), reports
    ERR_TIMEOUT through the status word, releases the other waiting threads through the abort flag,
    and leaves the device usable: the path every mbarrier wait of the tcgen05 kernels takes if its
    protocol is ever starved."""
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    rc = binding.adaspark_attn_debug_wait_timeout(1_000_000, status, waited)
    torch.cuda.synchronize()
    assert rc == binding.OK
    assert status.tolist() == [binding.ERR_TIMEOUT, 1]
    assert 1_000_000 <= int(waited.item()) < 50_000_000
    # the context is intact: another kernel of the library runs and is correct
    a = torch.ones(128, 128, dtype=torch.int8, device="cuda")
    d = torch.zeros(128, 128, dtype=torch.int32, device="cuda")
    st2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert binding.adaspark_attn_debug_imma_selftest(a, a, d, st2) == binding.OK
    torch.cuda.synchronize()
    assert int(st2.item()) == 0 and bool((d == 128).all())
