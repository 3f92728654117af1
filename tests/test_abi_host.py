"""CPU-only checks of the C-ABI library: it builds, exports every symbol the header declares,
validates arguments on the host, derives the partition sizes, and fails loudly without a GPU."""
import ctypes
import os
import re

import pytest
import torch

from paper_2604_08077_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def cfg(**kw):
    base = dict(cube_t=4, cube_h=4, cube_w=4, n_q_heads=28, n_kv_heads=4, head_dim=128, top_p=0.9,
                softmax_scale=0.0, device=0, top_k=0)
    base.update(kw)
    return binding.Config(*[base[f[0]] for f in binding.Config._fields_])


def test_every_declared_symbol_is_exported(lib):
    declared = set()
    inc = os.path.join(ROOT, "include")
    for name in os.listdir(inc):
        if name.endswith(".h"):
            text = open(os.path.join(inc, name)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)          # declarations only
            declared |= set(re.findall(r"\b(adaspark_attn_[a-z_0-9]+)\s*\(", text))
    assert {"adaspark_attn_create", "adaspark_attn_partition", "adaspark_attn_forward",
            "adaspark_attn_decode", "adaspark_attn_destroy"} <= declared
    for sym in declared:
        assert hasattr(lib, sym), f"{sym} declared in include/ but not exported"
    assert declared >= set(binding.EXPORTS)


def test_create_validation(lib):
    h = ctypes.c_void_p()
    assert lib.adaspark_attn_create(None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    for bad, code in [(dict(head_dim=96), binding.ERR_UNSUPPORTED),
                      (dict(cube_t=3), binding.ERR_UNSUPPORTED),          # C = 48
                      (dict(n_q_heads=30), binding.ERR_INVALID_ARG),      # 30 % 4 != 0
                      (dict(n_q_heads=68, n_kv_heads=4), binding.ERR_UNSUPPORTED),  # group 17
                      (dict(top_p=0.0), binding.ERR_INVALID_ARG),
                      (dict(top_k=-1), binding.ERR_INVALID_ARG),
                      (dict(cube_h=0), binding.ERR_INVALID_ARG)]:
        c = cfg(**bad)
        assert lib.adaspark_attn_create(ctypes.byref(c), ctypes.byref(h)) == code, bad
        assert h.value is None
    hd = binding.adaspark_attn_create(cfg())
    assert hd
    binding.adaspark_attn_destroy(hd)
    assert lib.adaspark_attn_destroy(None) == binding.OK


@pytest.mark.parametrize("T,H,W,cube,n_text,N,C", [
    (8, 8, 8, (2, 4, 4), 32, 16, 32), (64, 16, 16, (4, 4, 4), 128, 256, 64),
    (256, 16, 16, (4, 4, 4), 256, 1024, 64), (512, 16, 16, (4, 4, 4), 512, 2048, 64),
    (16, 16, 16, (4, 8, 8), 0, 16, 256)])
def test_partition_layout(lib, T, H, W, cube, n_text, N, C):
    hd = binding.adaspark_attn_create(cfg(cube_t=cube[0], cube_h=cube[1], cube_w=cube[2]))
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_get_layout(hd)
    assert e.value.status == binding.ERR_NOT_PARTITIONED
    ws = binding.adaspark_attn_partition(hd, 2, T, H, W, n_text)
    lay = binding.adaspark_attn_get_layout(hd)
    assert lay.n_cubes == N and lay.cube_tokens == C and lay.s_video == T * H * W
    assert lay.s_cap % 128 == 0 and lay.s_cap >= T * H * W + n_text + 1
    assert lay.bitmap_words == (N + 31) // 32
    assert lay.k_cube_bytes == 2 * 4 * lay.s_cap * 128 * 2 == lay.v_cube_bytes
    assert lay.cube_keys_bytes == 2 * 4 * N * 128 * 4
    assert ws == max(lay.forward_workspace_bytes, lay.decode_workspace_bytes) > 0
    binding.adaspark_attn_destroy(hd)


def test_partition_rejections(lib):
    hd = binding.adaspark_attn_create(cfg())
    for args, code in [((1, 1024, 32, 32, 0), binding.ERR_UNSUPPORTED),   # 16384 cubes > 4096
                       ((1, 1021, 30, 31, 0), binding.ERR_UNSUPPORTED),   # the same count with cut boundary cubes
                       ((0, 8, 16, 16, 0), binding.ERR_INVALID_ARG),
                       ((1, 8, 16, 16, -1), binding.ERR_INVALID_ARG)]:
        with pytest.raises(binding.AdasparkError) as e:
            binding.adaspark_attn_partition(hd, *args)
        assert e.value.status == code, args
    binding.adaspark_attn_destroy(hd)


def test_partition_of_a_grid_the_window_does_not_divide(lib):
    """ceil() cubes per axis; the cache holds C slots per cube, so s_video counts slots, not tokens."""
    hd = binding.adaspark_attn_create(cfg())
    binding.adaspark_attn_partition(hd, 1, 6, 18, 15, 5)
    lay = binding.adaspark_attn_get_layout(hd)
    assert lay.n_cubes == 2 * 5 * 4 and lay.s_video == 40 * 64 > 6 * 18 * 15
    assert lay.s_cap % 128 == 0 and lay.s_cap >= lay.s_video + 5 + 1
    binding.adaspark_attn_destroy(hd)


def test_forward_and_decode_argument_errors_are_found_on_the_host(lib):
    hd = binding.adaspark_attn_create(cfg())
    fake = 0x1000  # never dereferenced: every call below must fail before any launch
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_forward(hd, fake, fake, fake, 0, fake, fake, fake, fake, None, None,
                                      fake, 1 << 40)
    assert e.value.status == binding.ERR_NOT_PARTITIONED
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_decode(hd, fake, fake, fake, fake, fake, fake, fake, fake, None, fake,
                                     1 << 40)
    assert e.value.status == binding.ERR_NOT_PARTITIONED
    ws = binding.adaspark_attn_partition(hd, 1, 8, 16, 16, 16)
    cases = [
        (dict(k=None), binding.ERR_INVALID_ARG), (dict(out=None), binding.ERR_INVALID_ARG),
        (dict(n_text=17), binding.ERR_INVALID_ARG), (dict(n_text=-1), binding.ERR_INVALID_ARG),
        (dict(ws_bytes=ws - 1), binding.ERR_WORKSPACE_TOO_SMALL),
        (dict(ws=fake + 8), binding.ERR_INVALID_ARG), (dict(ws=None), binding.ERR_INVALID_ARG)]
    for kw, code in cases:
        a = dict(q=fake, k=fake, v=fake, n_text=16, out=fake, ws=fake * 256, ws_bytes=ws)
        a.update(kw)
        with pytest.raises(binding.AdasparkError) as e:
            binding.adaspark_attn_forward(hd, a["q"], a["k"], a["v"], a["n_text"], a["out"], fake,
                                          fake, fake, None, None, a["ws"], a["ws_bytes"])
        assert e.value.status == code, kw
        assert str(e.value)
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_decode(hd, fake, fake, None, fake, fake, fake, fake, fake, None,
                                     fake * 256, ws)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_decode(hd, fake, fake, fake, fake, fake, fake, fake, fake, None,
                                     fake * 256, 16)
    assert e.value.status == binding.ERR_WORKSPACE_TOO_SMALL
    binding.adaspark_attn_destroy(hd)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_compute_fails_loudly_without_a_gpu(lib):
    """No CPU fallback: with valid arguments but no CUDA device the call reports ERR_CUDA."""
    hd = binding.adaspark_attn_create(cfg())
    ws = binding.adaspark_attn_partition(hd, 1, 8, 16, 16, 0)
    fake = 0x100000
    with pytest.raises(binding.AdasparkError) as e:
        binding.adaspark_attn_forward(hd, fake, fake, fake, 0, fake, fake, fake, fake, None, None,
                                      fake, ws)
    assert e.value.status == binding.ERR_CUDA
    binding.adaspark_attn_destroy(hd)


def test_missing_library_raises(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load()


def test_index_division_matches_integer_division(lib):
    """The multiply-shift division behind the kernels' index arithmetic equals n // d on every
    divisor a partition can produce (small ones exhaustively, large ones sampled)."""
    import numpy as np
    rng = np.random.default_rng(0)
    divisors = list(range(1, 300)) + [511, 512, 513, 1023, 1025, 4095, 4096, 4097, 65535, 65536,
                                      1048575, 1048577, (1 << 30) - 1, (1 << 30) + 1, (1 << 31) - 1]
    for d in divisors:
        edge = [0, 1, d - 1, d, d + 1, 2 * d - 1, 2 * d, (1 << 31) - 1,
                ((1 << 31) - 1) // d * d, max(((1 << 31) - 1) // d * d - 1, 0)]
        ns = [int(x) for x in edge if 0 <= x < (1 << 31)] + [int(x) for x in rng.integers(0, 1 << 31, 40)]
        for n in ns:
            assert binding.adaspark_attn_debug_fastdiv(n, d) == n // d, (n, d)
    assert binding.adaspark_attn_debug_fastdiv(-1, 3) == -1
    assert binding.adaspark_attn_debug_fastdiv(5, 0) == -1


def test_wait_timeout_selftest_rejects_limits_outside_its_range(lib):
    """Host-side argument check only (no launch): the limit must lie in [1 us, 100 ms]."""
    fake = 0x1000
    for bad in (0, 999, 100_000_001):
        assert binding.adaspark_attn_debug_wait_timeout(bad, fake, fake) == binding.ERR_INVALID_ARG
    assert binding.adaspark_attn_debug_wait_timeout(1000, None, fake) == binding.ERR_INVALID_ARG


def test_partition_rejects_sequences_beyond_the_block_bitmap(lib):
    """The attention kernel keeps one bit per 64-key block of a sequence (32768 blocks = 2097152
    cache rows); a legal-looking partition beyond that is refused instead of overrunning it."""
    hd = binding.adaspark_attn_create(cfg(cube_t=4, cube_h=16, cube_w=16, n_q_heads=1, n_kv_heads=1))
    with pytest.raises(binding.AdasparkError) as e:                     # 4096 cubes of 1024 tokens
        binding.adaspark_attn_partition(hd, 1, 4 * 4096, 16, 16, 0)
    assert e.value.status == binding.ERR_UNSUPPORTED
    assert binding.adaspark_attn_partition(hd, 1, 4 * 2047, 16, 16, 100) > 0   # just below the limit
    with pytest.raises(binding.AdasparkError) as e:                     # a large text capacity
        binding.adaspark_attn_partition(hd, 1, 4 * 2047, 16, 16, 2 * 1024 * 1024)
    assert e.value.status == binding.ERR_UNSUPPORTED
    binding.adaspark_attn_destroy(hd)
