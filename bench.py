#!/usr/bin/env python
"""Benchmark of the AdaS-Attn hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole prefill path (re-layout + pooling, cube scoring, Top-p
selection, gathered attention) over one batch of the Qwen2-7B-shaped workload (config 2:
64x16x16 video tokens in 4x4x4 cubes + 128 text tokens, 28/4 heads, head_dim 128, p = 0.9,
bf16, seeded synthetic inputs).  Rank 0 prints ONE JSON line.  With N > 1 every rank runs
its own replica of the workload (independent sequences, no exchange step): weak scaling.

`--impl reference` times the CPU oracle (as it stands) on a bounded row sample of the same
workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_08077_b200 import inputs  # noqa: E402

METRIC = "AdaS-Attn prefill tokens/s"
UNIT = "tokens/s"
WORKLOAD = ("config2: AdaS-Attn prefill, batch 1, 64x16x16 video tokens (cube 4x4x4, 256 cubes) "
            "+ 128 text, 28/4 heads, head_dim 128, p=0.9")


def profiled_traffic(kernel_source: str, summary: str):
    """DRAM bytes per launch of a kernel from its committed ncu summary, or None when the kernel's
    source file no longer has the hash the summary was taken with (the counters are then stale).
    The summary carries two lines: `dram_bytes_per_launch: <n>` and `kernel_source_sha256: <hex>`."""
    import hashlib
    import re
    try:
        text = open(os.path.join(ROOT, "profiles", summary)).read()
        src = open(os.path.join(ROOT, "paper_2604_08077_b200", "csrc", kernel_source), "rb").read()
    except OSError:
        return None
    m_bytes = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", text)
    m_hash = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    if not m_bytes or not m_hash or hashlib.sha256(src).hexdigest() != m_hash.group(1):
        return None
    return float(m_bytes.group(1))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []          # (host time of arrival, line)
        self.t_begin = self.t_end = None

    def wait_first(self, timeout_s: float = 5.0):
        """nvidia-smi needs a fraction of a second before its first line: wait for it, so that the
        timed region (tens of milliseconds) is sampled from its start."""
        t0 = time.time()
        while self.proc is not None and not self.lines and time.time() - t0 < timeout_s:
            time.sleep(0.01)

    def begin(self):
        self.t_begin = time.time()

    def end(self):
        self.t_end = time.time()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        lines = self.lines
        if self.t_begin is not None and self.t_end is not None:
            # samples taken during the timed region; a region shorter than the sampling period may hold none:
            # then the samples within a quarter of a second around it
            inside = [ln for t, ln in lines if self.t_begin <= t <= self.t_end + 0.02]
            if len(inside) < 2:
                inside = [ln for t, ln in lines if self.t_begin - 0.25 <= t <= self.t_end + 0.25]
            lines = [(0.0, ln) for ln in inside]
        for _, line in lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # samples under load = the upper half (idle samples between steps pull the median down)
        sm_sorted = sorted(sm)
        load = sm_sorted[len(sm_sorted) // 2:] if sm_sorted else []
        return {"sm_mhz": statistics.median(load) if load else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's figure (replicas run independently; the job is as slow as its slowest rank)."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, ms_max: float) -> float:
    """Whole-job units per second: every rank processes units_per_rank in the slowest rank's time."""
    return world * units_per_rank / (ms_max * 1e-3)


def timed_steps(step_fn, steps, warmup, flush, dist_barrier, on_begin=None, on_end=None):
    """W warm-ups, then K steps each bracketed by CUDA events on the current stream, with an L2
    flush (not timed) before every step.  Returns per-step milliseconds."""
    for _ in range(warmup):
        flush()
        step_fn()
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    extra = []
    if on_begin:
        on_begin()
    for i in range(steps):
        flush()
        starts[i].record()
        r = step_fn()
        ends[i].record()
        if r is not None:
            extra.append(r())
    torch.cuda.synchronize()
    if on_end:
        on_end()
    dist_barrier()
    return [s.elapsed_time(e) for s, e in zip(starts, ends)], extra


def run_reference(args):
    """The CPU oracle timed on a bounded sample of config 2 (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    wl = inputs.config2()
    sh = oracle.shape_of(wl, top_p=float(np.float32(wl.top_p)))
    q, k, v = oracle.as_f32(wl.q), oracle.as_f32(wl.k), oracle.as_f32(wl.v)
    n_rows = args.ref_rows
    times = []
    for step in range(args.warmup + args.steps):
        rng = np.random.default_rng(step)
        rows = np.stack([np.zeros(n_rows, np.int64), rng.integers(0, wl.Hq, n_rows),
                         rng.integers(0, wl.S, n_rows)], axis=1)
        t0 = time.perf_counter()
        kbar = oracle.mean_keys(sh, k)
        oracle.rows(sh, q, k, v, rows, kbar=kbar)
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    tokens_per_s = (n_rows / wl.Hq) / sec
    cores = oracle.n_threads()
    sample = (f"{n_rows} uniformly sampled (head, token) rows of config 2 per step, mean keys "
              f"recomputed every step; tokens/s = rows / n_q_heads / seconds")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": tokens_per_s, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": tokens_per_s, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": tokens_per_s, "unit": UNIT, "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0}}))


def parity_check(wl, eng, q, k, v, n_rows=1200, n_sel_rows=12000):
    """The CUDA path against the CPU oracle on seeded rows of the bench workload, before anything is
    timed: selection on n_sel_rows rows, outputs on n_rows of them.  Rows outside the 1e-6 tie margin
    must match bit for bit; rows inside it are counted (`differing`) and their outputs compared with
    the oracle's attention on the GPU's own set.  Raises on a mismatch."""
    import oracle
    sh = oracle.shape_of(wl, top_p=float(np.float32(wl.top_p)))
    out, bitmap, _ = eng.forward(q, k, v, wl.n_text, want_selection=True)
    torch.cuda.synchronize()
    rng = np.random.default_rng(11)
    rows = np.stack([np.zeros(n_sel_rows, np.int64), rng.integers(0, wl.Hq, n_sel_rows),
                     rng.integers(0, wl.S, n_sel_rows)], axis=1)
    kbar = oracle.mean_keys(sh, wl.k)
    res = oracle.rows(sh, wl.q, wl.k, wl.v, rows, kbar=kbar, attend=False)
    dev = bitmap.device
    hh, nn = torch.from_numpy(rows[:, 1]).to(dev), torch.from_numpy(rows[:, 2]).to(dev)
    words = bitmap[0, hh, nn].cpu().numpy().view(np.uint32)
    got_sel = ((words[..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(len(rows), -1)[:, :sh.N].astype(np.uint8)
    same = (got_sel == res["sel"]).all(axis=1)
    near = res["margin"] < 1e-6
    if not (same | near).all():
        raise SystemExit("bench: selection differs from the oracle outside the 1e-6 tie margin")
    sub = rows[:n_rows]
    ref = oracle.rows(sh, wl.q, wl.k, wl.v, sub, kbar=kbar)["out"]
    if not same[:n_rows].all():
        bad = ~same[:n_rows]
        ref[bad] = oracle.attend_given(sh, wl.q, wl.k, wl.v, sub[bad], got_sel[:n_rows][bad])
    got = out[0, nn[:n_rows], hh[:n_rows]].float().cpu().numpy()
    max_abs = float(np.abs(got - ref).max())
    mean_rel = float(np.abs(got - ref).mean() / np.abs(ref).mean())
    if max_abs > 2e-2 or mean_rel > 1e-2:
        raise SystemExit(f"bench: outputs differ from the oracle (max abs {max_abs}, mean rel {mean_rel})")
    return {"rows": int(n_sel_rows), "output_rows": int(n_rows), "differing": int((~same).sum()),
            "near_tie": int(near.sum()), "max_abs": max_abs, "mean_rel": mean_rel,
            "fallback_rows": int(eng.header().fallback_rows)}


def cpu_baseline(wl, n_rows=32768):
    import oracle
    sh = oracle.shape_of(wl, top_p=float(np.float32(wl.top_p)))
    q, k, v = oracle.as_f32(wl.q), oracle.as_f32(wl.k), oracle.as_f32(wl.v)
    rng = np.random.default_rng(0)
    rows = np.stack([np.zeros(n_rows, np.int64), rng.integers(0, wl.Hq, n_rows),
                     rng.integers(0, wl.S, n_rows)], axis=1)
    t0 = time.perf_counter()
    kbar = oracle.mean_keys(sh, k)
    oracle.rows(sh, q, k, v, rows, kbar=kbar)
    sec = time.perf_counter() - t0
    return {"value": (n_rows / wl.Hq) / sec, "unit": UNIT, "cores": oracle.n_threads(),
            "kind": "oracle",
            "sample": f"{n_rows} uniformly sampled (head, token) rows of config 2 + all mean keys, "
                      f"{sec:.1f} s; tokens/s = rows / n_q_heads / seconds"}


GATHER_DEFAULT_THRESHOLD = 30.0    # the library's default decision threshold of the query-gather path
SWEEP_GATHER_BUDGET = 32 << 30     # workspace the query-gather path may use on the long-video workloads (library default: 24 GiB)

def one_config(wx, p, flush, local_rank, n_steps=3, gather=None, budget=SWEEP_GATHER_BUDGET, warmup=3):
    """One forward configuration timed with stage times: gather None = the library's own per-pair decision
    (default threshold), 0.0 = union path only."""
    from paper_2604_08077_b200 import binding
    e = binding.AdaSAttn(cube=wx.cube, n_q_heads=wx.Hq, n_kv_heads=wx.Hkv, head_dim=wx.D, top_p=p,
                         device=local_rank)
    e.set_gather(GATHER_DEFAULT_THRESHOLD if gather is None else gather, budget)
    e.partition(wx.B, wx.T, wx.H, wx.W, wx.n_text)
    binding.adaspark_attn_enable_stage_timing(e.handle, True)
    ox = torch.empty_like(wx.q)

    def stp():
        e.forward(wx.q, wx.k, wx.v, wx.n_text, out=ox)
        return lambda: binding.adaspark_attn_get_stage_times(e.handle)

    t, stg = timed_steps(stp, n_steps, warmup, flush, lambda: None)
    stg = np.asarray(stg).mean(axis=0)
    hx = e.header()
    _, _, cnt = e.forward(wx.q, wx.k, wx.v, wx.n_text, out=ox, want_selection=True)
    torch.cuda.synchronize()
    sel = int(cnt.sum().item())
    Cx = wx.C
    local_x = wx.S_v // Cx * (Cx * (Cx + 1) // 2) + wx.n_text * (wx.n_text + 1) // 2
    useful = 4.0 * wx.D * (sel * Cx + wx.B * wx.Hq * local_x)
    executed = float(hx.executed_kv_blocks) * 128 * 64 * wx.D * 4
    n_pairs = wx.B * wx.Hq * ((wx.S + 255) // 256)
    rec = {"p": p, "forward_ms": sum(t) / len(t),
           "stages_ms": {"relayout_pool": float(stg[0]), "score_select": float(stg[1]), "attention": float(stg[2])},
           "mean_selected_cubes_per_row": sel / (wx.B * wx.Hq * wx.S),
           "useful_over_executed": useful / max(executed, 1.0),
           "executed_tflops": executed / (float(stg[2]) * 1e-3) / 1e12,
           "kv_blocks_per_pair_tile": {"mean": float(hx.executed_kv_blocks) / 2 / n_pairs, "max": int(hx.max_tile_kv_blocks)},
           "gather": {"pair_tiles": int(hx.gather_pair_tiles), "of_pair_tiles": n_pairs,
                      "entries": int(hx.gather_entries), "items": int(hx.gather_items)},
           "fallback_rows": int(hx.fallback_rows), "status": int(hx.status)}
    e.close()
    del e, ox, cnt
    return rec



def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-rows", type=int, default=16384)
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cohesive", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the config-3 sweep and config 4")
    ap.add_argument("--decode-batch", type=int, default=16)
    ap.add_argument("--prefill-kernel", type=int, default=None)
    ap.add_argument("--point", default=None, metavar="SIGMA,P[,BUDGET_GIB[,THRESHOLD]]",
                    help="time only this point of the config-3 sweep (profiling runs) and print its record")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    from paper_2604_08077_b200 import binding, build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the AdaS-Attn path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()

    if rank == 0:
        build.build()
    barrier()
    binding.load()
    peaks = load_peaks()
    if args.point is not None:
        f = [float(x) for x in args.point.split(",")]
        wp = inputs.config3(sigma=f[0], device="cuda")
        fb = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        rec = one_config(wp, f[1], lambda: fb.fill_(1), local_rank, n_steps=args.steps, warmup=args.warmup,
                         budget=int(f[2] * 2**30) if len(f) > 2 else SWEEP_GATHER_BUDGET, gather=f[3] if len(f) > 3 else None)
        rec["sigma"] = f[0]
        print(json.dumps({"config3_point": rec}))
        return

    # ------------------------------------------------------------------ prefill (the metric)
    wl = inputs.config2(variant=rank)
    eng = binding.AdaSAttn(cube=wl.cube, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.D,
                           top_p=wl.top_p, device=local_rank)
    eng.partition(wl.B, wl.T, wl.H, wl.W, wl.n_text)
    if args.prefill_kernel is not None:
        binding.adaspark_attn_set_prefill_kernel(eng.handle, args.prefill_kernel)
    binding.adaspark_attn_enable_stage_timing(eng.handle, True)
    q_h, k_h, v_h = wl.q.pin_memory(), wl.k.pin_memory(), wl.v.pin_memory()
    q, k, v = q_h.cuda(non_blocking=True), k_h.cuda(non_blocking=True), v_h.cuda(non_blocking=True)
    out = torch.empty_like(q)
    out_h = torch.empty_like(q_h).pin_memory()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # 2x the 126 MB L2

    def flush():
        flush_buf.fill_(1)

    sampler = ClockSampler(local_rank)
    sampler.start()                    # early: the first line of nvidia-smi takes a while
    parity = None
    if rank == 0 and not args.no_parity:
        parity = parity_check(wl, eng, q, k, v)

    def step():
        eng.forward(q, k, v, wl.n_text, out=out)
        return lambda: binding.adaspark_attn_get_stage_times(eng.handle) + [binding.adaspark_attn_get_attention_kernel_ms(eng.handle)]

    sampler.wait_first()
    times, stages = timed_steps(step, args.steps, args.warmup, flush, barrier, on_begin=sampler.begin, on_end=sampler.end)
    clocks = sampler.stop()
    launches_per_step = eng.launches()
    hdr = eng.header()
    ms = sum(times) / len(times)
    ms_max = max_over_ranks(ms, dist, "cuda")
    tokens = wl.B * wl.S
    value = job_throughput(tokens, world, ms_max)

    # selection statistics -> useful FLOPs (4 * D * sum over rows of attended keys)
    _, bitmap, count = eng.forward(q, k, v, wl.n_text, out=out, want_selection=True)
    torch.cuda.synchronize()
    sel_total = int(count.sum().item())
    # attended keys outside the selection: own-cube prefix (video rows) / text prefix (text rows)
    C = wl.C
    local = wl.S_v // C * (C * (C + 1) // 2) + wl.n_text * (wl.n_text + 1) // 2
    useful_flops = 4.0 * wl.D * (sel_total * C + wl.B * wl.Hq * local)
    executed_flops = float(hdr.executed_kv_blocks) * 128 * 64 * wl.D * 4
    dense_flops = 4.0 * wl.D * wl.B * wl.Hq * (wl.S * (wl.S + 1) / 2)
    st = np.asarray(stages)          # [steps, 5]: relayout, score+select, attention stage, -, the attention kernel alone
    st_mean = st.mean(axis=0)
    attn_ms = float(st_mean[2])
    attn_kernel_ms = float(st_mean[4])   # the stage also holds the six small kernels of the query-gather decision
    achieved_tflops = executed_flops / (attn_kernel_ms * 1e-3) / 1e12
    peak_tflops = peaks["bf16_tflops"]

    # ------------------------------------------------------------------ end to end (host buffers)
    # Every step goes through adaspark_attn_forward_host: the library copies q, k, v from pinned host
    # memory, runs the prefill and copies the output back, all on the stream it is given.  Three streams with
    # a device buffer set, caches and a workspace each take turns, so that the upload, the kernels and the
    # download of neighbouring steps overlap (a handle's buffers belong to one step at a time).
    # Time = first upload to last download, per step.
    lanes = [(eng, (q, k, v, out), torch.cuda.Stream(), out_h)]
    for _ in range(2):                                        # three lanes: upload, kernels and download of different steps overlap
        e_x = binding.AdaSAttn(cube=wl.cube, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.D,
                               top_p=wl.top_p, device=local_rank)
        e_x.partition(wl.B, wl.T, wl.H, wl.W, wl.n_text)
        if args.prefill_kernel is not None:
            binding.adaspark_attn_set_prefill_kernel(e_x.handle, args.prefill_kernel)
        lanes.append((e_x, tuple(torch.empty_like(t) for t in (q, k, v, out)), torch.cuda.Stream(),
                      torch.empty_like(out_h).pin_memory()))

    def e2e_pipelined(n_steps):
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        barrier()
        t0.record()
        for _, _, s_, _ in lanes:
            s_.wait_event(t0)
        for i in range(n_steps):
            e_, staging, s_, oh = lanes[i % len(lanes)]
            e_.forward_host(q_h, k_h, v_h, wl.n_text, oh, staging, stream=s_)
        for _, _, s_, _ in lanes:
            torch.cuda.current_stream().wait_stream(s_)
        t1.record()
        torch.cuda.synchronize()
        barrier()
        return t0.elapsed_time(t1) / n_steps

    e2e_pipelined(6)                                          # warm-up
    e2e_ms = e2e_pipelined(max(9, args.steps))
    e2e_value = job_throughput(tokens, world, max_over_ranks(e2e_ms, dist, "cuda"))
    assert torch.equal(lanes[1][3], out_h) and torch.equal(lanes[2][3], out_h), "the end-to-end lanes disagree"
    for e_x, _, _, _ in lanes[1:]:
        e_x.close()
    del lanes
    h2d = q_h.numel() * 2 + k_h.numel() * 2 + v_h.numel() * 2
    d2h = out_h.numel() * 2

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "tokens_per_step_per_gpu": tokens,
                   "cache_policy": "L2 flushed (256 MB write) before every timed step; inputs "
                                   "(~290 MB) also exceed the 126 MB L2",
                   "multi_gpu": "independent replicas, no collective"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"kernel": "attn_prefill_tc_kernel (prefill attention)", "kernel_ms": attn_kernel_ms, "bound": "tensor", "achieved": achieved_tflops,
                     "peak": peak_tflops, "unit": "TFLOP/s", "frac": achieved_tflops / peak_tflops,
                     "traffic": profiled_traffic("attn_prefill_tc.cuh", "attn_prefill_tc_kernel_config2.md"),
                     "traffic_unit": "bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum)",
                     "peak_source": f"{peaks['source']} bf16 burst (kernel of ~ms inside a ~ms step)"},
        "stages_ms": {"relayout_pool": float(st_mean[0]), "score_select": float(st_mean[1]),
                      "attention": attn_ms},
        "parity": parity,
        "flops": {"executed": executed_flops, "useful": useful_flops, "dense_causal": dense_flops,
                  "useful_over_executed": useful_flops / max(executed_flops, 1.0),
                  "effective_tflops_executed": executed_flops / (ms_max * 1e-3) / 1e12,
                  "mean_selected_cubes_per_row": sel_total / (wl.B * wl.Hq * wl.S)},
    }

    # ------------------------------------------------------------------ dense comparison
    if not args.no_dense and rank == 0:
        try:
            qd = q.permute(0, 2, 1, 3)
            kd, vd = k.permute(0, 2, 1, 3), v.permute(0, 2, 1, 3)

            def sdpa():
                torch.nn.functional.scaled_dot_product_attention(qd, kd, vd, is_causal=True,
                                                                 enable_gqa=True)
            sd_times, _ = timed_steps(lambda: sdpa() or None, 5, 3, flush, lambda: None)
            eng1 = binding.AdaSAttn(cube=wl.cube, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv,
                                    head_dim=wl.D, top_p=1.0, device=local_rank)
            eng1.partition(wl.B, wl.T, wl.H, wl.W, wl.n_text)
            if args.prefill_kernel is not None:
                binding.adaspark_attn_set_prefill_kernel(eng1.handle, args.prefill_kernel)
            p1_times, _ = timed_steps(lambda: eng1.forward(q, k, v, wl.n_text, out=out) and None,
                                      5, 3, flush, lambda: None)
            result["dense"] = {"torch_sdpa_causal_ms": sum(sd_times) / len(sd_times),
                               "own_p1_forward_ms": sum(p1_times) / len(p1_times),
                               "adas_forward_ms": ms_max}
            eng1.close()
            del eng1
        except Exception as e:  # comparison only
            result["dense"] = {"error": repr(e)[:200]}

    # ------------------------------------------------------------------ rooflines of the other stages
    # re-layout + pooling (K/V once in, once out, fp32 keys): an HBM-bound copy (Q is not re-laid out)
    relayout_bytes = 2 * (k.numel() + v.numel()) * 2 + wl.B * wl.Hkv * wl.N * wl.D * 4
    rl_gbs = relayout_bytes / (float(st_mean[0]) * 1e-3) / 1e9
    # scoring + selection: candidate (row, cube) pairs; algorithmic bytes = Q once + mean keys + mask words
    n_tiles = (wl.S + 127) // 128
    pos = np.arange(wl.S)
    cand_per_row = np.where(pos < wl.S_v, pos // C, wl.N)
    pairs = float(cand_per_row.sum()) * wl.B * wl.Hq
    ss_bytes = q.numel() * 2 + wl.B * wl.Hkv * wl.N * wl.D * 4 + wl.B * wl.Hq * n_tiles * 128 * ((wl.N + 31) // 32) * 4
    ss_ms = float(st_mean[1])
    result["stage_rooflines"] = {
        "relayout": {"bound": "hbm", "bytes": relayout_bytes, "ms": float(st_mean[0]), "achieved": rl_gbs,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": rl_gbs / peaks["hbm_gbs"]},
        "score_select": {"bound": "alu", "candidate_pairs": pairs, "ms": ss_ms,
                         "achieved": pairs / (ss_ms * 1e-3) / 1e9, "unit": "G candidate (row, cube) pairs/s",
                         "algorithmic_bytes": ss_bytes, "hbm_floor_ms": ss_bytes / (peaks["hbm_gbs"] * 1e9) * 1e3,
                         "useful_flops": 2.0 * wl.D * pairs},
    }

    # ------------------------------------------------------------------ cohesive queries (extra workload)
    # (measured here, next to the dense comparison it is set against, before the long sweep heats the part)
    if not args.no_cohesive and rank == 0:
        try:
            wc = inputs.config2_cohesive(top_p=0.7, cube=(4, 8, 8), device="cuda")
            engc = binding.AdaSAttn(cube=wc.cube, n_q_heads=wc.Hq, n_kv_heads=wc.Hkv, head_dim=wc.D,
                                    top_p=wc.top_p, device=local_rank)
            engc.partition(wc.B, wc.T, wc.H, wc.W, wc.n_text)
            binding.adaspark_attn_enable_stage_timing(engc.handle, True)
            outc = torch.empty_like(wc.q)

            def cstep():
                engc.forward(wc.q, wc.k, wc.v, wc.n_text, out=outc)
                return lambda: binding.adaspark_attn_get_stage_times(engc.handle)

            c_times, c_stages = timed_steps(cstep, 10, 3, flush, lambda: None)
            cst = np.asarray(c_stages).mean(axis=0)
            hc = engc.header()
            _, _, ccount = engc.forward(wc.q, wc.k, wc.v, wc.n_text, out=outc, want_selection=True)
            torch.cuda.synchronize()
            result["cohesive_queries"] = {
                "workload": "config-2 shapes, cube 4x8x8 (256 tokens, the paper's default size), p=0.7; the video "
                            "queries of a cube share an N(0,1) offset per head plus an own N(0,0.25) part",
                "forward_ms": sum(c_times) / len(c_times),
                "stages_ms": {"relayout_pool": float(cst[0]), "score_select": float(cst[1]),
                              "attention": float(cst[2])},
                "executed_over_dense_flops": float(hc.executed_kv_blocks) * 128 * 64 * wc.D * 4 / dense_flops,
                "mean_selected_cubes_per_row": float(ccount.float().mean().item()),
                "torch_sdpa_causal_ms": result.get("dense", {}).get("torch_sdpa_causal_ms"),
            }
            engc.close()
            del engc, wc, outc, ccount
        except Exception as e:  # extra workload only
            result["cohesive_queries"] = {"error": repr(e)[:200]}

    # ------------------------------------------------------------------ config 3 sweep and config 4
    if not args.no_sweep and rank == 0:
        try:
            del bitmap, count
            torch.cuda.empty_cache()
            sweep = []
            sdpa_ms = None
            for sigma in (0.5, 1.5, 3.0):
                w3 = inputs.config3(sigma=sigma, device="cuda")
                if sdpa_ms is None and not args.no_dense:
                    q3, k3, v3 = (t.permute(0, 2, 1, 3) for t in (w3.q, w3.k, w3.v))

                    def sdpa3():
                        torch.nn.functional.scaled_dot_product_attention(q3, k3, v3, is_causal=True, enable_gqa=True)

                    sd3, _ = timed_steps(sdpa3, 3, 3, flush, lambda: None)
                    del q3, k3, v3
                    sdpa_ms = sum(sd3) / len(sd3)
                recs = {p: one_config(w3, p, flush, local_rank) for p in (1.0, 0.95, 0.9, 0.7, 0.5)}
                for p in (0.5, 0.7, 0.9, 0.95, 1.0):
                    r3 = recs[p]
                    if r3["gather"]["pair_tiles"] > 0:     # the same point with every pair on the union path
                        ru = one_config(w3, p, flush, local_rank, n_steps=2, gather=0.0)
                        r3["union_path_only"] = {"forward_ms": ru["forward_ms"], "attention_ms": ru["stages_ms"]["attention"],
                                                 "useful_over_executed": ru["useful_over_executed"]}
                    r3["sigma"] = sigma
                    r3["speedup_vs_own_p1"] = recs[1.0]["forward_ms"] / r3["forward_ms"]
                    r3["speedup_vs_torch_sdpa"] = sdpa_ms / r3["forward_ms"] if sdpa_ms else None
                    sweep.append(r3)
                del w3
                torch.cuda.empty_cache()
            result["config3_sweep"] = {"workload": "config3: 256x16x16 video tokens (1024 cubes) + 256 text, 28/4 heads, "
                                                   "head_dim 128; p=1.0 is the dense reference of the same kernels",
                                       "gather": {"pairs_per_block": GATHER_DEFAULT_THRESHOLD, "budget_gib": SWEEP_GATHER_BUDGET >> 30},
                                       "torch_sdpa_causal_ms": sdpa_ms, "points": sweep}
            w4 = inputs.config4(device="cuda")
            r4 = one_config(w4, w4.top_p, flush, local_rank, n_steps=2)
            r4["workload"] = "config4: 512x16x16 video tokens (2048 cubes), first half of the frames static, p=0.9"
            r4["tokens_per_s"] = w4.B * w4.S / (r4["forward_ms"] * 1e-3)
            result["config4"] = r4
            del w4
            torch.cuda.empty_cache()
        except Exception as e:  # extra measurements only
            result["config3_sweep"] = {"error": repr(e)[:300]}

    # ------------------------------------------------------------------ decode (config 5)
    if not args.no_decode:
        del q, k, v, out
        torch.cuda.empty_cache()
        wd = inputs.config5(variant=rank, B=args.decode_batch, device="cuda")
        engd = binding.AdaSAttn(cube=wd.cube, n_q_heads=wd.Hq, n_kv_heads=wd.Hkv, head_dim=wd.D,
                                top_p=wd.top_p, device=local_rank)
        engd.partition(wd.B, wd.T, wd.H, wd.W, wd.n_text)
        engd.forward(None, wd.k, wd.v, wd.n_text)
        torch.cuda.synchronize()
        wd.k = wd.v = None
        torch.cuda.empty_cache()
        binding.adaspark_attn_enable_stage_timing(engd.handle, True)
        tl = torch.full((wd.B,), wd.n_text, dtype=torch.int32, device="cuda")
        od = torch.empty_like(wd.q_new)

        def dstep():
            engd.decode(wd.q_new, wd.k_new, wd.v_new, tl, out=od)
            return lambda: binding.adaspark_attn_get_stage_times(engd.handle)

        d_times, d_stages = timed_steps(dstep, args.steps, args.warmup, flush, barrier)
        d_ms = sum(d_times) / len(d_times)
        d_ms = max_over_ranks(d_ms, dist, "cuda")
        hd = engd.header()
        gathered = float(hd.decode_kv_blocks) * 2 * 64 * wd.D * 2
        keys_bytes = wd.B * wd.Hkv * wd.N * wd.D * 4
        dst = np.asarray(d_stages).mean(axis=0)
        split_ms = float(dst[2])
        result["decode"] = {
            "workload": f"config5: batch {wd.B}, 131072-token video cache (2048 cubes) + 512 text, "
                        "28/4 heads, head_dim 128, p=0.9",
            "queries_per_s": world * wd.B / (d_ms * 1e-3), "ms_per_step": d_ms,
            "gathered_kv_bytes": gathered, "cube_key_bytes": keys_bytes,
            "gathered_fraction_of_cache": gathered / (wd.B * wd.Hkv * (wd.S_v + wd.n_text + 1) * wd.D * 4),
            "hbm_gbs_step": (gathered + keys_bytes) / (d_ms * 1e-3) / 1e9,
            "splitkv_kernel": {"ms": split_ms, "achieved_gbs": gathered / (split_ms * 1e-3) / 1e9,
                               "peak_gbs": peaks["hbm_gbs"],
                               "frac": gathered / (split_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "stages_ms": {"append": float(dst[0]), "score_select_plan": float(dst[1]),
                          "splitkv": split_ms, "combine": float(dst[3])},
            "gpu_launches": engd.launches() * args.steps,
        }

    # ------------------------------------------------------------------ CPU baseline (oracle)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl)

    if rank == 0:
        print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
