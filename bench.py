#!/usr/bin/env python
"""Benchmark of the attention hot path on B200: prefill TFLOP/s and decode HBM GB/s vs roofline.

One "step" is one pass of the whole hot path at the 8B-shaped sizes (Hq=32, Hkv=8, D=128):
  1. l4l_attn_prefill   causal prefill B=4, S=8192 with the KV cache written in the same pass
  2. l4l_kv_append      the current token's K/V of B=32 ragged sequences (512..4096 cached tokens)
  3. l4l_attn_decode    one query token per sequence over that ragged cache (split + merge)
`value` is the step's attention FLOPs (causal pairs only for prefill) divided by the step's time,
summed over GPUs; the per-kernel roofline fractions (tensor peak for prefill, HBM for decode) are
in `roofline` / `roofline_decode`. Inputs are seeded synthetic bf16 (see workloads.py).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
Under torchrun every rank runs the same step on its own GPU (sequences shard with no exchange).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_21836_b200 import workloads as wl  # noqa: E402

METRIC = "decode-attn HBM GB/s & prefill-attn TFLOP/s, each as % of B200 peak"
NOMINAL_TFLOPS, NOMINAL_GBS = 2250.0, 8000.0
FALLBACK_TFLOPS, FALLBACK_GBS = 1590.0, 6650.0
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/: prefill captured at B=1,S=8192 (160.2 MB) and scaled x4 to the bench's B=4 (traffic is proportional
# to B); decode captured on the bench's own batch.
NCU_TRAFFIC_PREFILL = 640.8e6   # 4 x (102.1 MB read + 58.1 MB written)
NCU_TRAFFIC_DECODE = 302.2e6    # 297.8 MB read + 4.4 MB written


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            mp = json.load(f)
        return {"hbm_gbs": float(mp["hbm_gbs"]), "bf16_tflops": float(mp["bf16_tflops"]),
                "bf16_tflops_sustained": float(mp.get("bf16_tflops_sustained", mp["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": FALLBACK_GBS, "bf16_tflops": FALLBACK_TFLOPS, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------------- multi-rank bookkeeping
def max_over_ranks(values, world: int, device="cpu"):
    """Every timing is the MAX over ranks (the job is as slow as its slowest replica). Works on any backend:
    NCCL with CUDA tensors in the benchmark, gloo with CPU tensors in the tests."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(world: int, step_flops: float, ms_per_step: float) -> float:
    """Aggregate throughput of `world` replicas, each doing `step_flops` per step (weak scaling), in TFLOP/s."""
    return world * step_flops / (ms_per_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------------- workload
def make_inputs():
    wp, wd = wl.WORKLOADS["long_prefill"], wl.WORKLOADS["batched_decode"]
    seq = wl.make_sequence(wp)
    db = wl.make_decode_batch(wd)
    g = torch.Generator().manual_seed(wd.seed + 7)
    k_new = torch.randn(wd.decode_B, 1, wd.Hkv, wd.D, generator=g).to(torch.bfloat16)
    v_new = torch.randn(wd.decode_B, 1, wd.Hkv, wd.D, generator=g).to(torch.bfloat16)
    return wp, wd, seq, db, k_new, v_new


def step_work(wp, wd, seq, db):
    pre_flops = wl.prefill_flops(wp.Hq, wp.D, [seq.S] * wp.prefill_B)
    dec_bytes = wl.decode_kv_bytes(wd.Hkv, wd.D, db.kv_len.tolist())
    dec_flops = 4 * wd.D * wd.Hq * int(db.kv_len.sum())
    return pre_flops, dec_bytes, dec_flops


def workload_name(wp, wd):
    return (f"8b_shaped: long_prefill(B={wp.prefill_B},S={wp.prefill_S},Hq={wp.Hq},Hkv={wp.Hkv},D={wp.D},cache write) + "
            f"batched_decode(B={wd.decode_B},kv_len~U[{wd.decode_len_lo},{wd.decode_len_hi}],append+decode)")


# ----------------------------------------------------------------------------------- oracle timing
def time_oracle_sample(wp, wd, seq, db, budget_s: float = 12.0):
    """Times the CPU oracle, as it stands, on a bounded sample of the step: a stratified set of prefill
    rows (grown until about budget_s of work) and the whole decode batch. Returns work and seconds."""
    from oracle import l4l_oracle as orc

    B, S, Hq, D = wp.prefill_B, seq.S, wp.Hq, wp.D
    lens = np.full(B, S, np.int32)
    rng = np.random.default_rng(2024)

    def rows(n):
        return np.stack([rng.integers(0, B, n), rng.integers(0, S, n), rng.integers(0, Hq, n)], axis=1).astype(np.int32)

    probe = rows(512)
    t0 = time.perf_counter()
    orc.prefill_rows(seq.q, seq.k, seq.v, lens, wp.scale, probe)
    t_probe = time.perf_counter() - t0
    n = int(min(200000, max(512, 512 * (0.7 * budget_s) / max(t_probe, 1e-3))))
    sample = rows(n)
    t0 = time.perf_counter()
    orc.prefill_rows(seq.q, seq.k, seq.v, lens, wp.scale, sample)
    t_pre = time.perf_counter() - t0
    pre_flops = int(4 * D * (sample[:, 1].astype(np.int64) + 1).sum())
    t0 = time.perf_counter()
    orc.decode(db.q, db.cache_k, db.cache_v, db.kv_len.numpy(), wd.scale)
    t_dec = time.perf_counter() - t0
    dec_bytes = wl.decode_kv_bytes(wd.Hkv, wd.D, db.kv_len.tolist())
    dec_flops = 4 * wd.D * wd.Hq * int(db.kv_len.sum())
    return {"pre_flops": pre_flops, "t_pre": t_pre, "rows": n, "dec_bytes": dec_bytes, "dec_flops": dec_flops,
            "t_dec": t_dec, "cores": orc.num_threads()}


def cpu_baseline_obj(s):
    total_t = s["t_pre"] + s["t_dec"]
    return {
        "value": (s["pre_flops"] + s["dec_flops"]) / total_t / 1e12, "unit": "TFLOP/s", "cores": s["cores"],
        "kind": "oracle",
        "sample": (f"{s['rows']} random (b,i,h) rows of the B=4,S=8192 causal prefill ({s['t_pre']:.1f} s) + the whole "
                   f"B=32 ragged decode batch ({s['t_dec']:.1f} s), fp64 C oracle with OpenMP"),
        "prefill_gflops": s["pre_flops"] / s["t_pre"] / 1e9,
        "decode_gbs": s["dec_bytes"] / s["t_dec"] / 1e9,
    }


def run_reference(args, rank, world=1):
    """--impl reference: the oracle, as it stands, on the host cores; each step is a bounded sample. It is a CPU
    program: under a multi-rank launch rank 0 alone runs and prints it, the other ranks leave without work."""
    if rank != 0:
        return
    wp, wd, seq, db, _, _ = make_inputs()
    per_step_budget = max(2.0, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        time_oracle_sample(wp, wd, seq, db, budget_s=min(2.0, per_step_budget))
    tot_fl, tot_t, last = 0.0, 0.0, None
    for _ in range(args.steps):
        last = time_oracle_sample(wp, wd, seq, db, budget_s=per_step_budget)
        tot_fl += last["pre_flops"] + last["dec_flops"]
        tot_t += last["t_pre"] + last["t_dec"]
    value = tot_fl / tot_t / 1e12
    cb = cpu_baseline_obj(last)
    cb["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "ranks_launched": world, "ranks_that_ran_the_oracle": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_t / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wp, wd), "note": "each step is a bounded sample of the workload"},
        "cpu_baseline": cb,
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ----------------------------------------------------------------------------------- our arm
def run_ours(args, rank, world):
    import torch.distributed as dist
    from paper_2608_21836_b200 import binding as l4l

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    l4l.load()

    wp, wd, seq, db, k_new, v_new = make_inputs()
    pre_flops, dec_bytes, dec_flops = step_work(wp, wd, seq, db)
    Bp, S, Hq, Hkv, D = wp.prefill_B, seq.S, wp.Hq, wp.Hkv, wp.D
    Bd, Lmax = wd.decode_B, wd.decode_Lmax

    # device-resident inputs
    q, k, v = seq.q.to(dev), seq.k.to(dev), seq.v.to(dev)
    o = torch.empty_like(q)
    pk = torch.empty(Bp, Hkv, S, D, dtype=torch.bfloat16, device=dev)
    pv = torch.empty_like(pk)
    plens = torch.full((Bp,), S, dtype=torch.int32, device=dev)
    ws_p = l4l.new_workspace(l4l.L4L_OP_PREFILL, Bp, Hq, Hkv, D, S, device=dev)
    dq, dck, dcv = db.q.to(dev), db.cache_k.to(dev), db.cache_v.to(dev)
    dlen = db.kv_len.to(dev)
    dpos = (db.kv_len - 1).to(torch.int32).to(dev)
    dkn, dvn = k_new.to(dev), v_new.to(dev)
    do = torch.empty_like(dq)
    ws_d = l4l.new_workspace(l4l.L4L_OP_DECODE, Bd, Hq, Hkv, D, Lmax, device=dev)

    def step(ev=None):
        if ev: ev[0].record()
        l4l.l4l_attn_prefill(q, k, v, o, plens, wp.scale, ws_p, cache_k=pk, cache_v=pv)
        if ev: ev[1].record()
        l4l.l4l_kv_append(dck, dcv, dkn, dvn, dpos)
        if ev: ev[2].record()
        l4l.l4l_attn_decode(dq, do, dck, dcv, dlen, Lmax, wd.scale, ws_d)
        if ev: ev[3].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    # ---- the decode kernel alone, over three rotating copies of the cache (1.6 GB, so every launch streams from
    # HBM), timed three ways:
    #   overlapped  N launches back to back between ONE pair of events: with programmatic stream serialization the
    #               prologue of a launch runs under the tail of the one before, so this mean is a pipelined rate
    #   pairs       the same loop with an event pair around every launch (median and best of the per-launch times)
    #   single      one launch alone: a pass over 1 GiB first (flushes L2, and keeps the GPU busy until the host has
    #               the launch and both events queued), then event, launch, event; median and best over repeats
    caches = [(dck, dcv)] + [(dck.clone(), dcv.clone()) for _ in range(2)]
    n_dec = max(60, args.steps)
    for i in range(3):
        l4l.l4l_attn_decode(dq, do, caches[i][0], caches[i][1], dlen, Lmax, wd.scale, ws_d)
    barrier()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # a few milliseconds of unrelated GPU work queued first, so that the host has every launch of the timed
    # run enqueued before the GPU reaches it: the figure is device time, not Python call overhead
    filler = torch.empty(1 << 28, dtype=torch.float32, device=dev)
    for _ in range(6):
        filler.zero_()
    d0.record()
    for i in range(n_dec):
        ck_i, cv_i = caches[i % 3]
        l4l.l4l_attn_decode(dq, do, ck_i, cv_i, dlen, Lmax, wd.scale, ws_d)
    d1.record()
    barrier()
    t_dec_b2b = d0.elapsed_time(d1) / n_dec

    def launch_times(fn, n, alone, flush="read"):
        """Per-launch device times (ms) of n calls of fn(i): back to back with an event pair around each, or each
        one alone behind an L2 flush over 1 GiB. flush = "read" (a reduction over the buffer: L2 ends up full of
        clean lines, so the launch sees a cold cache and nothing else) or "write" (a memset: L2 ends up full of
        DIRTY lines, whose write-back to HBM then competes with the launch's own traffic, as it does behind any
        kernel that has just written a large output)."""
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        if not alone:
            for _ in range(6):
                filler.zero_()
        for i, (a, b) in enumerate(pairs):
            if alone:
                filler.sum() if flush == "read" else filler.zero_()
            a.record()
            fn(i)
            b.record()
        barrier()
        return sorted(a.elapsed_time(b) for a, b in pairs)

    def decode_i(i):
        l4l.l4l_attn_decode(dq, do, caches[i % 3][0], caches[i % 3][1], dlen, Lmax, wd.scale, ws_d)

    dec_pairs = launch_times(decode_i, n_dec, alone=False)
    dec_single = launch_times(decode_i, 30, alone=True)
    dec_single_dirty = launch_times(decode_i, 30, alone=True, flush="write")
    sampler = ClockSampler(local)
    sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin.record()
    for i in range(args.steps):
        step(evs[i])
    t_end.record()
    barrier()
    clocks = sampler.stop()
    total_ms = t_begin.elapsed_time(t_end)
    pre_times = sorted(e[0].elapsed_time(e[1]) for e in evs)
    t_pre = float(np.mean(pre_times))
    t_app = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    t_dec = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))

    pre_single = launch_times(lambda i: l4l.l4l_attn_prefill(q, k, v, o, plens, wp.scale, ws_p, cache_k=pk, cache_v=pv),
                              8, alone=True)
    del caches

    # ---- the widened entry points, each timed alone after the same kind of filler (not part of the step):
    # rope + norm + cache update of the whole prompt (one streaming pass), attention of the prompt read from the
    # cache layout (the chunk entry with nothing cached before), and the decode step with the cache update fused
    def timed(fn, n):
        for _ in range(2):
            fn()
        barrier()
        for _ in range(4):
            filler.zero_()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(n):
            fn()
        a1.record()
        barrier()
        return a0.elapsed_time(a1) / n

    cos, sin = wl.make_rope_tables(S, D)
    cos, sin = cos.to(dev), sin.to(dev)
    gamma = torch.ones(D, dtype=torch.float32, device=dev)
    q_rot = q.clone()
    zeros_b = torch.zeros(Bp, dtype=torch.int32, device=dev)
    t_rope = timed(lambda: l4l.l4l_rope_kv_append(q_rot, k, v, pk, pv, zeros_b, None, cos, sin, gamma, gamma, 1e-6), 10)
    del q_rot
    rope_bytes = 2 * q.numel() * 2 + 2 * (k.numel() + v.numel()) * 2       # q read + written, k/v read, cache written
    t_chunk = timed(lambda: l4l.l4l_attn_prefill_chunk(q, o, pk, pv, zeros_b, plens, wp.scale, ws_p), 5)
    # a chunk of 4096 new tokens per sequence over 4096 cached ones, the chunk's K/V written by the same launch
    half = S // 2
    past_b = torch.full((Bp,), half, dtype=torch.int32, device=dev)
    qlen_b = torch.full((Bp,), half, dtype=torch.int32, device=dev)
    t_chunk_append = timed(lambda: l4l.l4l_attn_prefill_chunk_append(q[:, half:], k[:, half:], v[:, half:], o[:, half:], pk, pv,
                                                                     past_b, qlen_b, wp.scale, ws_p), 5)
    chunk_flops = 4 * D * Hq * Bp * (half * half + half * (half + 1) // 2)
    t_fused = timed(lambda: l4l.l4l_attn_decode_append(dq, do, dck, dcv, dkn, dvn, dlen, Lmax, wd.scale, ws_d), 20)
    # the whole decode step of a layer: rope + norm of the new token's q and k, append, attention: one launch, against
    # the three launches rope_kv_append (T = 1) + decode
    cos_d, sin_d = wl.make_rope_tables(Lmax, D)
    cos_d, sin_d = cos_d.to(dev), sin_d.to(dev)
    t_step1 = timed(lambda: l4l.l4l_attn_decode_rope_append(dq, do, dck, dcv, dkn, dvn, dlen, Lmax, wd.scale, cos_d, sin_d,
                                                            ws_d, q_weight=gamma, k_weight=gamma, eps=1e-6), 20)
    dq4 = dq.view(Bd, 1, Hq, D)

    def three_launches():
        l4l.l4l_rope_kv_append(dq4, dkn, dvn, dck, dcv, dpos, None, cos_d, sin_d, gamma, gamma, 1e-6)
        l4l.l4l_attn_decode(dq, do, dck, dcv, dlen, Lmax, wd.scale, ws_d)

    t_step3 = timed(three_launches, 20)
    # decode over a paged cache: the same batch cut into 64-token pages scattered over a pool, three pools in rotation
    page = 64
    n_per = Lmax // page
    pools = []
    for i in range(3):
        perm = torch.randperm(Bd * n_per, generator=torch.Generator().manual_seed(7 + i)).to(dev)
        pool_k = torch.empty(Bd * n_per, Hkv, page, D, dtype=torch.bfloat16, device=dev)
        pool_v = torch.empty_like(pool_k)
        pool_k[perm] = dck.view(Bd, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(Bd * n_per, Hkv, page, D)
        pool_v[perm] = dcv.view(Bd, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(Bd * n_per, Hkv, page, D)
        pools.append((pool_k, pool_v, perm.view(Bd, n_per).to(torch.int32).contiguous()))
    rot = [0]

    def paged_step():
        pk_i, pv_i, tbl_i = pools[rot[0] % 3]
        rot[0] += 1
        l4l.l4l_attn_decode_paged(dq, do, pk_i, pv_i, tbl_i, dlen, Lmax, wd.scale, ws_d)

    t_paged = timed(paged_step, 21)

    def paged_fused_step():                                   # the same with the cache update of the step fused in
        pk_i, pv_i, tbl_i = pools[rot[0] % 3]
        rot[0] += 1
        l4l.l4l_attn_decode_paged_append(dq, do, pk_i, pv_i, tbl_i, dkn, dvn, dlen, Lmax, wd.scale, ws_d)

    t_paged_fused = timed(paged_fused_step, 21)
    del pools
    # decode over an fp8 (e4m3) cache: the same batch quantised by the library's own append (N(0,1) data, 4.5 sigma
    # at full scale), three copies in rotation
    k_sc = torch.full((Hkv,), 4.5 / 448, dtype=torch.float32, device=dev)
    c8 = []
    for i in range(3):
        k8 = torch.zeros(Bd, Hkv, Lmax, D, dtype=torch.uint8, device=dev)
        v8 = torch.zeros_like(k8)
        l4l.l4l_kv_append_fp8(k8, v8, torch.nan_to_num(dck.float()).to(torch.bfloat16).permute(0, 2, 1, 3),
                              torch.nan_to_num(dcv.float()).to(torch.bfloat16).permute(0, 2, 1, 3),
                              torch.zeros(Bd, dtype=torch.int32, device=dev), k_sc, k_sc)
        c8.append((k8, v8))

    def fp8_step():
        k8, v8 = c8[rot[0] % 3]
        rot[0] += 1
        l4l.l4l_attn_decode_fp8(dq, do, k8, v8, k_sc, k_sc, dlen, Lmax, wd.scale, ws_d)

    t_fp8 = timed(fp8_step, 21)

    def fp8_fused_step():                                     # the new token quantised and appended in the same launch
        k8, v8 = c8[rot[0] % 3]
        rot[0] += 1
        l4l.l4l_attn_decode_append_fp8(dq, do, k8, v8, k_sc, k_sc, dkn, dvn, dlen, Lmax, wd.scale, ws_d)

    t_fp8_fused = timed(fp8_fused_step, 21)

    def fp8_rope_step():                                      # ... and with rope + norm of the new token's q and k fused in too
        k8, v8 = c8[rot[0] % 3]
        rot[0] += 1
        l4l.l4l_attn_decode_rope_append_fp8(dq, do, k8, v8, k_sc, k_sc, dkn, dvn, dlen, Lmax, wd.scale, cos_d, sin_d, ws_d,
                                            q_weight=gamma, k_weight=gamma, eps=1e-6)

    t_fp8_rope = timed(fp8_rope_step, 21)
    del c8
    # the same cache with 64 query heads on the 8 KV heads (groups of 8: the 70B-class shape), three copies in rotation
    Hq8 = 8 * Hkv
    dq8 = torch.randn(Bd, Hq8, D, generator=torch.Generator().manual_seed(9)).to(torch.bfloat16).to(dev)
    do8 = torch.empty_like(dq8)
    ws_d8 = l4l.new_workspace(l4l.L4L_OP_DECODE, Bd, Hq8, Hkv, D, Lmax, device=dev)
    c3 = [(dck, dcv)] + [(dck.clone(), dcv.clone()) for _ in range(2)]

    def g8_step():
        ck_i, cv_i = c3[rot[0] % 3]
        rot[0] += 1
        l4l.l4l_attn_decode(dq8, do8, ck_i, cv_i, dlen, Lmax, wd.scale, ws_d8)

    t_g8 = timed(g8_step, 21)
    err_g8 = l4l.l4l_last_device_error(ws_d8)
    del c3
    # The decode phase of the 8B-shaped layer config (B = 1, 2048-token prompt, 256 steps): latency-bound, so the
    # steps (cache update fused in) are replayed from a CUDA graph, as a serving loop would issue them; once on the
    # kernel the library picks for this size (a thread-block cluster per KV head) and once held on the split kernel.
    def small_batch_step_us(L, split_only, n=64):
        w8 = wl.WORKLOADS["layer8b"]
        sb = wl.make_decode_batch(w8, B=1, len_lo=L, len_hi=L, Lmax=L, poison_tail=False)
        sq, sck, scv, slen = sb.q.to(dev), sb.cache_k.to(dev), sb.cache_v.to(dev), sb.kv_len.to(dev)
        skn = torch.zeros(1, 1, w8.Hkv, w8.D, dtype=torch.bfloat16, device=dev)
        so = torch.empty_like(sq)
        sws = l4l.new_workspace(l4l.L4L_OP_DECODE, 1, w8.Hq, w8.Hkv, w8.D, L, device=dev)
        with l4l.decode_override(cluster=0 if split_only else -1):
            fn = lambda: l4l.l4l_attn_decode_append(sq, so, sck, scv, skn, skn, slen, L, w8.scale, sws)
            side = torch.cuda.Stream(dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                for _ in range(n):
                    fn()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(5):
            graph.replay()
        a1.record()
        torch.cuda.synchronize()
        err = l4l.l4l_last_device_error(sws)
        return a0.elapsed_time(a1) / (5 * n) * 1e3, err

    # hundreds of short sequences (B = 512 with 64 to 256 cached tokens, 338 MB > L2, three copies in rotation): the
    # library's choice (a warp per (sequence, KV head)) and the same call held on the split kernel
    def short_batch_us(split_only):
        sb = wl.make_decode_batch(wd, B=512, len_lo=64, len_hi=256, Lmax=256, poison_tail=False)
        nbytes = wl.decode_kv_bytes(wd.Hkv, wd.D, sb.kv_len.tolist())
        cp = [(sb.cache_k.to(dev), sb.cache_v.to(dev)) for _ in range(3)]
        sq, slen = sb.q.to(dev), sb.kv_len.to(dev)
        so = torch.empty_like(sq)
        sws = l4l.new_workspace(l4l.L4L_OP_DECODE, 512, wd.Hq, wd.Hkv, wd.D, 256, device=dev)
        with l4l.decode_override(warp=0 if split_only else -1):
            def step():
                ck_i, cv_i = cp[rot[0] % 3]
                rot[0] += 1
                l4l.l4l_attn_decode(sq, so, ck_i, cv_i, slen, 256, wd.scale, sws)
            t = timed(step, 21)
        return t, nbytes, l4l.l4l_last_device_error(sws)

    t_short, short_bytes, err_short = short_batch_us(False)
    t_short_split, _, err_short2 = short_batch_us(True)
    # the other configurations of the workload list, each as its own kernel timing: the prefill of the 8B-shaped layer
    # config (B = 1, S = 2048) and of the small MHA model (B = 8, S = 512, head_dim 64), and the MHA decode batch
    # (B = 64 at context 1024; 201 MB, three cache copies in rotation)
    def other_prefill(name):
        w2 = wl.WORKLOADS[name]
        sq = wl.make_sequence(w2, T=0)
        q2, k2, v2 = sq.q.to(dev), sq.k.to(dev), sq.v.to(dev)
        o2 = torch.empty_like(q2)
        B2, S2 = q2.shape[0], q2.shape[1]
        ck2 = torch.empty(B2, w2.Hkv, S2, w2.D, dtype=torch.bfloat16, device=dev)
        cv2 = torch.empty_like(ck2)
        l2 = torch.full((B2,), S2, dtype=torch.int32, device=dev)
        ws2 = l4l.new_workspace(l4l.L4L_OP_PREFILL, B2, w2.Hq, w2.Hkv, w2.D, S2, device=dev)
        fn = lambda: l4l.l4l_attn_prefill(q2, k2, v2, o2, l2, w2.scale, ws2, cache_k=ck2, cache_v=cv2)
        t = timed(fn, 20)
        single = launch_times(lambda i: fn(), 20, alone=True)
        fl = wl.prefill_flops(w2.Hq, w2.D, [S2] * B2)
        return {"us": t * 1e3, "tflops": fl / (t * 1e-3) / 1e12, "timing": "mean of 20 back-to-back launches",
                "single_launch_us": {"median": single[len(single) // 2] * 1e3, "best": single[0] * 1e3},
                "single_launch_tflops": fl / (single[len(single) // 2] * 1e-3) / 1e12,
                "pct_nominal_2250": 100 * fl / (t * 1e-3) / 1e12 / NOMINAL_TFLOPS,
                "device_error": l4l.l4l_last_device_error(ws2)}

    def other_decode(name):
        w2 = wl.WORKLOADS[name]
        sb = wl.make_decode_batch(w2, poison_tail=False)
        nbytes = wl.decode_kv_bytes(w2.Hkv, w2.D, sb.kv_len.tolist())
        cp = [(sb.cache_k.to(dev), sb.cache_v.to(dev)) for _ in range(3)]
        q2, l2 = sb.q.to(dev), sb.kv_len.to(dev)
        o2 = torch.empty_like(q2)
        ws2 = l4l.new_workspace(l4l.L4L_OP_DECODE, w2.decode_B, w2.Hq, w2.Hkv, w2.D, w2.decode_Lmax, device=dev)

        def step():
            ck_i, cv_i = cp[rot[0] % 3]
            rot[0] += 1
            l4l.l4l_attn_decode(q2, o2, ck_i, cv_i, l2, w2.decode_Lmax, w2.scale, ws2)
        t = timed(step, 21)
        single = launch_times(lambda i: step(), 21, alone=True)
        # the same batch over an fp8 cache (quantised by the library's own append)
        sc2 = torch.full((w2.Hkv,), 4.5 / 448, dtype=torch.float32, device=dev)
        cp8 = []
        for ck_i, cv_i in cp:
            k8 = torch.zeros(ck_i.shape, dtype=torch.uint8, device=dev)
            v8 = torch.zeros_like(k8)
            l4l.l4l_kv_append_fp8(k8, v8, ck_i.permute(0, 2, 1, 3), cv_i.permute(0, 2, 1, 3),
                                  torch.zeros(ck_i.shape[0], dtype=torch.int32, device=dev), sc2, sc2)
            cp8.append((k8, v8))

        def step8():
            k8, v8 = cp8[rot[0] % 3]
            rot[0] += 1
            l4l.l4l_attn_decode_fp8(q2, o2, k8, v8, sc2, sc2, l2, w2.decode_Lmax, w2.scale, ws2)
        t8 = timed(step8, 21)
        return {"us": t * 1e3, "kv_gbs": nbytes / (t * 1e-3) / 1e9, "timing": "mean of 21 back-to-back launches",
                "single_launch_us": {"median": single[len(single) // 2] * 1e3, "best": single[0] * 1e3},
                "single_launch_kv_gbs": nbytes / (single[len(single) // 2] * 1e-3) / 1e9,
                "fp8_cache_us": t8 * 1e3, "fp8_cache_kv_gbs_fp8_bytes": nbytes / 2 / (t8 * 1e-3) / 1e9,
                "device_error": l4l.l4l_last_device_error(ws2)}

    other = {"layer8b_prefill_B1_S2048": other_prefill("layer8b"), "mha_small_prefill_B8_S512": other_prefill("mha_small"),
             "mha_small_decode_B64_L1024": other_decode("mha_small")}
    err_other = 0
    for v_ in other.values():
        err_other |= v_.pop("device_error")
    t_small, err_small = small_batch_step_us(2304, False)
    t_small_split, err_small2 = small_batch_step_us(2304, True)
    # second workload: the RG-LRU recurrence of a RecurrentGemma-2B-sized block (2560 channels) over a long prompt
    rB, rT, rW = 4, 8192, 2560
    gen = torch.Generator(device="cpu").manual_seed(1006)
    rx = torch.randn(rB, rT, rW, generator=gen).to(torch.bfloat16).to(dev)
    rgx = (torch.randn(rB, rT, rW, generator=gen) * 2).to(torch.bfloat16).to(dev)
    rga = (torch.randn(rB, rT, rW, generator=gen) * 2).to(torch.bfloat16).to(dev)
    r_ap = torch.log(torch.expm1(-torch.log(torch.rand(rW, generator=gen) * 0.099 + 0.9) / 8)).float().to(dev)
    r_state = torch.zeros(rB, rW, dtype=torch.float32, device=dev)
    ry = torch.empty_like(rx)
    ws_r = l4l.new_rglru_workspace(rB, rT, rW, device=dev)
    t_rglru = timed(lambda: l4l.l4l_rglru_scan(rx, rgx, rga, r_ap, r_state, ry, ws_r), 10)
    rglru_bytes = rx.numel() * 8                          # 3 bf16 read + 1 written per (step, channel)
    dev_err_r = l4l.l4l_last_device_error(ws_r)
    # the same bytes as 16 sequences of 2048 steps: 640 CTAs instead of 160 (which is 148 SMs + 12: the 12 SMs that
    # get a second CTA set the time of the B=4 case)
    rB2, rT2 = 16, 2048
    r_state2 = torch.zeros(rB2, rW, dtype=torch.float32, device=dev)
    ws_r2 = l4l.new_rglru_workspace(rB2, rT2, rW, device=dev)
    v2 = lambda t: t.view(rB2, rT2, rW)
    t_rglru2 = timed(lambda: l4l.l4l_rglru_scan(v2(rx), v2(rgx), v2(rga), r_ap, r_state2, v2(ry), ws_r2), 10)
    dev_err_r |= l4l.l4l_last_device_error(ws_r2)
    # two long sequences: 80 strips, fewer than SMs, so the kernel runs its 16-warp teams (one CTA per SM)
    rB3 = 2
    r_state3 = torch.zeros(rB3, rW, dtype=torch.float32, device=dev)
    ws_r3 = l4l.new_rglru_workspace(rB3, rT, rW, device=dev)
    t_rglru3 = timed(lambda: l4l.l4l_rglru_scan(rx[:rB3], rgx[:rB3], rga[:rB3], r_ap, r_state3, ry[:rB3], ws_r3), 10)
    dev_err_r |= l4l.l4l_last_device_error(ws_r3)
    del rx, rgx, rga, ry, filler
    dev_err = l4l.l4l_last_device_error(ws_p) | l4l.l4l_last_device_error(ws_d) | dev_err_r | err_small | err_small2 | err_g8 | err_short | err_short2 | err_other

    # ---- end to end through the same entry points with HOST buffers (pinned), copies inside the timed region
    hq, hk, hv = seq.q.pin_memory(), seq.k.pin_memory(), seq.v.pin_memory()
    ho = torch.empty_like(hq).pin_memory()
    hdq, hkn, hvn = db.q.pin_memory(), k_new.pin_memory(), v_new.pin_memory()
    hdo = torch.empty_like(hdq).pin_memory()
    h2d = sum(t.numel() * 2 for t in (hq, hk, hv, hdq, hkn, hvn))
    d2h = sum(t.numel() * 2 for t in (ho, hdo))

    # Two sets of device buffers and three streams (copy in, compute, copy out), as a serving loop would run it:
    # the copies of step n+1 and of step n-1 travel while step n computes (PCIe is full duplex). Every step still
    # moves all of its inputs from pinned host memory and all of its outputs back, inside the timed region.
    s_in, s_comp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    sets = [dict(q=q, k=k, v=v, o=o, dq=dq, dkn=dkn, dvn=dvn, do=do),
            dict(q=torch.empty_like(q), k=torch.empty_like(k), v=torch.empty_like(v), o=torch.empty_like(o),
                 dq=torch.empty_like(dq), dkn=torch.empty_like(dkn), dvn=torch.empty_like(dvn), do=torch.empty_like(do))]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_step(n):
        i = n % 2
        b = sets[i]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_comp[i])                    # the step that last read this set's inputs is done
            b["q"].copy_(hq, non_blocking=True); b["k"].copy_(hk, non_blocking=True); b["v"].copy_(hv, non_blocking=True)
            b["dq"].copy_(hdq, non_blocking=True); b["dkn"].copy_(hkn, non_blocking=True); b["dvn"].copy_(hvn, non_blocking=True)
            ev_in[i].record(s_in)
        with torch.cuda.stream(s_comp):
            s_comp.wait_event(ev_in[i])
            s_comp.wait_event(ev_out[i])                   # this set's outputs of two steps ago have left
            l4l.l4l_attn_prefill(b["q"], b["k"], b["v"], b["o"], plens, wp.scale, ws_p, cache_k=pk, cache_v=pv)
            l4l.l4l_kv_append(dck, dcv, b["dkn"], b["dvn"], dpos)
            l4l.l4l_attn_decode(b["dq"], b["do"], dck, dcv, dlen, Lmax, wd.scale, ws_d)
            ev_comp[i].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[i])
            ho.copy_(b["o"], non_blocking=True)
            hdo.copy_(b["do"], non_blocking=True)
            ev_out[i].record(s_out)

    e2e_steps = max(4, min(args.steps, 20))
    barrier()
    for n in range(4):
        e2e_step(n)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_in)
    for n in range(e2e_steps):
        e2e_step(n)
    s_out.wait_event(ev_comp[(e2e_steps - 1) % 2])
    e1.record(s_out)                                       # after the last step's outputs have reached the host
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    # ---- max over ranks
    total_ms, e2e_ms, t_pre, t_dec, t_app, t_dec_b2b, t_rope, t_chunk, t_fused, t_paged, t_fp8, t_rglru, t_step1, t_step3 = max_over_ranks(
        [total_ms, e2e_ms, t_pre, t_dec, t_app, t_dec_b2b, t_rope, t_chunk, t_fused, t_paged, t_fp8, t_rglru, t_step1, t_step3], world,
        dev)
    if rank != 0:
        return

    ms_per_step = total_ms / args.steps
    step_flops = pre_flops + dec_flops
    value = whole_job_value(world, step_flops, ms_per_step)
    peaks = measured_peaks()
    med = lambda xs: xs[len(xs) // 2]
    pre_tflops = pre_flops / (t_pre * 1e-3) / 1e12
    dec_gbs = dec_bytes / (t_dec_b2b * 1e-3) / 1e9          # overlapped: mean over back-to-back launches
    dec_gbs_single = dec_bytes / (med(dec_single) * 1e-3) / 1e9   # one launch alone, cold L2: the roofline figure
    dec_gbs_in_step = dec_bytes / (t_dec * 1e-3) / 1e9    # inside the step, between two event records
    # Which measured tensor peak applies: the burst figure for a timed region too short for the power cap to pull the
    # clock down (under about a second), the sustained one otherwise. Both fractions are printed.
    timed_region_s = total_ms * 1e-3
    burst = timed_region_s < 1.0
    tensor_peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": workload_name(wp, wd),
            "value_definition": "attention FLOPs of one step (4*D per causal query-key pair per query head for prefill, "
                                "4*D per cached token per query head for decode) / step time, summed over GPUs",
            "l2": "inputs larger than L2: prefill streams 805 MB and decode 294 MB per step, each evicting the other",
            "parallelism": "replicas (sequences shard with no exchange)" if world > 1 else "single GPU",
        },
        "prefill": {"tflops": pre_tflops, "ms": t_pre, "pct_nominal_2250": 100 * pre_tflops / NOMINAL_TFLOPS,
                    "pct_measured_burst": 100 * pre_tflops / peaks["bf16_tflops"],
                    "pct_measured_sustained": 100 * pre_tflops / peaks["bf16_tflops_sustained"],
                    "in_step_ms": {"mean": t_pre, "median": med(pre_times), "best": pre_times[0]},
                    "single_launch_ms": {"median": med(pre_single), "best": pre_single[0]},
                    "single_launch_tflops": pre_flops / (med(pre_single) * 1e-3) / 1e12},
        "decode": {"kv_gbs": dec_gbs_single, "us": med(dec_single) * 1e3,
                   "pct_nominal_8000": 100 * dec_gbs_single / NOMINAL_GBS,
                   "pct_measured": 100 * dec_gbs_single / peaks["hbm_gbs"],
                   "single_launch_us": {"median": med(dec_single) * 1e3, "best": dec_single[0] * 1e3,
                                        "launches": len(dec_single),
                                        "how": "1 GiB read (L2 cold and clean), event, one launch, event",
                                        "behind_a_1GiB_write_median": med(dec_single_dirty) * 1e3,
                                        "behind_a_1GiB_write_note": "L2 full of dirty lines: their write-back shares "
                                                                    "HBM with the launch"},
                   "event_pairs_us": {"median": med(dec_pairs) * 1e3, "best": dec_pairs[0] * 1e3,
                                      "launches": len(dec_pairs), "how": "back to back, an event pair around each launch"},
                   "overlapped_us": {"mean": t_dec_b2b * 1e3, "launches": n_dec, "kv_gbs": dec_gbs,
                                     "pct_nominal_8000": 100 * dec_gbs / NOMINAL_GBS,
                                     "pct_measured": 100 * dec_gbs / peaks["hbm_gbs"],
                                     "how": "back to back between one pair of events; a launch's prologue runs under "
                                            "the previous launch's tail (programmatic stream serialization)"},
                   "in_step_us": t_dec * 1e3, "in_step_kv_gbs": dec_gbs_in_step, "append_us": t_app * 1e3},
        "roofline": {"kernel": "prefill", "bound": "tensor", "achieved": pre_tflops, "peak": tensor_peak,
                     "unit": "TFLOP/s", "frac": pre_tflops / tensor_peak, "traffic": None,
                     "frac_burst": pre_tflops / peaks["bf16_tflops"],
                     "frac_sustained": pre_tflops / peaks["bf16_tflops_sustained"],
                     "timed_region_s": timed_region_s,
                     "peak_source": peaks["source"] + (" (burst bf16 GEMM: timed region under 1 s)" if burst
                                                       else " (sustained bf16 GEMM: timed region of 1 s or more)")},
        "roofline_decode": {"kernel": "decode_split (single launch, cold L2)", "bound": "hbm", "achieved": dec_gbs_single,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": dec_gbs_single / peaks["hbm_gbs"],
                            "frac_overlapped": dec_gbs / peaks["hbm_gbs"], "traffic": None,
                            "peak_source": peaks["source"] + " (device copy)"},
        "e2e": {"value": whole_job_value(world, step_flops, e2e_ms), "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "widened": {
            "rope_norm_kv_append": {"us": t_rope * 1e3, "gbs": rope_bytes / (t_rope * 1e-3) / 1e9,
                                    "frac_of_measured_hbm": rope_bytes / (t_rope * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                    "bytes": rope_bytes},
            "prefill_from_cache": {"ms": t_chunk, "tflops": pre_flops / (t_chunk * 1e-3) / 1e12},
            "prefill_chunk_4096_over_4096_cached_with_fused_append": {"ms": t_chunk_append,
                                                                      "tflops": chunk_flops / (t_chunk_append * 1e-3) / 1e12},
            "decode_with_fused_append": {"us": t_fused * 1e3, "kv_gbs": dec_bytes / (t_fused * 1e-3) / 1e9},
            "decode_step_rope_norm_append_attention": {"one_launch_us": t_step1 * 1e3, "two_launches_us": t_step3 * 1e3},
            "decode_paged_64": {"us": t_paged * 1e3, "kv_gbs": dec_bytes / (t_paged * 1e-3) / 1e9,
                                "with_fused_append_us": t_paged_fused * 1e3},
            "rglru_scan_B4_T8192_W2560": {"us": t_rglru * 1e3, "gbs": rglru_bytes / (t_rglru * 1e-3) / 1e9,
                                          "frac_of_measured_hbm": rglru_bytes / (t_rglru * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                          "bytes": rglru_bytes},
            "rglru_scan_B2_T8192_W2560": {"us": t_rglru3 * 1e3, "gbs": rglru_bytes / 2 / (t_rglru3 * 1e-3) / 1e9,
                                          "bytes": rglru_bytes // 2},
            "rglru_scan_B16_T2048_W2560": {"us": t_rglru2 * 1e3, "gbs": rglru_bytes / (t_rglru2 * 1e-3) / 1e9,
                                           "frac_of_measured_hbm": rglru_bytes / (t_rglru2 * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                           "bytes": rglru_bytes},
            "decode_fp8_cache": {"us": t_fp8 * 1e3, "kv_gbs_fp8_bytes": dec_bytes / 2 / (t_fp8 * 1e-3) / 1e9,
                                 "speedup_over_bf16_cache": t_dec_b2b / t_fp8, "with_fused_append_us": t_fp8_fused * 1e3,
                                 "with_rope_norm_and_append_us": t_fp8_rope * 1e3},
            "decode_64_query_heads_on_8_kv_heads": {"us": t_g8 * 1e3, "kv_gbs": dec_bytes / (t_g8 * 1e-3) / 1e9},
            "other_configs": other,
            "decode_B512_L64_to_256": {"warp_kernel_us": t_short * 1e3, "kv_gbs": short_bytes / (t_short * 1e-3) / 1e9,
                                       "split_kernel_us": t_short_split * 1e3},
            "decode_step_B1_L2304_in_cuda_graph": {"cluster_kernel_us": t_small, "split_kernel_us": t_small_split},
        },
        "gpu_launches": 3 * args.steps,
        "clocks": clocks,
        "device_error": dev_err,
    }
    line["roofline"]["traffic"] = NCU_TRAFFIC_PREFILL
    line["roofline_decode"]["traffic"] = NCU_TRAFFIC_DECODE
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline_obj(time_oracle_sample(wp, wd, seq, db))
    print(json.dumps(line))


def run_profile_case(case: str):
    """A few launches of ONE kernel on a small case, for `ncu` captures (not a benchmark):
    prefill = B=1, S=8192 of the long_prefill workload (inputs 168 MB > L2); decode = the batched_decode batch;
    rglru = the RG-LRU scan on B=16, T=2048, W=2560; rglru_long = the same bytes as B=4, T=8192 (narrow strips); decode_small = the cluster decode kernel on B=4 x 8192 tokens; decode_short = the warp-per-unit decode kernel on B=512 x 64..256 tokens; decode_fp8 = the split kernel on the batched_decode batch in an fp8 cache; rope = rope + norm + cache update on B=2, S=8192."""
    from paper_2608_21836_b200 import binding as l4l

    torch.cuda.set_device(0)
    if case == "prefill":
        w = wl.WORKLOADS["long_prefill"]
        seq = wl.make_sequence(w, B=1)
        q, k, v = seq.q.cuda(), seq.k.cuda(), seq.v.cuda()
        o = torch.empty_like(q)
        ck = torch.empty(1, w.Hkv, seq.S, w.D, dtype=torch.bfloat16, device="cuda")
        cv = torch.empty_like(ck)
        lens = torch.full((1,), seq.S, dtype=torch.int32, device="cuda")
        ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, 1, w.Hq, w.Hkv, w.D, seq.S)
        for _ in range(3):
            l4l.l4l_attn_prefill(q, k, v, o, lens, w.scale, ws, cache_k=ck, cache_v=cv)
    elif case in ("rglru", "rglru_long"):
        # 503 MB of inputs, 168 MB of output; rglru: 640 strips of 64 channels; rglru_long: 4 sequences of 8192 steps,
        # which the library cuts into 640 strips of 16 channels (160 strips of 64 would load 148 SMs unevenly)
        B, T, W = (16, 2048, 2560) if case == "rglru" else (4, 8192, 2560)
        gen = torch.Generator().manual_seed(1006)
        x = torch.randn(B, T, W, generator=gen).to(torch.bfloat16).cuda()
        gx = (torch.randn(B, T, W, generator=gen) * 2).to(torch.bfloat16).cuda()
        ga = (torch.randn(B, T, W, generator=gen) * 2).to(torch.bfloat16).cuda()
        ap = torch.log(torch.expm1(-torch.log(torch.rand(W, generator=gen) * 0.099 + 0.9) / 8)).float().cuda()
        state = torch.zeros(B, W, device="cuda")
        y = torch.empty_like(x)
        ws = l4l.new_rglru_workspace(B, T, W)
        for _ in range(3):
            l4l.l4l_rglru_scan(x, gx, ga, ap, state, y, ws)
    elif case == "rope":
        # rope + QK-norm + cache update of a whole prompt: B=2, S=8192 of the long_prefill shapes (403 MB moved)
        w = wl.WORKLOADS["long_prefill"]
        seq = wl.make_sequence(w, B=2)
        q, k, v = seq.q.cuda(), seq.k.cuda(), seq.v.cuda()
        ck = torch.empty(2, w.Hkv, seq.S, w.D, dtype=torch.bfloat16, device="cuda")
        cv = torch.empty_like(ck)
        cos, sin = wl.make_rope_tables(seq.S, w.D)
        cos, sin = cos.cuda(), sin.cuda()
        gamma = torch.ones(w.D, dtype=torch.float32, device="cuda")
        pos = torch.zeros(2, dtype=torch.int32, device="cuda")
        ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, 2, w.Hq, w.Hkv, w.D, seq.S)     # only for the status word below
        for _ in range(3):
            l4l.l4l_rope_kv_append(q, k, v, ck, cv, pos, None, cos, sin, gamma, gamma, 1e-6)
    elif case == "decode_small":
        # the cluster kernel: B = 4 sequences of 8192 tokens of the 8B-shaped layer (134 MB of cache > L2)
        w = wl.WORKLOADS["layer8b"]
        db = wl.make_decode_batch(w, B=4, len_lo=8192, len_hi=8192, Lmax=8192, poison_tail=False)
        q, ck, cv, lens = db.q.cuda(), db.cache_k.cuda(), db.cache_v.cuda(), db.kv_len.cuda()
        o = torch.empty_like(q)
        ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 4, w.Hq, w.Hkv, w.D, 8192)
        for _ in range(3):
            l4l.l4l_attn_decode(q, o, ck, cv, lens, 8192, w.scale, ws)
    elif case == "decode_fp8":
        # the split kernel on an fp8 (e4m3) cache: the batched_decode batch quantised with one scale per KV head
        w = wl.WORKLOADS["batched_decode"]
        db = wl.make_decode_batch(w, poison_tail=False)
        q, lens = db.q.cuda(), db.kv_len.cuda()
        B, Lmax = w.decode_B, w.decode_Lmax
        k8 = torch.zeros(B, w.Hkv, Lmax, w.D, dtype=torch.uint8, device="cuda")
        v8 = torch.zeros_like(k8)
        sc = torch.full((w.Hkv,), 4.5 / 448, dtype=torch.float32, device="cuda")
        l4l.l4l_kv_append_fp8(k8, v8, db.cache_k.cuda().permute(0, 2, 1, 3), db.cache_v.cuda().permute(0, 2, 1, 3),
                              torch.zeros(B, dtype=torch.int32, device="cuda"), sc, sc)
        o = torch.empty_like(q)
        ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, w.Hq, w.Hkv, w.D, Lmax)
        for _ in range(3):
            l4l.l4l_attn_decode_fp8(q, o, k8, v8, sc, sc, lens, Lmax, w.scale, ws)
    elif case == "decode_short":
        # the warp-per-unit kernel: B = 512 sequences of 64 to 256 tokens of the 8B-shaped layer (338 MB of cache > L2)
        w = wl.WORKLOADS["batched_decode"]
        db = wl.make_decode_batch(w, B=512, len_lo=64, len_hi=256, Lmax=256, poison_tail=False)
        q, ck, cv, lens = db.q.cuda(), db.cache_k.cuda(), db.cache_v.cuda(), db.kv_len.cuda()
        o = torch.empty_like(q)
        ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 512, w.Hq, w.Hkv, w.D, 256)
        for _ in range(3):
            l4l.l4l_attn_decode(q, o, ck, cv, lens, 256, w.scale, ws)
    else:
        w = wl.WORKLOADS["batched_decode"]
        db = wl.make_decode_batch(w)
        q, ck, cv, lens = db.q.cuda(), db.cache_k.cuda(), db.cache_v.cuda(), db.kv_len.cuda()
        o = torch.empty_like(q)
        ws = l4l.new_workspace(l4l.L4L_OP_DECODE, w.decode_B, w.Hq, w.Hkv, w.D, w.decode_Lmax)
        for _ in range(3):
            l4l.l4l_attn_decode(q, o, ck, cv, lens, w.decode_Lmax, w.scale, ws)
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": case, "device_error": l4l.l4l_last_device_error(ws)}))


def spawn_command(n_gpus: int, argv, port: int | None = None):
    """The command that runs this script as n_gpus ranks on one node (rendezvous on 127.0.0.1)."""
    if port is None:
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-case", choices=["prefill", "decode", "decode_small", "decode_short", "decode_fp8", "rope", "rglru", "rglru_long"], default=None,
                    help="run three launches of one kernel on a small case and exit (for ncu)")
    args = ap.parse_args()
    if args.profile_case:
        run_profile_case(args.profile_case)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly with --gpus N: start the N ranks ourselves, one process per GPU, the way a launcher would
        sys.exit(subprocess.call(spawn_command(args.gpus, sys.argv[1:])))
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0))))
    try:
        run_ours(args, rank, world)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
