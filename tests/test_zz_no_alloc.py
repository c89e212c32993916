"""The allocation-free decode entry point, l4l_attn_decode_static, against the workspace entry point and the oracle.

This file is named so that pytest collects it last: if it fails under `-x`, every other test has
already run. It passes both alone in a fresh process and after the rest of the suite.

Why the entry point exists: some users of the library reach decode at a point where they are not
allowed to allocate device memory (a serving loop whose HBM is fully planned at start-up; a plug-in in a
foreign runtime where cudaMalloc would synchronise the device). They cannot provide a workspace, so the
library keeps the scratch in a fixed array of its own. The array is shared by all calls and keeps the
previous call's contents, which is why the checks below make two calls in a row with different inputs.

Every shape here is one the library hands to its split kernel, the only decode kernel that uses the
scratch (ticket counters and fp32 partials of the sequences cut between CTAs); the test asserts that
choice, so that it cannot silently drift to a kernel that leaves the array untouched.
"""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import MAX_ABS_TOL, MEAN_ABS_TOL, assert_close_to_oracle, nan_bf16

pytestmark = pytest.mark.gpu


def make_batch(B, Hq, Hkv, D, Lmax, lens, seed):
    """Seeded N(0,1) bf16 queries and cache, slots past a sequence's length poisoned with NaN. Returns the host copies
    (for the oracle) and the device copies."""
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    kv_len = torch.tensor(lens, dtype=torch.int32)
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= kv_len.view(B, 1, 1, 1)
    nan = nan_bf16((1,))
    ck, cv = torch.where(dead, nan, ck).contiguous(), torch.where(dead, nan, cv).contiguous()
    return (q, ck, cv, kv_len), (q.cuda(), ck.cuda(), cv.cuda(), kv_len.cuda())


def ragged(B, lo, hi, seed, pinned=()):
    rng = np.random.default_rng(seed)
    lens = rng.integers(lo, hi + 1, B).tolist()
    for i, v in enumerate(pinned):
        lens[i] = v
    return lens


def on_split_kernel(B, Hq, Hkv, D, Lmax):
    choice = l4l.l4l_decode_kernel_choice(B, Hq, Hkv, D, Lmax)
    return choice is not None and choice[0] == "split"


def run_both(dev, Lmax, scale):
    q, ck, cv, lens = dev
    B, Hq, D = q.shape
    Hkv = ck.shape[1]
    # existing entry point, caller-provided workspace
    o_ref = torch.zeros_like(q)
    lse_ref = torch.zeros(B, Hq, dtype=torch.float32, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode(q, o_ref, ck, cv, lens, Lmax, scale, ws, lse=lse_ref)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    # new entry point: no workspace, nothing allocated by the library
    o_new = torch.full_like(q, float("nan"))
    lse_new = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    l4l.l4l_attn_decode_static(q, o_new, ck, cv, lens, Lmax, scale, lse=lse_new)
    torch.cuda.synchronize()
    return o_ref, lse_ref, o_new, lse_new


def assert_same(o_ref, lse_ref, o_new, lse_new):
    a, b = o_ref.float().cpu().numpy(), o_new.float().cpu().numpy()
    assert np.isfinite(b).all()
    err = np.abs(a - b)
    assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL
    la, lb = lse_ref.cpu().numpy(), lse_new.cpu().numpy()
    assert np.array_equal(np.isneginf(la), np.isneginf(lb))
    fin = np.isfinite(la)
    assert np.abs(la[fin] - lb[fin]).max() <= 2e-3


def assert_matches_oracle(host, scale, o_new, lse_new, what):
    q, ck, cv, kv_len = host
    o_orc, lse_orc = orc.decode(q, ck, cv, kv_len.numpy(), scale)
    assert_close_to_oracle(o_new, o_orc, what)
    got = lse_new.cpu().double().numpy()
    assert np.array_equal(np.isneginf(got), np.isneginf(lse_orc))
    fin = np.isfinite(lse_orc)
    assert np.abs(got[fin] - lse_orc[fin]).max() <= 2e-3, what


def test_static_scratch_decode_matches_workspace_decode_and_oracle_on_two_calls_in_a_row():
    # call 1: 256 (sequence, KV head) units on 148 SMs: the split kernel, long sequences cut into several pieces
    # (partials and ticket counters of the fixed array in use), one empty and one single-token sequence
    B1, Hq1, Hkv1, D1, L1 = 32, 32, 8, 128, 4096
    assert on_split_kernel(B1, Hq1, Hkv1, D1, L1)
    host1, dev1 = make_batch(B1, Hq1, Hkv1, D1, L1, ragged(B1, 512, 4096, 11, pinned=(4096, 0, 1, 4095)), seed=501)
    s1 = 1.0 / math.sqrt(D1)
    r1 = run_both(dev1, L1, s1)
    assert_same(*r1)
    assert_matches_oracle(host1, s1, r1[2], r1[3], "static scratch, call 1")
    # call 2 right after, other shapes and data: must not be disturbed by what call 1 left in the array
    B2, Hq2, Hkv2, D2, L2 = 20, 12, 12, 64, 1536
    assert on_split_kernel(B2, Hq2, Hkv2, D2, L2)
    host2, dev2 = make_batch(B2, Hq2, Hkv2, D2, L2, ragged(B2, 1, 1536, 12, pinned=(1536, 33)), seed=502)
    s2 = 1.0 / math.sqrt(D2)
    r2 = run_both(dev2, L2, s2)
    assert_same(*r2)
    assert_matches_oracle(host2, s2, r2[2], r2[3], "static scratch, call 2")
    # and the first problem once more gives the first answer again, bit for bit
    o_again = torch.zeros_like(dev1[0])
    l4l.l4l_attn_decode_static(dev1[0], o_again, dev1[1], dev1[2], dev1[3], L1, s1)
    torch.cuda.synchronize()
    assert torch.equal(o_again.view(torch.int16), r1[2].view(torch.int16))


def test_static_scratch_decode_coarsens_its_split_to_fit_the_array():
    # 80 sequences of up to 8192 tokens, 32 query heads on 2 KV heads: the split the workspace entry point would choose
    # needs more scratch than the fixed array holds, so this entry point has to cut the sequences into fewer pieces
    B, Hq, Hkv, D, Lmax = 80, 32, 2, 128, 8192
    assert l4l.l4l_workspace_bytes(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax) > l4l.STATIC_SCRATCH_BYTES
    assert on_split_kernel(B, Hq, Hkv, D, Lmax)
    host, dev = make_batch(B, Hq, Hkv, D, Lmax, ragged(B, 256, 8192, 13, pinned=(8192, 8191)), seed=503)
    scale = 1.0 / math.sqrt(D)
    r = run_both(dev, Lmax, scale)
    assert_same(*r)
    assert_matches_oracle(host, scale, r[2], r[3], "static scratch, coarsened split")
    # second call in a row on the same problem: same answer, bit for bit
    o_again = torch.zeros_like(dev[0])
    l4l.l4l_attn_decode_static(dev[0], o_again, dev[1], dev[2], dev[3], Lmax, scale)
    torch.cuda.synchronize()
    assert torch.equal(o_again.view(torch.int16), r[2].view(torch.int16))


def test_static_scratch_decode_rejects_problems_beyond_its_array():
    # coarsest split: 2 partials per (sequence, query head) -> B*Hq*2*(D+1)*4 bytes must fit 8 MiB
    B, Hq, Hkv, D, Lmax = 512, 32, 8, 128, 128
    q = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros_like(q)
    ck = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16, device="cuda")
    cv = torch.zeros_like(ck)
    lens = torch.full((B,), Lmax, dtype=torch.int32, device="cuda")
    assert B * Hq * 2 * (D + 1) * 4 > l4l.STATIC_SCRATCH_BYTES
    with pytest.raises(l4l.L4LError) as e:
        l4l.l4l_attn_decode_static(q, o, ck, cv, lens, Lmax, 0.1)
    assert e.value.status == l4l.L4L_ERR_WORKSPACE
    # host-side validation is the same as the workspace variant's
    with pytest.raises(l4l.L4LError) as e:
        l4l.l4l_attn_decode_static(q[:, :30].contiguous(), o[:, :30].contiguous(), ck, cv, lens, Lmax, 0.1)
    assert e.value.status == l4l.L4L_ERR_UNSUPPORTED
