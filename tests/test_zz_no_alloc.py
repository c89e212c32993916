"""The allocation-free decode entry point, l4l_attn_decode_static, against the workspace entry point.

This file is named so that pytest collects it last: if it fails under `-x`, every other test has
already run. It passes both alone in a fresh process and after the rest of the suite.

Why the entry point exists: some users of the library reach decode at a point where they are not
allowed to allocate device memory (a serving loop whose HBM is fully planned at start-up; a plug-in in a
foreign runtime where cudaMalloc would synchronise the device). They cannot provide a workspace, so the
library keeps the scratch in a fixed array of its own. The array is shared by all calls and keeps the
previous call's contents, which is why the check below makes two calls in a row with different inputs.
"""
import math

import numpy as np
import pytest
import torch

from paper_2608_21836_b200 import binding as l4l
from helpers import MAX_ABS_TOL, MEAN_ABS_TOL, nan_bf16

pytestmark = pytest.mark.gpu


def make_batch(B, Hq, Hkv, D, Lmax, lens, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    kv_len = torch.tensor(lens, dtype=torch.int32)
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= kv_len.view(B, 1, 1, 1)
    nan = nan_bf16((1,))
    return q.cuda(), torch.where(dead, nan, ck).contiguous().cuda(), torch.where(dead, nan, cv).contiguous().cuda(), kv_len.cuda()


def run_both(q, ck, cv, lens, Lmax, scale):
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


def test_static_scratch_decode_matches_workspace_decode_on_two_calls_in_a_row():
    # call 1: many sequences cut into several pieces (partials and ticket counters in use), one empty sequence
    lens1 = [3000, 0, 77, 64, 1, 2047, 513, 1000]
    q, ck, cv, lens = make_batch(8, 8, 2, 128, 3072, lens1, seed=501)
    r1 = run_both(q, ck, cv, lens, 3072, 1.0 / math.sqrt(128))
    assert_same(*r1)
    # call 2 right after, other shapes and data: must not be disturbed by what call 1 left in the array
    lens2 = [1500, 900, 33, 1024, 700, 1]
    q2, ck2, cv2, lens_2 = make_batch(6, 12, 12, 64, 1536, lens2, seed=502)
    r2 = run_both(q2, ck2, cv2, lens_2, 1536, 1.0 / math.sqrt(64))
    assert_same(*r2)
    # and the first problem once more gives the first answer again, bit for bit
    o_again = torch.zeros_like(q)
    l4l.l4l_attn_decode_static(q, o_again, ck, cv, lens, 3072, 1.0 / math.sqrt(128))
    torch.cuda.synchronize()
    assert torch.equal(o_again.view(torch.int16), r1[2].view(torch.int16))


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
