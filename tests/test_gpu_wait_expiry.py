"""The bounded device-side waits: what happens when one runs out.

No production kernel is starved here and nothing faults, traps or hangs: the library's self-test launches one warp
that runs the same wait routine, with a budget of about 50 microseconds, on a barrier nothing completes. The wait gives
up, the kernel records the fact in the workspace's status block and returns normally. The test checks that the host
sees the code, that the workspace can be cleared, and that the same workspace then serves a normal decode."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import assert_close_to_oracle
from test_gpu_decode import random_batch

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_is_reported_and_the_workspace_recovers():
    B, Hq, Hkv, D, Lmax = 3, 8, 2, 128, 700
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    assert l4l.l4l_last_device_error(ws) == 0 and l4l.l4l_check_status(ws) == l4l.L4L_OK
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    l4l.l4l_selftest_wait_expiry(ws, budget_cycles=100_000)
    t1.record()
    torch.cuda.synchronize()                                   # the kernel returned by itself
    assert t0.elapsed_time(t1) < 100.0                         # ms: the budget is ~50 us, the clamp a few ms
    code = l4l.l4l_last_device_error(ws)
    assert code != 0 and (code & 8)
    assert l4l.l4l_check_status(ws) == l4l.L4L_ERR_TIMEOUT
    assert l4l.status_string(l4l.L4L_ERR_TIMEOUT)
    # the context is intact, the workspace is cleared and used again
    l4l.l4l_workspace_init(ws)
    assert l4l.l4l_last_device_error(ws) == 0 and l4l.l4l_check_status(ws) == l4l.L4L_OK
    q, ck, cv, kv_len = random_batch(B, Hq, Hkv, D, Lmax, [700, 1, 333], seed=77)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    scale = 1.0 / math.sqrt(D)
    l4l.l4l_attn_decode(q.cuda(), o, ck.cuda(), cv.cuda(), kv_len.cuda(), Lmax, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_check_status(ws) == l4l.L4L_OK
    ref, _ = orc.decode(q, ck, cv, kv_len.numpy(), scale)
    assert_close_to_oracle(o, ref, "decode on a workspace that had reported a time-out")


def test_budget_is_clamped_and_small_workspaces_are_refused():
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, 1, 4, 2, 64, 128)
    l4l.l4l_selftest_wait_expiry(ws, budget_cycles=1 << 62)    # clamped to 2^24 cycles (~10 ms)
    torch.cuda.synchronize()
    assert l4l.l4l_check_status(ws) == l4l.L4L_ERR_TIMEOUT
    l4l.l4l_workspace_init(ws)
    with pytest.raises(l4l.L4LError) as e:
        l4l.l4l_selftest_wait_expiry(ws[:64], budget_cycles=1000)
    assert e.value.status == l4l.L4L_ERR_WORKSPACE


def test_status_block_of_the_static_scratch_is_readable():
    q, ck, cv, kv_len = random_batch(2, 8, 2, 128, 512, [512, 100], seed=78)
    o = torch.zeros(2, 8, 128, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_static(q.cuda(), o, ck.cuda(), cv.cuda(), kv_len.cuda(), 512, 0.1)
    assert l4l.l4l_check_status(None) == l4l.L4L_OK
