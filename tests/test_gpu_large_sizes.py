"""Sizes well beyond the benchmark configurations: a 32k-token prompt (sampled rows against the oracle) and a
128k-token cache at decode (one sequence is then cut into more pieces than there are SMs)."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import MAX_ABS_TOL, MEAN_ABS_TOL, assert_close_to_oracle, bits_equal

pytestmark = pytest.mark.gpu


def test_prefill_32k_tokens_sampled_rows():
    B, S, Hq, Hkv, D = 1, 32768, 8, 2, 128
    g = torch.Generator().manual_seed(321)
    q = torch.randn(B, S, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    dq, dk, dv = q.cuda(), k.cuda(), v.cuda()
    o = torch.zeros_like(dq)
    ck = torch.zeros(B, Hkv, S, D, dtype=torch.bfloat16, device="cuda")
    cv = torch.zeros_like(ck)
    lens = torch.full((B,), S, dtype=torch.int32, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill(dq, dk, dv, o, lens, scale, ws, cache_k=ck, cache_v=cv)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    rng = np.random.default_rng(5)
    rows = [(0, int(i), int(h)) for i in np.concatenate([[0, 1, 127, 128, 255, 256, S - 1, S - 128, S - 129],
                                                          rng.integers(0, S, 150)]) for h in rng.integers(0, Hq, 2)]
    ref, _ = orc.prefill_rows(q, k, v, np.full(B, S, np.int32), scale, np.array(rows, np.int32))
    got = np.stack([o[b, i, h].float().cpu().double().numpy() for b, i, h in rows])
    err = np.abs(got - ref)
    assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL, (err.max(), err.mean())
    assert bits_equal(ck, k.permute(0, 2, 1, 3).contiguous()) and bits_equal(cv, v.permute(0, 2, 1, 3).contiguous())


def test_decode_128k_token_cache():
    B, Hq, Hkv, D, Lmax = 2, 8, 2, 128, 131072
    g = torch.Generator().manual_seed(322)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    lens = np.array([Lmax, 100001], np.int32)
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.decode(q, ck, cv, lens, scale)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, Hq, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode(q.cuda(), o, ck.cuda(), cv.cuda(), torch.from_numpy(lens).cuda(), Lmax, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, "decode over 128k tokens")
    assert np.abs(lse.cpu().double().numpy() - ref_lse).max() <= 2e-3
