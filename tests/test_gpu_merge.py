"""l4l_attn_merge and the context-parallel decode built on it. Only one GPU is available, so the R "ranks" are
R decode calls over disjoint shards of the same caches on that GPU (independent launches, no kernel waits on another);
the gather is a stack. The result must match the oracle's decode over the whole cache."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l, parallel
from helpers import assert_close_to_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("R", [1, 2, 5])
@pytest.mark.parametrize("D", [64, 128])
def test_sharded_decode_plus_merge_equals_full_decode(R, D):
    B, Hq, Hkv, Lmax = 5, 8, 2, 1500
    lens = [1500, 1, 0, 129, 640]
    g = torch.Generator().manual_seed(50 + R + D)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.decode(q, ck, cv, np.array(lens, np.int32), scale)
    dq = q.cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    o_parts = torch.zeros(R, B, Hq, D, dtype=torch.bfloat16, device="cuda")
    lse_parts = torch.zeros(R, B, Hq, device="cuda")
    for r in range(R):
        sk = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16)
        sv = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16)
        sl = []
        for b in range(B):
            t0, t1 = parallel.shard_bounds(lens[b], R, r)
            sl.append(t1 - t0)
            sk[b, :, :t1 - t0] = ck[b, :, t0:t1]
            sv[b, :, :t1 - t0] = cv[b, :, t0:t1]
        l4l.l4l_attn_decode(dq, o_parts[r], sk.cuda(), sv.cuda(), torch.tensor(sl, dtype=torch.int32).cuda(), Lmax, scale,
                            ws, lse=lse_parts[r])
    o = torch.full((B, Hq, D), 9.0, device="cuda").to(torch.bfloat16)
    lse = torch.zeros(B, Hq, device="cuda")
    l4l.l4l_attn_merge(o_parts, lse_parts, o, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, f"merge of {R} shards")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all() and (o.cpu()[2] == 0).all()        # the empty sequence


def test_single_rank_context_parallel_decode_is_plain_decode():
    B, Hq, Hkv, D, Lmax = 2, 8, 2, 128, 256
    g = torch.Generator().manual_seed(3)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16).cuda()
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16).cuda()
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16).cuda()
    lens = torch.tensor([256, 77], dtype=torch.int32, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    o1, o2 = torch.zeros_like(q), torch.zeros_like(q)
    parallel.gpu_context_parallel_decode(q, o1, ck, cv, lens, Lmax, 0.1, ws)
    l4l.l4l_attn_decode(q, o2, ck, cv, lens, Lmax, 0.1, ws)
    torch.cuda.synchronize()
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
