"""l4l_attn_prefill_chunk (new tokens over a populated cache, bottom-right causal alignment) against the oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, assert_close_to_oracle, bits_equal, nan_bf16

pytestmark = pytest.mark.gpu
SENTINEL = 0x4D4D


def sentinel_bf16(shape):
    return torch.full(shape, SENTINEL, dtype=torch.int16).view(torch.bfloat16)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4)])
def test_chunk_ragged_pasts_and_lengths(D, Hq, Hkv):
    past = [0, 1, 127, 128, 129, 300, 511, 64, 1000, 5]
    qlen = [257, 128, 1, 129, 200, 5, 130, 0, 64, 300]
    B, S, Lmax = len(past), 300, 1408
    g = torch.Generator().manual_seed(700 + D + Hq)
    q = torch.randn(B, S, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    tot = torch.tensor(past) + torch.tensor(qlen)
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= tot.view(B, 1, 1, 1)
    ck = torch.where(dead, nan_bf16((1,)), ck).contiguous()
    cv = torch.where(dead, nan_bf16((1,)), cv).contiguous()
    qdead = torch.arange(S).view(1, S, 1, 1) >= torch.tensor(qlen).view(B, 1, 1, 1)
    q = torch.where(qdead, nan_bf16((1,)), q).contiguous()
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.prefill_chunk(q, ck, cv, np.array(past, np.int32), np.array(qlen, np.int32), scale)

    gq, gk, gv = Guarded(q), Guarded(ck), Guarded(cv)
    go = Guarded(sentinel_bf16((B, S, Hq, D)))
    lse = torch.full((B, Hq, S), -12345.0, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill_chunk(gq.t, go.t, gk.t, gv.t, torch.tensor(past, dtype=torch.int32).cuda(),
                               torch.tensor(qlen, dtype=torch.int32).cuda(), scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for x in (gq, gk, gv, go):
        assert x.margins_intact()
    assert bits_equal(gk.t, ck) and bits_equal(gv.t, cv)                      # the cache is only read
    valid = torch.arange(S).view(1, S) < torch.tensor(qlen).view(B, 1)
    o_cpu, lse_cpu = go.t.cpu(), lse.cpu()
    assert_close_to_oracle(o_cpu[valid], ref[valid.numpy()], "chunk prefill o")
    vl = valid.view(B, 1, S).expand(B, Hq, S)
    assert np.abs(lse_cpu[vl].double().numpy() - ref_lse[vl.numpy()]).max() <= 2e-3
    assert (o_cpu[~valid].view(torch.int16) == SENTINEL).all()
    assert (lse_cpu[~vl] == -12345.0).all()


def test_chunks_after_a_prompt_equal_one_long_prefill():
    """A prompt of 700 tokens, then chunks of 300 and 24 tokens appended and prefilled over the cache: the
    three outputs together must match the oracle's causal prefill of all 1024 tokens."""
    B, Hq, Hkv, D, T = 2, 8, 2, 128, 1024
    g = torch.Generator().manual_seed(71)
    q = torch.randn(B, T, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    scale = 0.088
    ref, _ = orc.prefill(q, k, v, np.full(B, T, np.int32), scale)
    dq, dk, dv = q.cuda(), k.cuda(), v.cuda()
    ck = nan_bf16((B, Hkv, T, D)).cuda()
    cv = nan_bf16((B, Hkv, T, D)).cuda()
    out = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, T)
    lens = torch.full((B,), 700, dtype=torch.int32, device="cuda")
    l4l.l4l_attn_prefill(dq[:, :700], dk[:, :700], dv[:, :700], out[:, :700], lens, scale, ws, cache_k=ck, cache_v=cv)
    for a, b_ in ((700, 1000), (1000, 1024)):
        n = b_ - a
        pos = torch.full((B,), a, dtype=torch.int32, device="cuda")
        l4l.l4l_kv_append(ck, cv, dk[:, a:b_], dv[:, a:b_], pos)
        l4l.l4l_attn_prefill_chunk(dq[:, a:b_], out[:, a:b_], ck, cv, pos,
                                   torch.full((B,), n, dtype=torch.int32, device="cuda"), scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(out.cpu(), ref, "prompt + two chunks")
    assert bits_equal(ck, k.permute(0, 2, 1, 3).contiguous())
