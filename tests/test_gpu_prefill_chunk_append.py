"""l4l_attn_prefill_chunk_append (a chunk of new tokens over a populated cache, the chunk's K/V written to the cache in
the same launch) against the oracle's append followed by its chunk prefill; contiguous and paged caches."""
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


def as_bf16(bits_u16):
    return torch.from_numpy(bits_u16.view(np.int16)).view(torch.bfloat16)


def make_chunk(B, S, Hq, Hkv, D, qlen, seed):
    """Seeded chunk tensors; rows past a sequence's chunk length are NaN (they must not be looked at)."""
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, S, Hq, D, generator=g).to(torch.bfloat16)
    kn = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    vn = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    dead = torch.arange(S).view(1, S, 1, 1) >= torch.tensor(qlen).view(B, 1, 1, 1)
    nan = nan_bf16((1,))
    return [torch.where(dead, nan, x).contiguous() for x in (q, kn, vn)], g


def check_outputs(o_dev, lse_dev, ref, ref_lse, qlen, B, S, Hq, what):
    valid = torch.arange(S).view(1, S) < torch.tensor(qlen).view(B, 1)
    o_cpu, lse_cpu = o_dev.cpu(), lse_dev.cpu()
    assert_close_to_oracle(o_cpu[valid], ref[valid.numpy()], what)
    vl = valid.view(B, 1, S).expand(B, Hq, S)
    assert np.abs(lse_cpu[vl].double().numpy() - ref_lse[vl.numpy()]).max() <= 2e-3
    assert (o_cpu[~valid].view(torch.int16) == SENTINEL).all()               # rows past the chunk are never written
    assert (lse_cpu[~vl] == -12345.0).all()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4), (16, 1)])
def test_chunk_append_contiguous_ragged_pasts_and_lengths(D, Hq, Hkv):
    past = [0, 1, 127, 128, 129, 300, 511, 64, 1000, 5, 256]
    qlen = [257, 128, 1, 129, 200, 5, 130, 0, 64, 300, 256]
    B, S, Lmax = len(past), 300, 1408
    (q, kn, vn), g = make_chunk(B, S, Hq, Hkv, D, qlen, seed=900 + D + Hq)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    # slots from `past` on hold NaN before the call: whatever is read from them must come through k_new / v_new
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= torch.tensor(past).view(B, 1, 1, 1)
    ck = torch.where(dead, nan_bf16((1,)), ck).contiguous()
    cv = torch.where(dead, nan_bf16((1,)), cv).contiguous()
    scale = 1.0 / math.sqrt(D)
    pa, ql = np.array(past, np.int32), np.array(qlen, np.int32)
    ek, ev = orc.kv_append(ck, cv, kn, vn, pa, ql)
    ref, ref_lse = orc.prefill_chunk(q, as_bf16(ek), as_bf16(ev), pa, ql, scale)

    gq, gkn, gvn, gk, gv = Guarded(q), Guarded(kn), Guarded(vn), Guarded(ck), Guarded(cv)
    go = Guarded(sentinel_bf16((B, S, Hq, D)))
    lse = torch.full((B, Hq, S), -12345.0, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill_chunk_append(gq.t, gkn.t, gvn.t, go.t, gk.t, gv.t, torch.from_numpy(pa).cuda(),
                                      torch.from_numpy(ql).cuda(), scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for x in (gq, gkn, gvn, gk, gv, go):
        assert x.margins_intact()
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)                     # exactly the chunk's rows were written
    check_outputs(go.t, lse, ref, ref_lse, qlen, B, S, Hq, "chunk prefill + append")


@pytest.mark.parametrize("page", [16, 32, 64, 128, 256])
def test_chunk_append_paged(page):
    Hq, Hkv, D = 8, 2, 128
    past = [0, 1, 127, 128, 129, 300, 511, 64, 700, 5]
    qlen = [257, 128, 1, 129, 200, 5, 130, 0, 64, 300]
    B, S, Lmax = len(past), 300, 1024
    n_per = Lmax // page
    (q, kn, vn), g = make_chunk(B, S, Hq, Hkv, D, qlen, seed=950 + page)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= torch.tensor(past).view(B, 1, 1, 1)
    ck = torch.where(dead, nan_bf16((1,)), ck).contiguous()
    cv = torch.where(dead, nan_bf16((1,)), cv).contiguous()
    # scatter the sequences' pages over a pool with a few spare pages; pages wholly past past+qlen are not mapped
    n_pages = B * n_per + 3
    perm = torch.randperm(n_pages, generator=g)[:B * n_per].view(B, n_per)
    table = perm.clone().to(torch.int32)
    for b in range(B):
        first_unused = (past[b] + qlen[b] + page - 1) // page
        table[b, first_unused:] = -1
    pool_k = nan_bf16((n_pages, Hkv, page, D)).clone()
    pool_v = nan_bf16((n_pages, Hkv, page, D)).clone()
    for b in range(B):
        for i in range(n_per):
            if table[b, i] >= 0:
                pool_k[table[b, i]] = ck[b, :, i * page:(i + 1) * page]
                pool_v[table[b, i]] = cv[b, :, i * page:(i + 1) * page]
    scale = 1.0 / math.sqrt(D)
    pa, ql = np.array(past, np.int32), np.array(qlen, np.int32)
    epk, epv = orc.kv_append_paged(pool_k, pool_v, table.numpy(), kn, vn, pa, ql)
    ek = orc.gather_pages(as_bf16(epk), table.numpy(), Lmax)
    ev = orc.gather_pages(as_bf16(epv), table.numpy(), Lmax)
    ref, ref_lse = orc.prefill_chunk(q, as_bf16(ek), as_bf16(ev), pa, ql, scale)

    gpk, gpv = Guarded(pool_k), Guarded(pool_v)
    go = Guarded(sentinel_bf16((B, S, Hq, D)))
    lse = torch.full((B, Hq, S), -12345.0, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill_chunk_append(q.cuda(), kn.cuda(), vn.cuda(), go.t, gpk.t, gpv.t, torch.from_numpy(pa).cuda(),
                                      torch.from_numpy(ql).cuda(), scale, ws, lse=lse, block_table=table.cuda())
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert gpk.margins_intact() and gpv.margins_intact() and go.margins_intact()
    assert bits_equal(gpk.t, epk) and bits_equal(gpv.t, epv)                 # the pool got exactly the chunk's rows
    check_outputs(go.t, lse, ref, ref_lse, qlen, B, S, Hq, f"paged chunk prefill + append, page {page}")


def test_chunk_append_steps_equal_one_long_prefill_and_feed_decode():
    """A prompt of 700 tokens, then chunks of 300 and 24 tokens through the fused call, then one decode step: the
    outputs together match the oracle's causal prefill of all 1025 tokens, and the cache is the bit copy of K/V."""
    B, Hq, Hkv, D, T = 2, 8, 2, 128, 1025
    g = torch.Generator().manual_seed(73)
    q = torch.randn(B, T, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    scale = 0.088
    ref, _ = orc.prefill(q, k, v, np.full(B, T, np.int32), scale)
    dq, dk, dv = q.cuda(), k.cuda(), v.cuda()
    ck, cv = nan_bf16((B, Hkv, 1152, D)).cuda(), nan_bf16((B, Hkv, 1152, D)).cuda()
    out = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, T)
    for a, b_ in ((0, 700), (700, 1000), (1000, 1024)):
        n = b_ - a
        l4l.l4l_attn_prefill_chunk_append(dq[:, a:b_], dk[:, a:b_], dv[:, a:b_], out[:, a:b_], ck, cv,
                                          torch.full((B,), a, dtype=torch.int32, device="cuda"),
                                          torch.full((B,), n, dtype=torch.int32, device="cuda"), scale, ws)
    wsd = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, 1152)
    od = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_append(dq[:, 1024].contiguous(), od, ck, cv, dk[:, 1024:1025], dv[:, 1024:1025],
                               torch.full((B,), 1025, dtype=torch.int32, device="cuda"), 1152, scale, wsd)
    out[:, 1024] = od
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0 and l4l.l4l_last_device_error(wsd) == 0
    assert_close_to_oracle(out, ref, "prompt + fused chunks + decode step")
    assert bits_equal(ck[:, :, :T], k.permute(0, 2, 1, 3).contiguous()) and bits_equal(cv[:, :, :T], v.permute(0, 2, 1, 3).contiguous())


def test_chunk_append_drops_rows_the_cache_has_no_slot_for():
    B, Hq, Hkv, D, S, Lmax = 1, 4, 2, 128, 200, 256
    (q, kn, vn), g = make_chunk(B, S, Hq, Hkv, D, [200], seed=75)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    past = np.array([100], np.int32)
    gk, gv = Guarded(ck), Guarded(cv)
    o = torch.zeros(B, S, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill_chunk_append(q.cuda(), kn.cuda(), vn.cuda(), o, gk.t, gv.t, torch.from_numpy(past).cuda(),
                                      torch.tensor([200], dtype=torch.int32).cuda(), 0.09, ws)
    torch.cuda.synchronize()
    assert gk.margins_intact() and gv.margins_intact()                       # slots 256..299 do not exist: nothing written there
    ek, ev = orc.kv_append(ck, cv, kn[:, :156], vn[:, :156], past, np.array([156], np.int32))
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)
    # the attention itself still covers all 200 new tokens (they are read from k_new / v_new)
    big_k = torch.cat([ck[:, :, :100], kn.permute(0, 2, 1, 3)], dim=2).contiguous()
    big_v = torch.cat([cv[:, :, :100], vn.permute(0, 2, 1, 3)], dim=2).contiguous()
    ref, _ = orc.prefill_chunk(q, big_k, big_v, past, np.array([200], np.int32), 0.09)
    assert_close_to_oracle(o, ref, "chunk larger than the cache's free slots")
