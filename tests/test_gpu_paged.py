"""Paged KV cache: l4l_attn_decode_paged and l4l_kv_append_paged against the oracle (decode over the pages laid
end to end) for page sizes below, at and above the kernel's tile."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, assert_close_to_oracle, bits_equal, nan_bf16

pytestmark = pytest.mark.gpu


def build_pool(B, Hkv, D, page, lens, seed, spare=5):
    """Random pool; every sequence gets the pages its length needs, in shuffled order; the rest of the table is -1;
    unused pages and the tail of each last page are NaN."""
    g = torch.Generator().manual_seed(seed)
    need = [(L + page - 1) // page for L in lens]
    n_pages = sum(need) + spare
    table_stride = max(max(need), 1) + 1
    perm = torch.randperm(n_pages, generator=g).tolist()
    table = np.full((B, table_stride), -1, np.int32)
    pool_k = nan_bf16((n_pages, Hkv, page, D))
    pool_v = nan_bf16((n_pages, Hkv, page, D))
    it = iter(perm)
    for b in range(B):
        for i in range(need[b]):
            pg = next(it)
            table[b, i] = pg
            n = min(page, lens[b] - i * page)
            pool_k[pg, :, :n] = torch.randn(Hkv, n, D, generator=g).to(torch.bfloat16)
            pool_v[pg, :, :n] = torch.randn(Hkv, n, D, generator=g).to(torch.bfloat16)
    return pool_k, pool_v, table


@pytest.mark.parametrize("page", [16, 32, 64, 128, 256])
@pytest.mark.parametrize("Hq,Hkv,D", [(32, 8, 128), (12, 12, 64)])
def test_paged_decode_matches_oracle(page, Hq, Hkv, D):
    lens = [1, 15, 16, 17, 127, 128, 129, 700, 1024, 2049, 333, 0]
    B = len(lens)
    pool_k, pool_v, table = build_pool(B, Hkv, D, page, lens, seed=900 + page + D)
    g = torch.Generator().manual_seed(page)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.decode_paged(q, pool_k, pool_v, table, np.array(lens, np.int32), scale)
    gk, gv = Guarded(pool_k), Guarded(pool_v)
    go = Guarded(torch.zeros(B, Hq, D, dtype=torch.bfloat16))
    lse = torch.zeros(B, Hq, device="cuda")
    max_len = max(lens)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, max_len)
    l4l.l4l_attn_decode_paged(q.cuda(), go.t, gk.t, gv.t, torch.from_numpy(table).cuda(),
                              torch.tensor(lens, dtype=torch.int32).cuda(), max_len, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert gk.margins_intact() and gv.margins_intact() and go.margins_intact()
    assert bits_equal(gk.t, pool_k) and bits_equal(gv.t, pool_v)
    assert_close_to_oracle(go.t.cpu(), ref, f"paged decode, page {page}")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


def test_paged_decode_equals_contiguous_decode_bit_for_bit():
    """With pages as large as the kernel's tile the paged path does the same arithmetic in the same order as the
    contiguous one: the outputs must be identical, not just close."""
    B, Hq, Hkv, D, page = 6, 32, 8, 128, 128
    lens = [1000, 128, 3000, 77, 2048, 513]
    pool_k, pool_v, table = build_pool(B, Hkv, D, page, lens, seed=5)
    Lmax = 3072
    ck = torch.from_numpy(orc.gather_pages(pool_k, table, Lmax).view(np.int16)).view(torch.bfloat16).cuda()
    cv = torch.from_numpy(orc.gather_pages(pool_v, table, Lmax).view(np.int16)).view(torch.bfloat16).cuda()
    q = torch.randn(B, Hq, D, generator=torch.Generator().manual_seed(6)).to(torch.bfloat16).cuda()
    dl = torch.tensor(lens, dtype=torch.int32).cuda()
    o1, o2 = torch.zeros_like(q), torch.zeros_like(q)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode(q, o1, ck, cv, dl, Lmax, 0.09, ws)
    l4l.l4l_attn_decode_paged(q, o2, pool_k.cuda(), pool_v.cuda(), torch.from_numpy(table).cuda(), dl, Lmax, 0.09, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert bits_equal(o1, o2)


@pytest.mark.parametrize("page", [16, 128])
def test_paged_append_then_decode(page):
    B, Hq, Hkv, D, T = 4, 8, 2, 128, 37
    lens = [0, 100, 255, 16]
    pool_k, pool_v, table = build_pool(B, Hkv, D, page, [L + T for L in lens], seed=31)
    g = torch.Generator().manual_seed(32)
    k_new = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    v_new = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    n_new = [T, 5, T, 0]
    table[2, -2:] = -1                           # sequence 2 loses its last pages: those tokens are dropped
    ref_k, ref_v = orc.kv_append_paged(pool_k, pool_v, table, k_new, v_new, lens, n_new)
    gk, gv = Guarded(pool_k), Guarded(pool_v)
    l4l.l4l_kv_append_paged(gk.t, gv.t, torch.from_numpy(table).cuda(), k_new.cuda(), v_new.cuda(),
                            torch.tensor(lens, dtype=torch.int32).cuda(), torch.tensor(n_new, dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    assert gk.margins_intact() and gv.margins_intact()
    assert np.array_equal(orc.bits(gk.t.cpu()), ref_k) and np.array_equal(orc.bits(gv.t.cpu()), ref_v)
    # decode over what was appended (sequences 0, 1 and 3 only: sequence 2's tail has no pages)
    new_lens = [lens[0] + T, lens[1] + 5, 0, lens[3]]
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ref, _ = orc.decode_paged(q, ref_k, ref_v, table, np.array(new_lens, np.int32), 0.1)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, max(new_lens))
    l4l.l4l_attn_decode_paged(q.cuda(), o, gk.t, gv.t, torch.from_numpy(table).cuda(),
                              torch.tensor(new_lens, dtype=torch.int32).cuda(), max(new_lens), 0.1, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, "decode after paged append")


def test_paged_rejects_bad_pools():
    q = torch.zeros(1, 4, 64, dtype=torch.bfloat16, device="cuda")
    table = torch.zeros(1, 2, dtype=torch.int32, device="cuda")
    lens = torch.ones(1, dtype=torch.int32, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 1, 4, 2, 64, 48)
    for page in (8, 24):                          # below 16, not a power of two
        pool = torch.zeros(3, 2, page, 64, dtype=torch.bfloat16, device="cuda")
        with pytest.raises(l4l.L4LError):
            l4l.l4l_attn_decode_paged(q, q.clone(), pool, pool.clone(), table, lens, page, 0.1, ws)
    pool = torch.zeros(3, 2, 16, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(l4l.L4LError):             # longer than the table can describe
        l4l.l4l_attn_decode_paged(q, q.clone(), pool, pool.clone(), table, lens, 33, 0.1, ws)
