"""Sizes well past the benchmark's: one sequence of 200 000 cached tokens through decode (every kernel choice the library
makes for it, contiguous and as a pool of 16-token pages), and a 32 768-token prompt through prefill on sampled rows.
They guard the index arithmetic (tile counts, partition of the tile stream, slot and page offsets) where it grows."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import assert_close_to_oracle, bits_equal, nan_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("D,Hq,Hkv", [(128, 8, 2), (64, 4, 4)])
def test_decode_of_a_very_long_sequence(D, Hq, Hkv):
    L, Lmax, B = 200_003, 200_064, 2
    g = torch.Generator().manual_seed(D)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = (torch.randn(B, Hkv, Lmax, D, generator=g)).to(torch.bfloat16)
    cv = (torch.randn(B, Hkv, Lmax, D, generator=g)).to(torch.bfloat16)
    lens = np.array([L, 777], np.int32)
    for b in range(B):
        ck[b, :, lens[b]:] = nan_bf16((1,))
        cv[b, :, lens[b]:] = nan_bf16((1,))
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.decode(q, ck, cv, lens, scale)
    dq, dck, dcv, dl = q.cuda(), ck.cuda(), cv.cuda(), torch.from_numpy(lens).cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    for cluster in (-1, 0):                                   # the library's choice, then the split kernel
        with l4l.decode_override(cluster=cluster):
            o = torch.zeros_like(dq)
            lse = torch.zeros(B, Hq, device="cuda")
            l4l.l4l_attn_decode(dq, o, dck, dcv, dl, Lmax, scale, ws, lse=lse)
            torch.cuda.synchronize()
            assert l4l.l4l_last_device_error(ws) == 0
            assert_close_to_oracle(o.cpu(), ref, f"decode of {L} tokens (cluster={cluster})")
            assert np.abs(lse.cpu().double().numpy() - ref_lse).max() <= 2e-3
    # the same cache as a pool of 16-token pages in reverse order
    page = 16
    n_per = Lmax // page
    tbl = torch.arange(B * n_per - 1, -1, -1, dtype=torch.int32).view(B, n_per)
    pool_k = torch.empty(B * n_per, Hkv, page, D, dtype=torch.bfloat16)
    pool_v = torch.empty_like(pool_k)
    pool_k[tbl.reshape(-1).long()] = ck.view(B, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(-1, Hkv, page, D)
    pool_v[tbl.reshape(-1).long()] = cv.view(B, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(-1, Hkv, page, D)
    o = torch.zeros_like(dq)
    l4l.l4l_attn_decode_paged(dq, o, pool_k.cuda(), pool_v.cuda(), tbl.cuda(), dl, Lmax, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, f"paged decode of {L} tokens")


def test_prefill_of_a_very_long_prompt_on_sampled_rows():
    B, S, Hq, Hkv, D = 1, 32_768, 4, 2, 128
    g = torch.Generator().manual_seed(9)
    q = torch.randn(B, S, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    L = S - 37                                                 # a ragged end inside the last block
    scale = 1.0 / math.sqrt(D)
    o = torch.zeros(B, S, Hq, D, dtype=torch.bfloat16, device="cuda")
    ck, cv = nan_bf16((B, Hkv, S, D)).cuda(), nan_bf16((B, Hkv, S, D)).cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill(q.cuda(), k.cuda(), v.cuda(), o, torch.tensor([L], dtype=torch.int32).cuda(), scale, ws,
                         cache_k=ck, cache_v=cv)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    want_k, want_v = k.permute(0, 2, 1, 3)[:, :, :L].contiguous(), v.permute(0, 2, 1, 3)[:, :, :L].contiguous()
    assert bits_equal(ck[:, :, :L].contiguous(), want_k) and bits_equal(cv[:, :, :L].contiguous(), want_v)
    rng = np.random.default_rng(11)
    toks = sorted(set([0, 1, 127, 128, 255, 256, 16383, 16384, L - 129, L - 128, L - 2, L - 1] + rng.integers(0, L, 200).tolist()))
    rows = [(0, i, h) for i in toks for h in range(Hq)]
    ref, _ = orc.prefill_rows(q, k, v, np.array([L], np.int32), scale, rows)
    idx = torch.as_tensor(rows)
    assert_close_to_oracle(o.cpu()[idx[:, 0], idx[:, 1], idx[:, 2]], ref, "32768-token prompt, sampled rows")
    assert (o[:, L:] == 0).all()                               # rows past the prompt's end are not written
