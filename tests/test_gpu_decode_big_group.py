"""Query-head groups of 5 to 16 at head_dim 128 on the split decode kernel: the consumer warps hand their results to one
finisher warp per 4 heads in 16-bit rows (one rounding to bf16 per warp and piece ahead of the merge; 5 to 8 heads on
the 8-warp shape, 9 to 16 on a 6-warp shape with 96-token tiles), so these shapes get their own parity cases: long
ragged sequences cut between CTAs, the fused append, the fp8 cache."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, assert_close_to_oracle, bits_equal, nan_bf16
from test_gpu_decode import check_decode, random_batch

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def split_kernel_only():
    with l4l.decode_override(cluster=0):
        yield


@pytest.mark.parametrize("Hq,Hkv", [(40, 8), (48, 8), (56, 8), (64, 8), (8, 1), (5, 1), (72, 8), (96, 8), (128, 8), (16, 1),
                                    (13, 1)])
def test_big_group_decode_long_ragged(Hq, Hkv):
    lens = [4096, 0, 1, 129, 3000, 2049, 513, 17, 4000, 1234, 3333, 640]
    q, ck, cv, kv_len = random_batch(len(lens), Hq, Hkv, 128, 4096, lens, seed=300 + Hq)
    _, stats = check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128))


@pytest.mark.parametrize("Hq", [64, 128])
def test_big_group_decode_many_sequences_cut_between_ctas(Hq):
    # enough tiles that every CTA streams a range and most sequences are cut once
    g = torch.Generator().manual_seed(77)
    lens = torch.randint(512, 4097, (40,), generator=g).tolist()
    q, ck, cv, kv_len = random_batch(len(lens), Hq, 8, 128, 4096, lens, seed=78)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128))


@pytest.mark.parametrize("Hq", [64, 128])
def test_big_group_decode_with_fused_append(Hq):
    from test_gpu_decode_append import make_case

    Hkv, D = 8, 128
    lens = [0, 1, 2, 16, 17, 128, 129, 300, 1000, 2048]
    B, Lmax = len(lens), 2048
    q, ck, cv, kn, vn, kv_len = make_case(B, Hq, Hkv, D, Lmax, lens, seed=41)
    scale = 1.0 / math.sqrt(D)
    pos = (kv_len - 1).clamp(min=0).numpy()
    n_new = (kv_len > 0).to(torch.int32).numpy()
    ek, ev = orc.kv_append(ck, cv, kn, vn, pos, n_new)
    ek_t = torch.from_numpy(ek.view(np.int16)).view(torch.bfloat16)
    ev_t = torch.from_numpy(ev.view(np.int16)).view(torch.bfloat16)
    ref, _ = orc.decode(q, ek_t, ev_t, kv_len.numpy(), scale)
    gk, gv, go = Guarded(ck), Guarded(cv), Guarded(nan_bf16((B, Hq, D)))
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_append(q.cuda(), go.t, gk.t, gv.t, kn.cuda(), vn.cuda(), kv_len.cuda(), Lmax, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for gd in (gk, gv, go):
        assert gd.margins_intact()
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)
    assert_close_to_oracle(go.t, ref, "big-group decode_append o")


def test_big_group_decode_fp8_cache():
    from test_gpu_fp8 import test_fp8_decode_matches_oracle as fp8_case

    fp8_case(64, 8, 128)
    fp8_case(40, 8, 128)
    fp8_case(128, 8, 128)


@pytest.mark.parametrize("Hq,page_size", [(64, 64), (64, 16), (128, 256), (128, 64), (128, 32), (128, 16)])
def test_big_group_decode_paged(Hq, page_size):
    # groups of 8 on the 8-warp shape; groups of 16 on the 6-warp shape with pages of 16 or 32 tokens (its 96-token
    # tiles do not line up with larger pages: those stay on the 4-warp shape)
    B, Hkv, D = 6, 8, 128
    lens = np.array([0, 1, 130, 700, 2048, 1999], np.int32)
    g = torch.Generator().manual_seed(4321 + page_size + Hq)
    max_pages = (2048 + page_size - 1) // page_size
    n_pages = B * max_pages + 3
    pool_k = torch.randn(n_pages, Hkv, page_size, D, generator=g).to(torch.bfloat16)
    pool_v = torch.randn(n_pages, Hkv, page_size, D, generator=g).to(torch.bfloat16)
    perm = torch.randperm(n_pages, generator=g)[:B * max_pages].to(torch.int32).view(B, max_pages)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    ref, _ = orc.decode_paged(q, pool_k, pool_v, perm.numpy(), lens, scale)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, 2048)
    l4l.l4l_attn_decode_paged(q.cuda(), o, pool_k.cuda(), pool_v.cuda(), perm.cuda(), torch.from_numpy(lens).cuda(),
                              2048, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o, ref, "big-group paged decode")
