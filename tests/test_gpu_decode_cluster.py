"""The small-batch decode kernel (one thread-block cluster per (sequence, KV head), partials merged through
distributed shared memory) against the fp64 oracle, at every cluster width, through the public entry points."""
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


@pytest.fixture
def cluster_width(request):
    with l4l.decode_override(cluster=int(request.param)):
        yield request.param


WIDTHS = [1, 2, 4, 8]


@pytest.mark.parametrize("cluster_width", WIDTHS, indirect=True)
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (8, 8), (16, 1), (3, 1), (6, 2)])
def test_cluster_decode_ragged_edge_lengths(cluster_width, D, Hq, Hkv):
    # lengths around every boundary: empty, one token, 16-token groups, tiles, fewer tiles than CTAs, many tiles
    lens = [0, 1, 2, 15, 16, 17, 127, 128, 129, 255, 257, 1000, 2047, 2048]
    q, ck, cv, kv_len = random_batch(len(lens), Hq, Hkv, D, 2048, lens, seed=900 + D + Hq + cluster_width)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(D))


@pytest.mark.parametrize("cluster_width", [2, 8], indirect=True)
def test_cluster_decode_long_sequence_ring_wraps(cluster_width):
    # more tiles per CTA than ring stages: the producer waits for the consumers
    lens = [8191, 5000]
    q, ck, cv, kv_len = random_batch(2, 8, 2, 128, 8192, lens, seed=31 + cluster_width)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128))


@pytest.mark.parametrize("cluster_width", [1, 4, 8], indirect=True)
def test_cluster_decode_extreme_scores_and_negative_scale(cluster_width):
    lens = [300, 1, 129]
    # scale 1 on N(0,1) inputs: scores with a standard deviation of ~11, a few keys take all the weight
    q, ck, cv, kv_len = random_batch(3, 8, 2, 128, 384, lens, seed=77)
    check_decode(q, ck, cv, kv_len, 1.0)
    check_decode(q, ck, cv, kv_len, -0.25)


@pytest.mark.parametrize("cluster_width", [1, 4, 8], indirect=True)
def test_cluster_decode_token_major_cache_and_max_kv_len_clamp(cluster_width):
    lens = [500, 64, 0, 333]
    q, ck, cv, kv_len = random_batch(4, 8, 2, 128, 512, lens, seed=5)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128), strided_cache=True)
    # kv_lens above max_kv_len are clamped to it
    B, Hq, D = q.shape
    clamp = 256
    ref, _ = orc.decode(q, ck, cv, np.minimum(kv_len.numpy(), clamp), 0.1)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, 2, D, clamp)
    l4l.l4l_attn_decode(q.cuda(), o, ck.cuda(), cv.cuda(), kv_len.cuda(), clamp, 0.1, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o, ref, "clamped decode")


@pytest.mark.parametrize("cluster_width", WIDTHS, indirect=True)
@pytest.mark.parametrize("D,Hq,Hkv", [(128, 8, 2), (64, 4, 4), (128, 16, 1)])
def test_cluster_decode_with_fused_append(cluster_width, D, Hq, Hkv):
    from test_gpu_decode_append import make_case

    lens = [0, 1, 2, 16, 17, 128, 129, 300, 1000, 1024]
    B, Lmax = len(lens), 1024
    q, ck, cv, kn, vn, kv_len = make_case(B, Hq, Hkv, D, Lmax, lens, seed=40 + D + cluster_width)
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
    for g in (gk, gv, go):
        assert g.margins_intact()
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)
    assert_close_to_oracle(go.t, ref, "cluster decode_append o")


@pytest.mark.parametrize("cluster_width", [1, 4, 8], indirect=True)
@pytest.mark.parametrize("page_size", [16, 64, 256])
def test_cluster_decode_paged(cluster_width, page_size):
    B, Hq, Hkv, D = 5, 8, 2, 128
    lens = np.array([0, 1, 130, 700, 1024], np.int32)
    g = torch.Generator().manual_seed(1234 + page_size)
    max_pages = (1024 + page_size - 1) // page_size
    n_pages = B * max_pages + 3
    pool_k = torch.randn(n_pages, Hkv, page_size, D, generator=g).to(torch.bfloat16)
    pool_v = torch.randn(n_pages, Hkv, page_size, D, generator=g).to(torch.bfloat16)
    perm = torch.randperm(n_pages, generator=g)[:B * max_pages].to(torch.int32).view(B, max_pages)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    ref, _ = orc.decode_paged(q, pool_k, pool_v, perm.numpy(), lens, scale)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, 1024)
    l4l.l4l_attn_decode_paged(q.cuda(), o, pool_k.cuda(), pool_v.cuda(), perm.cuda(), torch.from_numpy(lens).cuda(),
                              1024, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o, ref, "cluster paged decode")


@pytest.mark.parametrize("cluster_width", WIDTHS, indirect=True)
@pytest.mark.parametrize("D,Hq,Hkv,norm", [(128, 8, 2, True), (64, 4, 4, False), (128, 16, 1, True)])
def test_cluster_decode_step_with_rope_and_append(cluster_width, D, Hq, Hkv, norm):
    from test_gpu_rope_append import test_decode_step_with_rope_and_append_in_one_launch as rope_step_case

    rope_step_case(D, Hq, Hkv, norm)


@pytest.mark.parametrize("cluster_width", WIDTHS, indirect=True)
def test_cluster_decode_fp8_cache(cluster_width):
    from test_gpu_fp8 import test_fp8_decode_matches_oracle as fp8_case

    fp8_case(16, 2, 128)
    fp8_case(8, 8, 128)


@pytest.mark.parametrize("cluster_width", [1, 4, 8], indirect=True)
@pytest.mark.parametrize("page", [16, 64, 256])
def test_cluster_decode_fp8_paged(cluster_width, page):
    from test_gpu_fp8 import test_fp8_paged_decode_matches_oracle as fp8_paged_case

    fp8_paged_case(page, 128)


def test_library_choice_matches_split_kernel_result():
    # the same call on both kernels: results agree to rounding of the merge order
    lens = [2304]
    q, ck, cv, kv_len = random_batch(1, 32, 8, 128, 2304, lens, seed=3)
    outs = []
    for mode in (0, -1):
        with l4l.decode_override(cluster=mode):
            o = torch.zeros(1, 32, 128, dtype=torch.bfloat16, device="cuda")
            ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 1, 32, 8, 128, 2304)
            l4l.l4l_attn_decode(q.cuda(), o, ck.cuda(), cv.cuda(), kv_len.cuda(), 2304, 1.0 / math.sqrt(128), ws)
            torch.cuda.synchronize()
            assert l4l.l4l_last_device_error(ws) == 0
            outs.append(o.float().cpu())
    assert (outs[0] - outs[1]).abs().max() <= 2e-2
