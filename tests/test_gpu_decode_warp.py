"""The decode kernel for many short sequences (one warp per (sequence, KV head), no merge) against the fp64 oracle,
forced on through the tuning override for small shapes, and chosen by the library for the regime it is made for."""
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
def warp_kernel(request):
    """'1': every eligible decode call runs on the warp kernel; '0': never; None: the library's choice."""
    mode = getattr(request, "param", "1")
    with l4l.decode_override(warp=-1 if mode is None else int(mode)):
        yield mode


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (8, 8), (8, 1), (3, 1), (6, 2), (32, 8), (16, 1), (24, 2)])
def test_warp_decode_ragged_edge_lengths(warp_kernel, D, Hq, Hkv):
    # around every boundary: empty, one token, 16-token chunks, more chunks than ring stages
    lens = [0, 1, 2, 15, 16, 17, 31, 32, 33, 47, 48, 127, 128, 129, 255, 300, 0, 7]
    q, ck, cv, kv_len = random_batch(len(lens), Hq, Hkv, D, 304, lens, seed=1900 + D + Hq)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(D))


@pytest.mark.parametrize("B", [1, 7, 200, 1024, 1500])
def test_warp_decode_batch_sizes(warp_kernel, B):
    # fewer units than warps, one full launch slice, more than one slice
    g = np.random.default_rng(B)
    lens = g.integers(0, 200, size=B).tolist()
    q, ck, cv, kv_len = random_batch(B, 8, 2, 128, 208, lens, seed=B)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128))


def test_warp_decode_long_sequences_too(warp_kernel):
    # not its regime, but correct there as well: hundreds of chunks per unit
    lens = [4000, 2500, 1, 4096]
    q, ck, cv, kv_len = random_batch(4, 8, 2, 128, 4096, lens, seed=3)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128))


def test_warp_decode_extreme_scores_token_major_cache_and_clamp(warp_kernel):
    lens = [300, 1, 129, 64]
    q, ck, cv, kv_len = random_batch(4, 8, 2, 128, 384, lens, seed=77)
    check_decode(q, ck, cv, kv_len, 1.0)
    check_decode(q, ck, cv, kv_len, -0.25)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(128), strided_cache=True)
    B, Hq, D = q.shape
    clamp = 100                                   # kv_lens above max_kv_len are clamped to it
    ref, _ = orc.decode(q, ck, cv, np.minimum(kv_len.numpy(), clamp), 0.1)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, 2, D, clamp)
    l4l.l4l_attn_decode(q.cuda(), o, ck.cuda(), cv.cuda(), kv_len.cuda(), clamp, 0.1, ws)
    torch.cuda.synchronize()
    assert_close_to_oracle(o, ref, "clamped decode")


@pytest.mark.parametrize("D,Hq,Hkv", [(128, 8, 2), (64, 4, 4), (128, 8, 1), (128, 32, 8), (128, 16, 1), (64, 26, 2)])
def test_warp_decode_with_fused_append(warp_kernel, D, Hq, Hkv):
    from test_gpu_decode_append import make_case

    lens = [0, 1, 2, 16, 17, 32, 33, 128, 129, 300, 255, 256]
    B, Lmax = len(lens), 304
    q, ck, cv, kn, vn, kv_len = make_case(B, Hq, Hkv, D, Lmax, lens, seed=140 + D + Hq)
    scale = 1.0 / math.sqrt(D)
    pos = (kv_len - 1).clamp(min=0).numpy()
    n_new = (kv_len > 0).to(torch.int32).numpy()
    ek, ev = orc.kv_append(ck, cv, kn, vn, pos, n_new)
    ek_t = torch.from_numpy(ek.view(np.int16)).view(torch.bfloat16)
    ev_t = torch.from_numpy(ev.view(np.int16)).view(torch.bfloat16)
    ref, ref_lse = orc.decode(q, ek_t, ev_t, kv_len.numpy(), scale)
    gk, gv, go = Guarded(ck), Guarded(cv), Guarded(nan_bf16((B, Hq, D)))
    lse = torch.zeros(B, Hq, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_append(q.cuda(), go.t, gk.t, gv.t, kn.cuda(), vn.cuda(), kv_len.cuda(), Lmax, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for g in (gk, gv, go):
        assert g.margins_intact()
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)
    assert_close_to_oracle(go.t, ref, "warp decode_append o")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


@pytest.mark.parametrize("page", [16, 64, 256])
@pytest.mark.parametrize("Hq,Hkv,D", [(32, 8, 128), (12, 12, 64)])
def test_warp_decode_paged_with_and_without_append(warp_kernel, page, Hq, Hkv, D):
    from test_gpu_paged import test_paged_decode_matches_oracle
    from test_gpu_paged_append import run_case

    test_paged_decode_matches_oracle(page, Hq, Hkv, D)
    lens = [1, 16, 17, 128, 129, 257, 300, 33, 0, 64]
    run_case(len(lens), Hq, Hkv, D, page, lens, seed=2200 + page + D)
    run_case(len(lens), Hq, Hkv, D, page, lens, seed=2300 + page + D, drop=(1, 4, 6))


@pytest.mark.parametrize("warp_kernel", [None, "0"], indirect=True)
def test_library_picks_the_warp_kernel_for_many_short_sequences(warp_kernel):
    """B = 400 sequences of 1 to 256 tokens on 8 KV heads is inside the regime the library hands to the warp kernel;
    the same call kept off it must agree within the tolerance of both."""
    B, Hq, Hkv, D = 400, 32, 8, 128
    g = np.random.default_rng(11)
    lens = g.integers(1, 257, size=B).tolist()
    q, ck, cv, kv_len = random_batch(B, Hq, Hkv, D, 256, lens, seed=12)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(D))


@pytest.mark.parametrize("warp_kernel", [None], indirect=True)
def test_kernel_choice_by_problem_size(warp_kernel):
    """The three decode kernels and the regimes the library gives them (8B-shaped layer: 32 query heads on 8 KV heads)."""
    with l4l.decode_override(cluster=-1):
        assert l4l.l4l_decode_kernel_choice(1, 32, 8, 128, 2304) == ("cluster", 8)          # one sequence: latency-bound
        assert l4l.l4l_decode_kernel_choice(4, 32, 8, 128, 2304)[0] == "cluster"
        assert l4l.l4l_decode_kernel_choice(32, 32, 8, 128, 4096) == ("split", 8)            # the benchmark batch
        assert l4l.l4l_decode_kernel_choice(64, 12, 12, 64, 1024) == ("split", 4)            # small MHA model
        assert l4l.l4l_decode_kernel_choice(512, 32, 8, 128, 256) == ("warp", 0)             # hundreds of short sequences
        assert l4l.l4l_decode_kernel_choice(512, 32, 8, 128, 4096)[0] == "split"             # ... but not long ones
        assert l4l.l4l_decode_kernel_choice(512, 32, 8, 128, 256, fp8=True)[0] == "warp"     # also with an fp8 cache
        assert l4l.l4l_decode_kernel_choice(32, 128, 8, 128, 4096) == ("split", 6)           # groups of 16 query heads
        assert l4l.l4l_decode_kernel_choice(1, 32, 8, 96, 128) is None                       # unsupported head_dim


@pytest.mark.parametrize("seed", range(16))
def test_warp_decode_random_shapes(warp_kernel, seed):
    """Seeded random shapes, length mixes, page sizes and group sizes through the warp-per-unit kernel (forced on),
    without and with the fused append: a net for the index arithmetic of its unit queue and rings."""
    from test_gpu_random_shapes import random_lengths
    from test_gpu_paged import build_pool

    rng = np.random.default_rng(7000 + seed)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    G = int(rng.choice([1, 2, 4, 5, 8, 12, 16]))
    Hq = Hkv * G
    B = int(rng.choice([1, 2, 9, 40, 150, 700]))
    Lmax = int(rng.choice([48, 96, 300, 700]))
    lens = random_lengths(rng, B, Lmax)
    q, ck, cv, kv_len = random_batch(B, Hq, Hkv, D, Lmax, lens.tolist(), seed=seed)
    scale = float(rng.choice([1.0 / math.sqrt(D), 0.05, -0.03]))
    check_decode(q, ck, cv, kv_len, scale)
    # fused append over a paged copy of the same lengths (the new token is the last one of every sequence)
    page = int(rng.choice([16, 32, 64, 128]))
    g = torch.Generator().manual_seed(100 + seed)
    pool_k, pool_v, table = build_pool(B, Hkv, D, page, lens.tolist(), seed=200 + seed)
    kn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
    vn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
    pos = np.maximum(lens - 1, 0)
    ref_k, ref_v = orc.kv_append_paged(pool_k, pool_v, table, kn, vn, pos, (lens > 0).astype(np.int32))
    ref, _ = orc.decode_paged(q, ref_k, ref_v, table, lens, scale)
    gk, gv = Guarded(pool_k), Guarded(pool_v)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    max_len = max(int(lens.max()), 1)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, max_len)
    l4l.l4l_attn_decode_paged_append(q.cuda(), o, gk.t, gv.t, torch.from_numpy(table).cuda(), kn.cuda(), vn.cuda(),
                                     torch.from_numpy(lens).cuda(), max_len, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert gk.margins_intact() and gv.margins_intact()
    assert np.array_equal(orc.bits(gk.t.cpu()), ref_k) and np.array_equal(orc.bits(gv.t.cpu()), ref_v)
    assert_close_to_oracle(o.cpu(), ref, f"paged decode + append, seed {seed}")


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (8, 8), (16, 2), (16, 1)])
def test_warp_decode_fp8_cache(warp_kernel, Hq, Hkv):
    """The fp8 (e4m3) variant of the warp-per-unit kernel against the oracle over the codes: contiguous and paged
    caches; the fused append of an fp8 cache is not this kernel's (the call must still be served, by the split kernel)."""
    import test_gpu_fp8 as f8

    assert l4l.l4l_decode_kernel_choice(13, Hq, Hkv, 128, 2304, fp8=True)[0] == "warp"       # forced on by the fixture
    f8.test_fp8_decode_matches_oracle(Hq, Hkv, 128)
    f8._fp8_append_case(Hq, Hkv, [1, 16, 17, 33, 255, 300, 0], seed=3500 + Hq, Lmax=320)


@pytest.mark.parametrize("page", [16, 64, 256])
def test_warp_decode_fp8_paged_cache(warp_kernel, page):
    import test_gpu_fp8 as f8

    f8.test_fp8_paged_decode_matches_oracle(page, 128)


def test_warp_decode_fp8_many_short_sequences(warp_kernel):
    import test_gpu_fp8 as f8

    rng = np.random.default_rng(5)
    B, Hq, Hkv, D, Lmax = 600, 8, 4, 128, 160
    lens = rng.integers(0, Lmax + 1, size=B)
    g = torch.Generator().manual_seed(6)
    ck8 = f8.random_codes((B, Hkv, Lmax, D), g, 7)
    cv8 = f8.random_codes((B, Hkv, Lmax, D), g, 7)
    for b, L in enumerate(lens):
        ck8[b, :, L:] = 0x7F
        cv8[b, :, L:] = 0xFF
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ks, vs = torch.rand(Hkv, generator=g) + 0.5, torch.rand(Hkv, generator=g) + 0.25
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.decode_fp8(q, ck8, cv8, lens.astype(np.int32), ks.numpy(), vs.numpy(), scale)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, Hq, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_fp8(q.cuda(), o, ck8.cuda(), cv8.cuda(), ks.cuda(), vs.cuda(),
                            torch.from_numpy(lens.astype(np.int32)).cuda(), Lmax, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert_close_to_oracle(o.cpu(), ref, "fp8 decode, many short sequences")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4), (16, 1), (32, 8)])
@pytest.mark.parametrize("norm", [False, True])
@pytest.mark.parametrize("page", [None, 32])
def test_warp_decode_step_with_rope_and_append_in_one_launch(warp_kernel, D, Hq, Hkv, norm, page):
    """The whole decode step (rotary embedding and optional RMS norm of the new token's q and k, cache update,
    attention) on the warp-per-unit kernel, against the oracle chain rope -> append -> decode over several steps."""
    from paper_2608_21836_b200.workloads import make_rope_tables
    from test_gpu_rope_append import assert_bf16_close

    B, Lmax, steps, n_pos = 9, 320, 3, 320
    lens = np.array([1, 2, 16, 17, 33, 128, 129, 250, 310], np.int32)     # kv_len INCLUDING the new token at the first step
    g = torch.Generator().manual_seed(1900 + D + Hq + norm)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cos, sin = make_rope_tables(n_pos, D)
    qw = (torch.rand(D, generator=g) + 0.5) if norm else None
    kw = (torch.rand(D, generator=g) + 0.5) if norm else None
    eps = 1e-6 if norm else 0.0
    scale = 1.0 / math.sqrt(D)
    ock, ocv = orc.bits(ck), orc.bits(cv)
    if page is None:
        dck, dcv, table = ck.cuda(), cv.cuda(), None
    else:
        n_per = Lmax // page
        table = torch.randperm(B * n_per, generator=g).view(B, n_per).to(torch.int32)
        pool_k = torch.zeros(B * n_per, Hkv, page, D, dtype=torch.bfloat16)
        pool_v = torch.zeros_like(pool_k)
        for b in range(B):
            for i in range(n_per):
                pool_k[table[b, i]] = ck[b, :, i * page:(i + 1) * page]
                pool_v[table[b, i]] = cv[b, :, i * page:(i + 1) * page]
        dck, dcv = pool_k.cuda(), pool_v.cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    dcos, dsin = cos.cuda(), sin.cuda()
    assert l4l.l4l_decode_kernel_choice(B, Hq, Hkv, D, Lmax)[0] == "warp"           # forced on by the fixture
    for s in range(steps):
        q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
        kn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
        vn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
        cur = lens + s
        oq, ock, ocv, _, _ = orc.rope_kv_append(q.view(B, 1, Hq, D), kn, vn, ock, ocv, cur - 1, None, cos.numpy(),
                                                sin.numpy(), None if qw is None else qw.numpy(),
                                                None if kw is None else kw.numpy(), eps)
        ref, _ = orc.decode(oq[:, 0], ock, ocv, cur, scale)
        o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
        kwargs = dict(q_weight=None if qw is None else qw.cuda(), k_weight=None if kw is None else kw.cuda(), eps=eps)
        if page is None:
            l4l.l4l_attn_decode_rope_append(q.cuda(), o, dck, dcv, kn.cuda(), vn.cuda(), torch.from_numpy(cur).cuda(), Lmax,
                                            scale, dcos, dsin, ws, **kwargs)
        else:
            l4l.l4l_attn_decode_paged_rope_append(q.cuda(), o, dck, dcv, table.cuda(), kn.cuda(), vn.cuda(),
                                                  torch.from_numpy(cur).cuda(), Lmax, scale, dcos, dsin, ws, **kwargs)
        torch.cuda.synchronize()
        assert l4l.l4l_last_device_error(ws) == 0
        assert_close_to_oracle(o.cpu(), ref, f"warp kernel: rope + append + decode, step {s}")
    if page is None:
        assert_bf16_close(dck, ock, "cache k after the fused steps")
        assert np.array_equal(orc.bits(dcv.cpu()), ocv)
    else:
        got_k = orc.gather_pages(dck.cpu(), table.numpy(), Lmax)
        assert_bf16_close(torch.from_numpy(got_k.view(np.int16)).view(torch.bfloat16), ock, "paged cache k after the fused steps")
        assert np.array_equal(orc.gather_pages(dcv.cpu(), table.numpy(), Lmax), ocv)
