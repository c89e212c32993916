"""Seeded random shapes and length mixes through the decode family and the prefill family, each against the oracle:
a net for index arithmetic that the hand-picked edge cases might miss (tile partition over CTAs, batch slicing,
page tables, group sizes, ragged tails)."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import assert_close_to_oracle, nan_bf16

pytestmark = pytest.mark.gpu


def random_lengths(rng, B, Lmax):
    kind = rng.integers(0, 4)
    if kind == 0:
        lens = rng.integers(0, Lmax + 1, B)
    elif kind == 1:                                     # mostly short, a few very long
        lens = np.where(rng.random(B) < 0.15, rng.integers(Lmax // 2, Lmax + 1, B), rng.integers(0, 40, B))
    elif kind == 2:                                     # around tile boundaries
        lens = np.clip(rng.choice([16, 64, 128, 256, 512], B) + rng.integers(-2, 3, B), 0, Lmax)
    else:
        lens = np.full(B, rng.integers(1, Lmax + 1))
    return lens.astype(np.int32)


@pytest.mark.parametrize("seed", range(12))
def test_decode_family_random(seed):
    rng = np.random.default_rng(4000 + seed)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    G = int(rng.choice([1, 2, 4, 5, 8, 16]))
    Hq = Hkv * G
    B = int(rng.choice([1, 2, 7, 33, 70]))
    Lmax = int(rng.choice([96, 700, 2100]))
    lens = random_lengths(rng, B, Lmax)
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= torch.from_numpy(lens).view(B, 1, 1, 1)
    ck = torch.where(dead, nan_bf16((1,)), ck).contiguous()
    cv = torch.where(dead, nan_bf16((1,)), cv).contiguous()
    scale = float(rng.choice([1.0 / math.sqrt(D), 0.05, -0.03]))
    ref, ref_lse = orc.decode(q, ck, cv, lens, scale)
    dq, dck, dcv, dl = q.cuda(), ck.cuda(), cv.cuda(), torch.from_numpy(lens).cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    o = torch.zeros_like(dq)
    lse = torch.zeros(B, Hq, device="cuda")
    l4l.l4l_attn_decode(dq, o, dck, dcv, dl, Lmax, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, f"decode seed {seed}")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    # the same cache cut into pages of a random size, scattered
    page = int(rng.choice([16, 32, 64, 128]))
    n_per = (Lmax + page - 1) // page
    perm = rng.permutation(B * n_per + 3)[: B * n_per].reshape(B, n_per).astype(np.int32)
    pool_k = nan_bf16((B * n_per + 3, Hkv, page, D))
    pool_v = nan_bf16((B * n_per + 3, Hkv, page, D))
    pad = n_per * page - Lmax
    ckp = torch.cat([ck, nan_bf16((B, Hkv, pad, D))], 2) if pad else ck
    cvp = torch.cat([cv, nan_bf16((B, Hkv, pad, D))], 2) if pad else cv
    pool_k[torch.from_numpy(perm.reshape(-1)).long()] = ckp.view(B, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(-1, Hkv, page, D)
    pool_v[torch.from_numpy(perm.reshape(-1)).long()] = cvp.view(B, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(-1, Hkv, page, D)
    o2 = torch.zeros_like(dq)
    l4l.l4l_attn_decode_paged(dq, o2, pool_k.cuda(), pool_v.cuda(), torch.from_numpy(perm).cuda(), dl, Lmax, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o2.cpu(), ref, f"paged decode seed {seed}, page {page}")
    if D == 128:
        codes_k = torch.from_numpy(rng.integers(0, 256, (B, Hkv, Lmax, D), dtype=np.uint8))
        codes_v = torch.from_numpy(rng.integers(0, 256, (B, Hkv, Lmax, D), dtype=np.uint8))
        for c in (codes_k, codes_v):                    # no NaN codes, magnitudes below 2
            c[(c & 0x78) > 0x38] &= 0xBF
        ks = torch.from_numpy(rng.uniform(0.5, 1.5, Hkv).astype(np.float32))
        vs = torch.from_numpy(rng.uniform(0.5, 1.5, Hkv).astype(np.float32))
        ref8, _ = orc.decode_fp8(q, codes_k, codes_v, lens, ks.numpy(), vs.numpy(), abs(scale))
        o3 = torch.zeros_like(dq)
        l4l.l4l_attn_decode_fp8(dq, o3, codes_k.cuda(), codes_v.cuda(), ks.cuda(), vs.cuda(), dl, Lmax, abs(scale), ws)
        torch.cuda.synchronize()
        assert l4l.l4l_last_device_error(ws) == 0
        assert_close_to_oracle(o3.cpu(), ref8, f"fp8 decode seed {seed}")


def test_decode_more_sequences_than_one_launch_slices():
    """600 short sequences: beyond the per-launch limit of the prefix-sum array, so the call is cut into slices."""
    B, Hq, Hkv, D, Lmax = 600, 4, 2, 64, 48
    rng = np.random.default_rng(77)
    lens = rng.integers(0, Lmax + 1, B).astype(np.int32)
    g = torch.Generator().manual_seed(77)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    ref, _ = orc.decode(q, ck, cv, lens, 0.125)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode(q.cuda(), o, ck.cuda(), cv.cuda(), torch.from_numpy(lens).cuda(), Lmax, 0.125, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, "decode, 600 sequences")


@pytest.mark.parametrize("seed", range(8))
def test_prefill_family_random(seed):
    rng = np.random.default_rng(5000 + seed)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hq = Hkv * G
    B = int(rng.choice([1, 2, 3]))
    S = int(rng.choice([100, 257, 600]))
    lens = rng.integers(0, S + 1, B).astype(np.int32)
    lens[rng.integers(0, B)] = S
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, S, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    ref, _ = orc.prefill(q, k, v, lens, scale)
    dq, dk, dv, dl = q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(lens).cuda()
    ck = nan_bf16((B, Hkv, S, D)).cuda()
    cv = nan_bf16((B, Hkv, S, D)).cuda()
    o = torch.zeros_like(dq)
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill(dq, dk, dv, o, dl, scale, ws, cache_k=ck, cache_v=cv)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    valid = (torch.arange(S).view(1, S) < torch.from_numpy(lens).view(B, 1))
    assert_close_to_oracle(o.cpu()[valid], ref[valid.numpy()], f"prefill seed {seed}")
    # the same sequences as a cached prefix of random length plus a chunk, read from the cache the prefill wrote
    past = np.array([int(rng.integers(0, L + 1)) for L in lens], np.int32)
    qlen = (lens - past).astype(np.int32)
    Sc = max(int(qlen.max()), 1)
    qc = torch.zeros(B, Sc, Hq, D, dtype=torch.bfloat16)
    for b in range(B):
        qc[b, :qlen[b]] = q[b, past[b]:lens[b]]
    oc = torch.zeros(B, Sc, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_prefill_chunk(qc.cuda(), oc, ck, cv, torch.from_numpy(past).cuda(), torch.from_numpy(qlen).cuda(), scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for b in range(B):
        if qlen[b] > 0:
            assert_close_to_oracle(oc[b, :qlen[b]].cpu(), ref[b, past[b]:lens[b]], f"chunk seed {seed} sequence {b}")
    # ... and the same cut through the fused call: a fresh cache that holds only the prefix, the chunk's K/V handed in
    # and written by the same launch; once contiguous, once as a page pool of a random page size
    kc = torch.zeros(B, Sc, Hkv, D, dtype=torch.bfloat16)
    vc = torch.zeros(B, Sc, Hkv, D, dtype=torch.bfloat16)
    for b in range(B):
        kc[b, :qlen[b]] = k[b, past[b]:lens[b]]
        vc[b, :qlen[b]] = v[b, past[b]:lens[b]]
    want_k, want_v = k.permute(0, 2, 1, 3).contiguous(), v.permute(0, 2, 1, 3).contiguous()       # [B, Hkv, S, D]
    live = torch.arange(S).view(1, 1, S, 1) < torch.from_numpy(lens).view(B, 1, 1, 1)
    prefix = torch.arange(S).view(1, 1, S, 1) < torch.from_numpy(past).view(B, 1, 1, 1)
    nan = nan_bf16((1,))
    ck2 = torch.where(prefix, want_k, nan).contiguous().cuda()
    cv2 = torch.where(prefix, want_v, nan).contiguous().cuda()
    oc2 = torch.zeros(B, Sc, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_prefill_chunk_append(qc.cuda(), kc.cuda(), vc.cuda(), oc2, ck2, cv2, torch.from_numpy(past).cuda(),
                                      torch.from_numpy(qlen).cuda(), scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert torch.equal(torch.where(live, ck2.cpu(), nan).view(torch.int16), torch.where(live, want_k, nan).view(torch.int16))
    assert torch.equal(torch.where(live, cv2.cpu(), nan).view(torch.int16), torch.where(live, want_v, nan).view(torch.int16))
    page = int(rng.choice([16, 32, 64, 128]))
    n_per = (S + page - 1) // page
    perm = torch.from_numpy(rng.permutation(B * n_per + 2)[:B * n_per].astype(np.int32)).view(B, n_per)
    pool_k = nan_bf16((B * n_per + 2, Hkv, page, D)).clone()
    pool_v = nan_bf16((B * n_per + 2, Hkv, page, D)).clone()
    pad_k = torch.cat([torch.where(prefix, want_k, nan), nan_bf16((B, Hkv, n_per * page - S, D))], dim=2)
    pad_v = torch.cat([torch.where(prefix, want_v, nan), nan_bf16((B, Hkv, n_per * page - S, D))], dim=2)
    for b in range(B):
        for i in range(n_per):
            pool_k[perm[b, i]] = pad_k[b, :, i * page:(i + 1) * page]
            pool_v[perm[b, i]] = pad_v[b, :, i * page:(i + 1) * page]
    dpk, dpv = pool_k.cuda(), pool_v.cuda()
    oc3 = torch.zeros(B, Sc, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_prefill_chunk_append(qc.cuda(), kc.cuda(), vc.cuda(), oc3, dpk, dpv, torch.from_numpy(past).cuda(),
                                      torch.from_numpy(qlen).cuda(), scale, ws, block_table=perm.cuda())
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    got_k = torch.from_numpy(orc.gather_pages(dpk.cpu(), perm.numpy(), S).view(np.int16)).view(torch.bfloat16)
    assert torch.equal(torch.where(live, got_k, nan).view(torch.int16), torch.where(live, want_k, nan).view(torch.int16))
    for b in range(B):
        if qlen[b] > 0:
            assert_close_to_oracle(oc2[b, :qlen[b]].cpu(), ref[b, past[b]:lens[b]], f"fused chunk seed {seed} sequence {b}")
            assert_close_to_oracle(oc3[b, :qlen[b]].cpu(), ref[b, past[b]:lens[b]], f"paged fused chunk seed {seed} sequence {b}")
