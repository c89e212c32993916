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


@pytest.mark.parametrize("seed", range(10))
def test_decode_step_family_random(seed):
    """The fused decode steps on seeded random shapes: cache update fused in (contiguous and paged), the same with rope +
    norm of the new token, and both over an fp8 cache, each against the oracle chain (rope ->) append -> decode."""
    from paper_2608_21836_b200.workloads import make_rope_tables
    from test_gpu_decode_append import make_case
    from test_gpu_fp8 import random_codes
    from helpers import bits_equal

    rng = np.random.default_rng(6000 + seed)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 8]))
    G = int(rng.choice([1, 2, 4, 5, 8]))
    Hq = Hkv * G
    B = int(rng.choice([1, 3, 9, 40]))
    page = int(rng.choice([16, 32, 64, 128]))
    Lmax = int(rng.choice([128, 640, 2176]))                       # multiples of every page size
    lens = np.maximum(random_lengths(rng, B, Lmax), rng.integers(0, 2, B)).astype(np.int32)   # kv_len INCLUDING the new token
    q, ck, cv, kn, vn, kv_len = make_case(B, Hq, Hkv, D, Lmax, lens.tolist(), seed=seed)
    scale = 1.0 / math.sqrt(D)
    pos, n_new = np.maximum(lens - 1, 0), (lens > 0).astype(np.int32)
    dl = torch.from_numpy(lens).cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    as_t = lambda bits: torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    n_per = Lmax // page
    perm = torch.from_numpy(rng.permutation(B * n_per + 3)[: B * n_per].astype(np.int32)).view(B, n_per)

    def to_pool(c, fill):
        pool = fill((B * n_per + 3, Hkv, page, D))
        pool[perm.reshape(-1).long()] = c.view(B, Hkv, n_per, page, D).permute(0, 2, 1, 3, 4).reshape(-1, Hkv, page, D)
        return pool.cuda()

    def from_pool(pool):
        return pool.cpu()[perm.reshape(-1).long()].view(B, n_per, Hkv, page, D).permute(0, 2, 1, 3, 4).reshape(B, Hkv, Lmax, D)

    def done(o, ref, what):
        torch.cuda.synchronize()
        assert l4l.l4l_last_device_error(ws) == 0
        assert_close_to_oracle(o.cpu(), ref, f"{what}, seed {seed}")

    # ---- bf16 cache: fused append, contiguous and paged
    ek, ev = orc.kv_append(ck, cv, kn, vn, pos, n_new)
    ref, _ = orc.decode(q, as_t(ek), as_t(ev), lens, scale)
    dck, dcv, o = ck.cuda(), cv.cuda(), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_append(q.cuda(), o, dck, dcv, kn.cuda(), vn.cuda(), dl, Lmax, scale, ws)
    done(o, ref, "fused append")
    assert bits_equal(dck, ek) and bits_equal(dcv, ev)
    pk, pv, o = to_pool(ck, nan_bf16), to_pool(cv, nan_bf16), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_paged_append(q.cuda(), o, pk, pv, perm.cuda(), kn.cuda(), vn.cuda(), dl, Lmax, scale, ws)
    done(o, ref, f"paged fused append, page {page}")
    assert bits_equal(from_pool(pk), ek) and bits_equal(from_pool(pv), ev)

    # ---- the same with rope + norm of the new token (table over every position)
    cos, sin = make_rope_tables(Lmax, D)
    g = torch.Generator().manual_seed(seed + 77)
    norm = bool(rng.integers(0, 2))
    qw = (torch.rand(D, generator=g) + 0.5) if norm else None
    kw = (torch.rand(D, generator=g) + 0.5) if norm else None
    eps = 1e-6 if norm else 0.0
    oq, rk, rv, _, _ = orc.rope_kv_append(q.view(B, 1, Hq, D), kn, vn, ck, cv, pos, n_new, cos.numpy(), sin.numpy(),
                                          None if qw is None else qw.numpy(), None if kw is None else kw.numpy(), eps)
    ref_r, _ = orc.decode(as_t(oq[:, 0]), as_t(rk), as_t(rv), lens, scale)
    wargs = dict(q_weight=None if qw is None else qw.cuda(), k_weight=None if kw is None else kw.cuda(), eps=eps)
    dck, dcv, o = ck.cuda(), cv.cuda(), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_rope_append(q.cuda(), o, dck, dcv, kn.cuda(), vn.cuda(), dl, Lmax, scale, cos.cuda(), sin.cuda(), ws, **wargs)
    done(o, ref_r, "rope step")
    assert bits_equal(dcv, rv)
    pk, pv, o = to_pool(ck, nan_bf16), to_pool(cv, nan_bf16), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_paged_rope_append(q.cuda(), o, pk, pv, perm.cuda(), kn.cuda(), vn.cuda(), dl, Lmax, scale, cos.cuda(),
                                          sin.cuda(), ws, **wargs)
    done(o, ref_r, f"paged rope step, page {page}")
    assert bits_equal(from_pool(pv), rv)

    # ---- fp8 cache (head_dim 64: on the split kernel, which wants an even number of slots): fused append and rope step
    if D == 64:
        return
    tg = torch.Generator().manual_seed(seed + 99)
    c8k, c8v = random_codes((B, Hkv, Lmax, D), tg, 7), random_codes((B, Hkv, Lmax, D), tg, 7)
    for b in range(B):
        c8k[b, :, max(int(lens[b]) - 1, 0):] = 0x7F
        c8v[b, :, max(int(lens[b]) - 1, 0):] = 0xFF
    ks = torch.from_numpy(rng.uniform(0.5, 1.5, Hkv).astype(np.float32))
    vs = torch.from_numpy(rng.uniform(0.25, 1.25, Hkv).astype(np.float32))
    kn7, vn7 = (kn.float() * 0.7).to(torch.bfloat16), (vn.float() * 0.7).to(torch.bfloat16)
    e8k, e8v = orc.kv_append_fp8(c8k, c8v, kn7, vn7, pos, n_new, ks.numpy(), vs.numpy())
    ref8, _ = orc.decode_fp8(q, e8k, e8v, lens, ks.numpy(), vs.numpy(), scale)
    u8 = lambda shape: torch.full(shape, 0x7F, dtype=torch.uint8)
    d8k, d8v, o = c8k.cuda(), c8v.cuda(), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_append_fp8(q.cuda(), o, d8k, d8v, ks.cuda(), vs.cuda(), kn7.cuda(), vn7.cuda(), dl, Lmax, scale, ws)
    done(o, ref8, "fp8 fused append")
    assert np.array_equal(d8k.cpu().numpy(), e8k) and np.array_equal(d8v.cpu().numpy(), e8v)
    p8k, p8v, o = to_pool(c8k, u8), to_pool(c8v, u8), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_append_fp8(q.cuda(), o, p8k, p8v, ks.cuda(), vs.cuda(), kn7.cuda(), vn7.cuda(), dl, Lmax, scale, ws,
                                   block_table=perm.cuda())
    done(o, ref8, f"fp8 paged fused append, page {page}")
    assert np.array_equal(from_pool(p8k).numpy(), e8k) and np.array_equal(from_pool(p8v).numpy(), e8v)
    # rope step over the fp8 cache: the rotated k row of the oracle (bf16), quantised by the oracle
    scratch = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16)
    oq7, sk, _, _, _ = orc.rope_kv_append(q.view(B, 1, Hq, D), kn7, vn7, scratch, scratch, pos, n_new, cos.numpy(), sin.numpy(),
                                          None if qw is None else qw.numpy(), None if kw is None else kw.numpy(), eps)
    k_rot = as_t(np.stack([sk[b, :, pos[b], :] for b in range(B)])[:, None])
    r8k, r8v = orc.kv_append_fp8(c8k, c8v, k_rot, vn7, pos, n_new, ks.numpy(), vs.numpy())
    ref8r, _ = orc.decode_fp8(as_t(oq7[:, 0]), r8k, r8v, lens, ks.numpy(), vs.numpy(), scale)
    d8k, d8v, o = c8k.cuda(), c8v.cuda(), torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_attn_decode_rope_append_fp8(q.cuda(), o, d8k, d8v, ks.cuda(), vs.cuda(), kn7.cuda(), vn7.cuda(), dl, Lmax, scale,
                                        cos.cuda(), sin.cuda(), ws, **wargs)
    done(o, ref8r, "fp8 rope step")
    assert np.array_equal(d8v.cpu().numpy(), r8v)
