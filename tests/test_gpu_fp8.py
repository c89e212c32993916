"""fp8 (e4m3) KV cache: l4l_kv_append_fp8 (bit-exact codes) and l4l_attn_decode_fp8 against the oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, assert_close_to_oracle

pytestmark = pytest.mark.gpu


def random_codes(shape, g, max_exp_field=11):
    """Random e4m3 codes without NaN, magnitudes below 2^(max_exp_field - 6)."""
    c = torch.randint(0, 256, shape, generator=g, dtype=torch.uint8)
    e = (c >> 3) & 15
    c = torch.where(e > max_exp_field, c & 0x87 | (max_exp_field << 3), c)
    return c


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (8, 8), (16, 2), (12, 12)])
def test_fp8_decode_matches_oracle(Hq, Hkv, D):
    Lmax = 2304
    lens = [1, 15, 16, 17, 127, 128, 129, 700, 1024, 2049, 2304, 0, 333]
    B = len(lens)
    g = torch.Generator().manual_seed(1000 + Hq + D)
    ck8 = random_codes((B, Hkv, Lmax, D), g, 7)              # |k| < 2
    cv8 = random_codes((B, Hkv, Lmax, D), g, 7)              # |v| < 2: the absolute tolerance presumes O(1) outputs
    for b, L in enumerate(lens):                             # slots past the end hold the NaN code
        ck8[b, :, L:] = 0x7F
        cv8[b, :, L:] = 0xFF
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ks = (torch.rand(Hkv, generator=g) + 0.5)
    vs = (torch.rand(Hkv, generator=g) + 0.25)
    scale = 1.0 / math.sqrt(D)
    ref, ref_lse = orc.decode_fp8(q, ck8, cv8, np.array(lens, np.int32), ks.numpy(), vs.numpy(), scale)
    gk, gv = Guarded(ck8), Guarded(cv8)
    go = Guarded(torch.zeros(B, Hq, D, dtype=torch.bfloat16))
    lse = torch.zeros(B, Hq, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_fp8(q.cuda(), go.t, gk.t, gv.t, ks.cuda(), vs.cuda(), torch.tensor(lens, dtype=torch.int32).cuda(),
                            Lmax, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert gk.margins_intact() and gv.margins_intact() and go.margins_intact()
    assert torch.equal(gk.t.cpu(), ck8) and torch.equal(gv.t.cpu(), cv8)
    assert_close_to_oracle(go.t.cpu(), ref, "fp8 decode")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


def test_fp8_decode_on_the_benchmark_batch_and_against_the_bf16_path():
    """The ragged B=32 batch quantised with the library's own append: the fp8 kernel must match the oracle on the
    codes, and (a sanity check of the whole idea) stay near the bf16 kernel on the unquantised cache."""
    from paper_2608_21836_b200 import workloads as wl

    w = wl.WORKLOADS["batched_decode"]
    db = wl.make_decode_batch(w)
    B, Hq, Hkv, D, Lmax = w.decode_B, w.Hq, w.Hkv, w.D, w.decode_Lmax
    ck = torch.nan_to_num(db.cache_k.float(), nan=0.0).to(torch.bfloat16).cuda()     # the NaN tails would not quantise
    cv = torch.nan_to_num(db.cache_v.float(), nan=0.0).to(torch.bfloat16).cuda()
    ks = torch.full((Hkv,), 4.5 / 448, device="cuda")                                # N(0,1) data: 4.5 sigma full scale
    vs = torch.full((Hkv,), 4.5 / 448, device="cuda")
    ck8 = torch.zeros(B, Hkv, Lmax, D, dtype=torch.uint8, device="cuda")
    cv8 = torch.zeros_like(ck8)
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    l4l.l4l_kv_append_fp8(ck8, cv8, ck.permute(0, 2, 1, 3), cv.permute(0, 2, 1, 3), zero, ks, vs)
    q, lens = db.q.cuda(), db.kv_len.cuda()
    o8, o16 = torch.zeros_like(q), torch.zeros_like(q)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_fp8(q, o8, ck8, cv8, ks, vs, lens, Lmax, w.scale, ws)
    l4l.l4l_attn_decode(q, o16, ck, cv, lens, Lmax, w.scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    ref, _ = orc.decode_fp8(db.q, ck8.cpu(), cv8.cpu(), db.kv_len.numpy(), ks.cpu().numpy(), vs.cpu().numpy(), w.scale)
    assert_close_to_oracle(o8.cpu(), ref, "fp8 decode, benchmark batch")
    assert (o8.float() - o16.float()).abs().max().item() < 0.05                       # quantisation noise only


@pytest.mark.parametrize("D", [64, 128])
def test_fp8_append_is_bit_exact(D):
    B, T, Hkv, Lmax = 3, 19, 4, 40
    g = torch.Generator().manual_seed(D)
    k = (torch.randn(B, T, Hkv, D, generator=g) * 3).to(torch.bfloat16)
    v = (torch.randn(B, T, Hkv, D, generator=g) * torch.exp(torch.randn(B, T, Hkv, D, generator=g) * 4)).to(torch.bfloat16)
    v[0, 0, 0, :4] = torch.tensor([float("inf"), -float("inf"), 1e30, -448.0]).to(torch.bfloat16)
    ck8 = torch.full((B, Hkv, Lmax, D), 0x55, dtype=torch.uint8)
    cv8 = ck8.clone()
    ks, vs = torch.rand(Hkv, generator=g) + 0.1, torch.rand(Hkv, generator=g) * 3 + 0.1
    pos, n_new = [0, 30, 21], [19, 19, 7]                    # sequence 1 runs off the end of the cache
    ref_k, ref_v = orc.kv_append_fp8(ck8, cv8, k, v, pos, n_new, ks.numpy(), vs.numpy())
    gk, gv = Guarded(ck8), Guarded(cv8)
    l4l.l4l_kv_append_fp8(gk.t, gv.t, k.cuda(), v.cuda(), torch.tensor(pos, dtype=torch.int32).cuda(), ks.cuda(),
                          vs.cuda(), n_new=torch.tensor(n_new, dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    assert gk.margins_intact() and gv.margins_intact()
    assert np.array_equal(gk.t.cpu().numpy(), ref_k) and np.array_equal(gv.t.cpu().numpy(), ref_v)


def test_fp8_decode_at_head_dim_64_wants_dense_token_rows_in_pairs():
    """At head_dim 64 two tokens share a 128-byte tile row: the cache's token rows must lie back to back (stride 64)
    and the slot count must be even; anything else is refused on the host."""
    q = torch.zeros(1, 4, 64, dtype=torch.bfloat16, device="cuda")
    sc = torch.ones(2, device="cuda")
    one = torch.ones(1, dtype=torch.int32, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 1, 4, 2, 64, 32)
    odd = torch.zeros(1, 2, 33, 64, dtype=torch.uint8, device="cuda")                       # odd number of slots
    with pytest.raises(l4l.L4LError) as e:
        l4l.l4l_attn_decode_fp8(q, q.clone(), odd, odd.clone(), sc, sc, one, 32, 0.1, ws)
    assert e.value.status == l4l.L4L_ERR_UNSUPPORTED
    wide = torch.zeros(1, 2, 32, 128, dtype=torch.uint8, device="cuda")[..., :64]           # token rows 128 bytes apart
    with pytest.raises(l4l.L4LError) as e:
        l4l.l4l_attn_decode_fp8(q, q.clone(), wide, torch.zeros(1, 2, 32, 128, dtype=torch.uint8, device="cuda")[..., :64],
                                sc, sc, one, 32, 0.1, ws)
    assert e.value.status == l4l.L4L_ERR_UNSUPPORTED
    ok = torch.zeros(1, 2, 32, 64, dtype=torch.uint8, device="cuda")
    l4l.l4l_attn_decode_fp8(q, q.clone(), ok, ok.clone(), sc, sc, one, 32, 0.1, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0


def test_fp8_decode_small_mha_shape_at_full_size():
    """The small MHA model's decode batch (Hq = Hkv = 12, head_dim 64, B = 64 at context 1024) over an fp8 cache written
    by the library's own append."""
    from paper_2608_21836_b200 import workloads as wl

    w = wl.WORKLOADS["mha_small"]
    db = wl.make_decode_batch(w, poison_tail=False)
    B, Hq, Hkv, D, Lmax = w.decode_B, w.Hq, w.Hkv, w.D, w.decode_Lmax
    sc = torch.full((Hkv,), 4.5 / 448, dtype=torch.float32)
    k8 = torch.zeros(B, Hkv, Lmax, D, dtype=torch.uint8, device="cuda")
    v8 = torch.zeros_like(k8)
    l4l.l4l_kv_append_fp8(k8, v8, db.cache_k.cuda().permute(0, 2, 1, 3), db.cache_v.cuda().permute(0, 2, 1, 3),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), sc.cuda(), sc.cuda())
    torch.cuda.synchronize()
    # the codes against the oracle's quantisation on a slice (the oracle's encoder is slow): two sequences, 96 slots
    nb, nt = 2, 96
    ref_k, ref_v = orc.kv_append_fp8(np.zeros((nb, Hkv, nt, D), np.uint8), np.zeros((nb, Hkv, nt, D), np.uint8),
                                     db.cache_k[:nb, :, :nt].permute(0, 2, 1, 3).contiguous(),
                                     db.cache_v[:nb, :, :nt].permute(0, 2, 1, 3).contiguous(),
                                     np.zeros(nb, np.int32), None, sc.numpy(), sc.numpy())
    assert np.array_equal(k8[:nb, :, :nt].cpu().numpy(), ref_k) and np.array_equal(v8[:nb, :, :nt].cpu().numpy(), ref_v)
    ref_k, ref_v = k8.cpu().numpy(), v8.cpu().numpy()
    ref, _ = orc.decode_fp8(db.q, ref_k, ref_v, db.kv_len.numpy(), sc.numpy(), sc.numpy(), w.scale)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    assert l4l.l4l_decode_kernel_choice(B, Hq, Hkv, D, Lmax, fp8=True)[0] == "split"
    l4l.l4l_attn_decode_fp8(db.q.cuda(), o, k8, v8, sc.cuda(), sc.cuda(), db.kv_len.cuda(), Lmax, w.scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, "fp8 decode, small MHA shape")


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("page", [16, 64, 256])
def test_fp8_paged_decode_matches_oracle(page, D):
    """An fp8 page pool behind a block table: the oracle gathers the pages (codes are bytes: the gather is the same
    indexing as for bf16) and decodes over the codes."""
    Hq, Hkv = 16, 4
    lens = [1, 17, 255, 256, 257, 1500, 0, 640]
    B = len(lens)
    g = torch.Generator().manual_seed(2000 + page + D)
    need = [(L + page - 1) // page for L in lens]
    n_pages = sum(need) + 4
    table = np.full((B, max(need) + 1), -1, np.int32)
    perm = iter(torch.randperm(n_pages, generator=g).tolist())
    pool_k = torch.full((n_pages, Hkv, page, D), 0x7F, dtype=torch.uint8)
    pool_v = torch.full((n_pages, Hkv, page, D), 0xFF, dtype=torch.uint8)
    for b in range(B):
        for i in range(need[b]):
            pg = next(perm)
            table[b, i] = pg
            n = min(page, lens[b] - i * page)
            pool_k[pg, :, :n] = random_codes((Hkv, n, D), g, 7)
            pool_v[pg, :, :n] = random_codes((Hkv, n, D), g, 7)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ks, vs = torch.rand(Hkv, generator=g) + 0.5, torch.rand(Hkv, generator=g) + 0.25
    Lmax = max(lens)
    # gather the code pages into contiguous code caches (reusing the bf16 gather on 16-bit views is not possible for
    # bytes, so index directly: slot s of sequence b = row s % page of page table[b, s // page])
    ck8 = torch.zeros(B, Hkv, Lmax, D, dtype=torch.uint8)
    cv8 = torch.zeros(B, Hkv, Lmax, D, dtype=torch.uint8)
    for b in range(B):
        for s0 in range(0, lens[b], page):
            n = min(page, lens[b] - s0)
            ck8[b, :, s0:s0 + n] = pool_k[table[b, s0 // page], :, :n]
            cv8[b, :, s0:s0 + n] = pool_v[table[b, s0 // page], :, :n]
    ref, _ = orc.decode_fp8(q, ck8, cv8, np.array(lens, np.int32), ks.numpy(), vs.numpy(), 0.09)
    o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_paged_fp8(q.cuda(), o, pool_k.cuda(), pool_v.cuda(), ks.cuda(), vs.cuda(),
                                  torch.from_numpy(table).cuda(), torch.tensor(lens, dtype=torch.int32).cuda(), Lmax,
                                  0.09, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert_close_to_oracle(o.cpu(), ref, f"fp8 paged decode, page {page}")


# ---- the decode step that appends the newest token to the fp8 cache itself ----

def _fp8_append_case(Hq, Hkv, lens, seed, page=None, Lmax=2304, D=128):
    """Reference = the oracle's fp8 append at slot kv_len - 1 followed by its fp8 decode; the codes in the cache must
    come back bit for bit. With `page`, the cache is a page pool behind a shuffled block table."""
    B = len(lens)
    g = torch.Generator().manual_seed(seed)
    ck8 = random_codes((B, Hkv, Lmax, D), g, 7)
    cv8 = random_codes((B, Hkv, Lmax, D), g, 7)
    for b, L in enumerate(lens):                             # the new token's slot and everything after it: NaN codes
        ck8[b, :, max(L - 1, 0):] = 0x7F
        cv8[b, :, max(L - 1, 0):] = 0xFF
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    kn = (torch.randn(B, 1, Hkv, D, generator=g) * 0.7).to(torch.bfloat16)
    vn = (torch.randn(B, 1, Hkv, D, generator=g) * 0.7).to(torch.bfloat16)
    ks, vs = torch.rand(Hkv, generator=g) + 0.5, torch.rand(Hkv, generator=g) + 0.25
    scale = 1.0 / math.sqrt(D)
    kv = np.array(lens, np.int32)
    pos, n_new = np.maximum(kv - 1, 0), (kv > 0).astype(np.int32)
    ref_k, ref_v = orc.kv_append_fp8(ck8, cv8, kn, vn, pos, n_new, ks.numpy(), vs.numpy())
    ref, ref_lse = orc.decode_fp8(q, ref_k, ref_v, kv, ks.numpy(), vs.numpy(), scale)
    go = Guarded(torch.zeros(B, Hq, D, dtype=torch.bfloat16))
    lse = torch.zeros(B, Hq, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    if page is None:
        gk, gv = Guarded(ck8), Guarded(cv8)
        l4l.l4l_attn_decode_append_fp8(q.cuda(), go.t, gk.t, gv.t, ks.cuda(), vs.cuda(), kn.cuda(), vn.cuda(),
                                       torch.from_numpy(kv).cuda(), Lmax, scale, ws, lse=lse)
        torch.cuda.synchronize()
        got_k, got_v = gk.t.cpu().numpy(), gv.t.cpu().numpy()
        assert gk.margins_intact() and gv.margins_intact()
    else:
        per = Lmax // page
        n_pages = B * per + 3
        perm = torch.randperm(n_pages, generator=g)[:B * per].view(B, per)
        pool_k = torch.full((n_pages, Hkv, page, D), 0x7F, dtype=torch.uint8)
        pool_v = torch.full((n_pages, Hkv, page, D), 0xFF, dtype=torch.uint8)
        for b in range(B):
            for i in range(per):
                pool_k[perm[b, i]] = ck8[b, :, i * page:(i + 1) * page]
                pool_v[perm[b, i]] = cv8[b, :, i * page:(i + 1) * page]
        gk, gv = Guarded(pool_k), Guarded(pool_v)
        l4l.l4l_attn_decode_append_fp8(q.cuda(), go.t, gk.t, gv.t, ks.cuda(), vs.cuda(), kn.cuda(), vn.cuda(),
                                       torch.from_numpy(kv).cuda(), Lmax, scale, ws, lse=lse,
                                       block_table=perm.to(torch.int32).cuda())
        torch.cuda.synchronize()
        assert gk.margins_intact() and gv.margins_intact()
        pk, pv = gk.t.cpu(), gv.t.cpu()
        got_k = torch.stack([torch.cat([pk[perm[b, i]] for i in range(per)], dim=1) for b in range(B)]).numpy()
        got_v = torch.stack([torch.cat([pv[perm[b, i]] for i in range(per)], dim=1) for b in range(B)]).numpy()
    assert l4l.l4l_last_device_error(ws) == 0
    assert go.margins_intact()
    assert np.array_equal(got_k, ref_k) and np.array_equal(got_v, ref_v)
    assert_close_to_oracle(go.t.cpu(), ref, "fp8 decode + append")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (8, 8), (16, 2), (64, 8)])
def test_fp8_decode_with_fused_append(Hq, Hkv):
    # the new token at the start, in the middle and at the end of 32-token steps and 256-token tiles; an empty sequence
    lens = [1, 2, 16, 17, 32, 33, 255, 256, 257, 700, 1024, 2049, 2304, 0, 333]
    _fp8_append_case(Hq, Hkv, lens, seed=3000 + Hq)


@pytest.mark.parametrize("page", [16, 64, 256])
def test_fp8_paged_decode_with_fused_append(page):
    lens = [1, 17, 255, 256, 257, 1500, 0, 640, 2304]
    _fp8_append_case(16, 4, lens, seed=3100 + page, page=page)


@pytest.mark.parametrize("width", [1, 2, 8])
def test_fp8_fused_append_on_the_cluster_kernel(width):
    with l4l.decode_override(cluster=width):
        _fp8_append_case(8, 2, [1, 32, 33, 256, 257, 1000, 0, 2304], seed=3200 + width)
        _fp8_append_case(8, 2, [1, 33, 257, 1000, 0, 2304], seed=3300 + width, page=64)


def test_fp8_fused_append_batch_of_several_launch_slices():
    g = np.random.default_rng(23)
    lens = g.integers(0, 300, size=420).tolist()             # more than the 384 sequences of one launch
    _fp8_append_case(8, 2, lens, seed=3400, Lmax=320)
    _fp8_append_case(8, 2, lens, seed=3401, page=32, Lmax=320)


@pytest.mark.parametrize("page", [None, 16, 128])
def test_fp8_fused_append_at_head_dim_64(page, decode_kernel_choice):
    lens = [1, 2, 31, 32, 33, 255, 256, 257, 1000, 0, 2303, 2304]
    _fp8_append_case(12, 12, lens, seed=3500 + (page or 0), page=page, D=64)
    _fp8_append_case(8, 2, lens, seed=3600 + (page or 0), page=page, D=64)
