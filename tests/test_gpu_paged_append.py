"""l4l_attn_decode_paged_append: the decode step over a paged cache that also writes the step's newest token into its
page. Reference = the oracle's paged append at slot kv_len - 1 followed by its paged decode; the pools must come
back bit for bit as the oracle's."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, assert_close_to_oracle
from test_gpu_paged import build_pool

pytestmark = pytest.mark.gpu


def run_case(B, Hq, Hkv, D, page, lens, seed, drop=()):
    """lens = kv_len per sequence INCLUDING the new token. `drop`: sequences whose page for the new slot is taken out
    of the table (nothing may be written for them)."""
    pool_k, pool_v, table = build_pool(B, Hkv, D, page, lens, seed=seed)
    for b in drop:
        table[b, (lens[b] - 1) // page] = -1
    g = torch.Generator().manual_seed(seed + 1)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    k_new = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
    v_new = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    kv = np.array(lens, np.int32)
    pos = np.maximum(kv - 1, 0)
    ref_k, ref_v = orc.kv_append_paged(pool_k, pool_v, table, k_new, v_new, pos, (kv > 0).astype(np.int32))
    ref, ref_lse = orc.decode_paged(q, ref_k, ref_v, table, kv, scale)
    gk, gv = Guarded(pool_k), Guarded(pool_v)
    go = Guarded(torch.zeros(B, Hq, D, dtype=torch.bfloat16))
    lse = torch.zeros(B, Hq, device="cuda")
    max_len = max(max(lens), 1)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, max_len)
    l4l.l4l_attn_decode_paged_append(q.cuda(), go.t, gk.t, gv.t, torch.from_numpy(table).cuda(), k_new.cuda(),
                                     v_new.cuda(), torch.from_numpy(kv).cuda(), max_len, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert gk.margins_intact() and gv.margins_intact() and go.margins_intact()
    assert np.array_equal(orc.bits(gk.t.cpu()), ref_k) and np.array_equal(orc.bits(gv.t.cpu()), ref_v)
    assert_close_to_oracle(go.t.cpu(), ref, f"paged decode + append, page {page}")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 2e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


@pytest.fixture
def kernel_choice(request):
    with l4l.decode_override(cluster=-1 if request.param is None else int(request.param)):
        yield request.param


# None: the library's own choice; 0: split kernel; 1..8: cluster kernel of that width
@pytest.mark.parametrize("kernel_choice", [None, 0, 1, 2, 8], indirect=True)
@pytest.mark.parametrize("page", [16, 64, 256])
@pytest.mark.parametrize("Hq,Hkv,D", [(32, 8, 128), (12, 12, 64)])
def test_paged_decode_append_matches_oracle(kernel_choice, page, Hq, Hkv, D):
    # new token at the start of a page, at its end, in the middle, first token of a sequence, empty sequence
    lens = [1, 16, 17, 128, 129, 257, 700, 1024, 1025, 2049, 333, 0]
    run_case(len(lens), Hq, Hkv, D, page, lens, seed=1200 + page + D)


@pytest.mark.parametrize("kernel_choice", [0, 4], indirect=True)
@pytest.mark.parametrize("page", [16, 128])
def test_paged_decode_append_without_a_page_writes_nothing(kernel_choice, page):
    lens = [513, 40, 2048, 129, 1, 300]
    run_case(len(lens), 32, 8, 128, page, lens, seed=77 + page, drop=(1, 2, 4))


@pytest.mark.parametrize("kernel_choice", [0], indirect=True)
@pytest.mark.parametrize("Hq,Hkv,page", [(64, 8, 64), (128, 8, 32), (128, 8, 128), (40, 8, 16)])
def test_paged_decode_append_large_groups(kernel_choice, Hq, Hkv, page):
    lens = [3000, 1, 96, 97, 1500, 192, 193, 64, 2047]
    run_case(len(lens), Hq, Hkv, 128, page, lens, seed=500 + Hq + page)


@pytest.mark.parametrize("kernel_choice", [None], indirect=True)
def test_paged_decode_append_many_sequences(kernel_choice):
    g = np.random.default_rng(9)
    lens = g.integers(1, 1500, size=150).tolist()
    run_case(len(lens), 32, 8, 128, 16, lens, seed=4242)


def test_paged_decode_append_rejects_bad_arguments():
    q = torch.zeros(2, 4, 64, dtype=torch.bfloat16, device="cuda")
    table = torch.zeros(2, 2, dtype=torch.int32, device="cuda")
    lens = torch.ones(2, dtype=torch.int32, device="cuda")
    pool = torch.zeros(3, 2, 16, 64, dtype=torch.bfloat16, device="cuda")
    kn = torch.zeros(2, 1, 2, 64, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 2, 4, 2, 64, 32)
    with pytest.raises(l4l.L4LError):             # longer than the table can describe
        l4l.l4l_attn_decode_paged_append(q, q.clone(), pool, pool.clone(), table, kn, kn.clone(), lens, 33, 0.1, ws)
    with pytest.raises(ValueError):               # one new token per sequence
        l4l.l4l_attn_decode_paged_append(q, q.clone(), pool, pool.clone(), table, kn[:, :, :1], kn, lens, 16, 0.1, ws)


# ---- the rope-fused step over a paged cache ----

@pytest.mark.parametrize("kernel_choice", [None, 0, 2], indirect=True)
@pytest.mark.parametrize("page", [16, 128])
@pytest.mark.parametrize("Hq,Hkv,D,norm", [(32, 8, 128, True), (8, 2, 64, False), (64, 8, 128, True)])
def test_paged_decode_rope_append_matches_oracle_chain(kernel_choice, page, Hq, Hkv, D, norm):
    """Oracle chain: rotate (and normalise) q and k_new at position kv_len - 1, write the page slot, decode over the
    pages; three consecutive steps on the same pool."""
    from paper_2608_21836_b200.workloads import make_rope_tables
    from test_gpu_rope_append import assert_bf16_close

    lens = np.array([1, 16, 17, 128, 129, 600, 255, 0], np.int32)      # INCLUDING the new token at the first step
    B, steps = len(lens), 3
    pool_k, pool_v, table = build_pool(B, Hkv, D, page, [int(x) + steps for x in lens], seed=300 + page + Hq)
    pool_k = torch.nan_to_num(pool_k, nan=0.5)                           # slots past the lengths: finite fill
    pool_v = torch.nan_to_num(pool_v, nan=-0.25)
    n_pos = 640
    cos, sin = make_rope_tables(n_pos, D)
    g = torch.Generator().manual_seed(31 + D + page)
    qw = (torch.rand(D, generator=g) + 0.5) if norm else None
    kw = (torch.rand(D, generator=g) + 0.5) if norm else None
    eps = 1e-6 if norm else 0.0
    scale = 1.0 / math.sqrt(D)
    dpk, dpv = pool_k.cuda(), pool_v.cuda()
    opk, opv = orc.bits(pool_k), orc.bits(pool_v)
    dtab = torch.from_numpy(table).cuda()
    max_len = int(lens.max()) + steps
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, max_len)
    dcos, dsin = cos.cuda(), sin.cuda()
    for s in range(steps):
        q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
        kn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
        vn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
        cur = np.where(lens > 0, lens + s, 0).astype(np.int32)
        pos = np.maximum(cur - 1, 0)
        # the oracle's rotation through a one-slot-per-position scratch cache, read back at the written slot
        sk = np.zeros((B, Hkv, n_pos, D), np.uint16)
        oq, sk, _, _, _ = orc.rope_kv_append(q.view(B, 1, Hq, D), kn, vn, sk, sk.copy(), pos, None, cos.numpy(), sin.numpy(),
                                             None if qw is None else qw.numpy(), None if kw is None else kw.numpy(), eps)
        k_rot = np.stack([sk[b, :, pos[b]] for b in range(B)])[:, None]           # [B, 1, Hkv, D] bits
        opk, opv = orc.kv_append_paged(opk, opv, table, k_rot, vn, pos, (cur > 0).astype(np.int32))
        ref, _ = orc.decode_paged(oq[:, 0], opk, opv, table, cur, scale)
        o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
        l4l.l4l_attn_decode_paged_rope_append(q.cuda(), o, dpk, dpv, dtab, kn.cuda(), vn.cuda(), torch.from_numpy(cur).cuda(),
                                              max_len, scale, dcos, dsin, ws, q_weight=None if qw is None else qw.cuda(),
                                              k_weight=None if kw is None else kw.cuda(), eps=eps)
        torch.cuda.synchronize()
        assert l4l.l4l_last_device_error(ws) == 0
        assert_close_to_oracle(o.cpu(), ref, f"paged rope + append + decode, step {s}")
    assert_bf16_close(dpk, opk, "pool k after the fused steps")
    assert np.array_equal(orc.bits(dpv.cpu()), opv)


# ---- batches larger than one launch slice (384 sequences on the split kernel, 1024 on the warp-per-unit kernel) ----

@pytest.mark.parametrize("kernel_choice", [None], indirect=True)
def test_paged_decode_append_batch_of_several_launch_slices_split_kernel(kernel_choice):
    g = np.random.default_rng(21)
    lens = g.integers(0, 700, size=450).tolist()             # longer than the warp-per-unit kernel's regime
    assert l4l.l4l_decode_kernel_choice(len(lens), 8, 2, 128, max(lens))[0] == "split"
    run_case(len(lens), 8, 2, 128, 64, lens, seed=515)


@pytest.mark.parametrize("kernel_choice", [None], indirect=True)
def test_paged_decode_append_batch_of_several_launch_slices_warp_kernel(kernel_choice):
    g = np.random.default_rng(22)
    lens = g.integers(0, 120, size=1100).tolist()
    assert l4l.l4l_decode_kernel_choice(len(lens), 8, 2, 128, max(lens))[0] == "warp"
    run_case(len(lens), 8, 2, 128, 16, lens, seed=516)
