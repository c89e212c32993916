"""The whole decode step over an e4m3 cache in one launch (l4l_attn_decode_rope_append_fp8): rotary embedding (+ RMS
norm) of q and k_new, quantisation of the rotated k and of v_new into the cache, attention. Reference = the oracle
chain rope -> fp8 append -> fp8 decode."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from paper_2608_21836_b200.workloads import make_rope_tables
from helpers import Guarded, assert_close_to_oracle, bits_equal
from test_gpu_fp8 import random_codes

pytestmark = pytest.mark.gpu


def code_order(c: np.ndarray) -> np.ndarray:
    """e4m3 codes -> integers in the order of their values (neighbouring codes differ by 1)."""
    m = (c & 0x7F).astype(np.int32)
    return np.where(c & 0x80, -m, m)


def _case(Hq, Hkv, lens, seed, D=128, norm=False, page=None, Lmax=1280):
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
    cos, sin = make_rope_tables(Lmax, D)
    qw = (torch.rand(D, generator=g) + 0.5) if norm else None
    kw = (torch.rand(D, generator=g) + 0.5) if norm else None
    eps = 1e-6 if norm else 0.0
    scale = 1.0 / math.sqrt(D)
    kv = np.array(lens, np.int32)
    pos, n_new = np.maximum(kv - 1, 0), (kv > 0).astype(np.int32)

    # oracle: rotate q and k_new at the new token's position (through a scratch bf16 cache), then quantise the rotated
    # row into the fp8 cache, then attend
    scratch = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16)
    oq, ock, _, _, _ = orc.rope_kv_append(q.view(B, 1, Hq, D), kn, vn, scratch, scratch, pos, n_new, cos.numpy(),
                                          sin.numpy(), None if qw is None else qw.numpy(),
                                          None if kw is None else kw.numpy(), eps)
    k_rot = np.stack([ock[b, :, pos[b], :] for b in range(B)])[:, None]                    # [B, 1, Hkv, D] bf16 bits
    k_rot_t = torch.from_numpy(k_rot.view(np.int16).copy()).view(torch.bfloat16)
    ref_k, ref_v = orc.kv_append_fp8(ck8, cv8, k_rot_t, vn, pos, n_new, ks.numpy(), vs.numpy())
    oq_t = torch.from_numpy(oq[:, 0].view(np.int16).copy()).view(torch.bfloat16)
    # sequences without a token keep their q unrotated in the oracle's output; they have no output either way
    ref, ref_lse = orc.decode_fp8(oq_t, ref_k, ref_v, kv, ks.numpy(), vs.numpy(), scale)

    go = Guarded(torch.zeros(B, Hq, D, dtype=torch.bfloat16))
    lse = torch.zeros(B, Hq, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    dq = q.cuda()
    q_before = dq.clone()
    kw_args = dict(q_weight=None if qw is None else qw.cuda(), k_weight=None if kw is None else kw.cuda(), eps=eps, lse=lse)
    if page is None:
        gk, gv = Guarded(ck8), Guarded(cv8)
        l4l.l4l_attn_decode_rope_append_fp8(dq, go.t, gk.t, gv.t, ks.cuda(), vs.cuda(), kn.cuda(), vn.cuda(),
                                            torch.from_numpy(kv).cuda(), Lmax, scale, cos.cuda(), sin.cuda(), ws, **kw_args)
        torch.cuda.synchronize()
        assert gk.margins_intact() and gv.margins_intact()
        got_k, got_v = gk.t.cpu().numpy(), gv.t.cpu().numpy()
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
        l4l.l4l_attn_decode_rope_append_fp8(dq, go.t, gk.t, gv.t, ks.cuda(), vs.cuda(), kn.cuda(), vn.cuda(),
                                            torch.from_numpy(kv).cuda(), Lmax, scale, cos.cuda(), sin.cuda(), ws,
                                            block_table=perm.to(torch.int32).cuda(), **kw_args)
        torch.cuda.synchronize()
        assert gk.margins_intact() and gv.margins_intact()
        pk, pv = gk.t.cpu(), gv.t.cpu()
        got_k = torch.stack([torch.cat([pk[perm[b, i]] for i in range(per)], dim=1) for b in range(B)]).numpy()
        got_v = torch.stack([torch.cat([pv[perm[b, i]] for i in range(per)], dim=1) for b in range(B)]).numpy()
    assert l4l.l4l_last_device_error(ws) == 0
    assert go.margins_intact()
    assert bits_equal(dq, q_before)                                            # q is read only
    assert np.array_equal(got_v, ref_v)                                        # v is not rotated: bit for bit
    # k: the GPU rotates in fp32 and rounds once, the oracle rounds the fp64 value; where those differ by one bf16 ulp
    # the e4m3 code may be the neighbouring one. Everything but the new rows is untouched, bit for bit.
    d = np.abs(code_order(got_k) - code_order(ref_k))
    new_row = np.zeros(got_k.shape, bool)
    for b in range(B):
        if kv[b] > 0:
            new_row[b, :, pos[b], :] = True
    assert (d[~new_row] == 0).all()
    assert d.max() <= 1, f"k codes off by {d.max()}"
    assert (d[new_row] != 0).mean() <= 5e-3, f"{(d[new_row] != 0).mean():.2e} of the new k codes differ"
    assert_close_to_oracle(go.t.cpu(), ref, "rope + fp8 append + decode")
    fin = np.isfinite(ref_lse)
    assert np.abs(lse.cpu().double().numpy()[fin] - ref_lse[fin]).max() <= 3e-3
    assert (lse.cpu().numpy()[~fin] == -np.inf).all()


LENS = [1, 2, 16, 17, 32, 33, 255, 256, 257, 700, 1024, 1280, 0, 333]


@pytest.mark.parametrize("norm", [False, True])
@pytest.mark.parametrize("Hq,Hkv", [(32, 8), (8, 8), (16, 2), (64, 8)])
def test_fp8_rope_step_on_the_split_kernel(Hq, Hkv, norm):
    with l4l.decode_override(cluster=0):
        _case(Hq, Hkv, LENS, seed=5000 + Hq + norm, norm=norm)


@pytest.mark.parametrize("norm", [False, True])
@pytest.mark.parametrize("page", [16, 64, 256])
def test_fp8_rope_step_paged(page, norm):
    with l4l.decode_override(cluster=0):
        _case(16, 4, [1, 17, 255, 256, 257, 1000, 0, 640, 1280], seed=5100 + page + norm, norm=norm, page=page)


@pytest.mark.parametrize("norm", [False, True])
@pytest.mark.parametrize("width", [1, 2, 8])
def test_fp8_rope_step_on_the_cluster_kernel(width, norm):
    with l4l.decode_override(cluster=width):
        _case(8, 2, [1, 32, 33, 256, 257, 1000, 0, 1280], seed=5200 + width + norm, norm=norm)
        _case(8, 2, [1, 33, 257, 1000, 0, 1280], seed=5300 + width + norm, norm=norm, page=64)


@pytest.mark.parametrize("norm", [False, True])
@pytest.mark.parametrize("page", [None, 32])
def test_fp8_rope_step_at_head_dim_64(page, norm):
    _case(12, 12, [1, 2, 31, 32, 33, 255, 256, 257, 1000, 0, 1279, 1280], seed=5400 + (page or 0) + norm, norm=norm, page=page, D=64)


def test_fp8_rope_step_library_choice_and_many_sequences():
    g = np.random.default_rng(29)
    _case(8, 2, g.integers(0, 300, size=420).tolist(), seed=5500, norm=True, Lmax=320)      # several launch slices
    _case(32, 8, [2304 // 2, 1, 900], seed=5501, norm=True)                                  # the library's own choice
