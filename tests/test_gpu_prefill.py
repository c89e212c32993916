"""Parity of l4l_attn_prefill (CUDA, through the C ABI) with the fp64 oracle; cache writes bit-exact."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from paper_2608_21836_b200 import workloads as wl
from helpers import Guarded, assert_close_to_oracle, bits_equal, nan_bf16

pytestmark = pytest.mark.gpu

SENTINEL = 0x4D4D   # bf16 bit pattern pre-filled into outputs; rows that must stay untouched keep it


def sentinel_bf16(shape):
    return torch.full(shape, SENTINEL, dtype=torch.int16).view(torch.bfloat16)


def poison_padding(x, lens):
    """NaN in every token row >= len[b] of a [B, S, H, D] tensor."""
    B, S = x.shape[:2]
    dead = torch.arange(S).view(1, S, 1, 1) >= torch.as_tensor(lens).view(B, 1, 1, 1)
    return torch.where(dead, nan_bf16((1,)), x).contiguous()


def run_prefill(q, k, v, lens, scale, with_cache=True, Lmax=None, want_lse=True, token_major_cache=False):
    B, S, Hq, D = q.shape
    Hkv = k.shape[2]
    Lmax = S if Lmax is None else Lmax
    gq, gk, gv = Guarded(q), Guarded(k), Guarded(v)
    go = Guarded(sentinel_bf16((B, S, Hq, D)))
    glse = Guarded(torch.full((B, Hq, S), -12345.0))
    dk = dv = gck = gcv = None
    if with_cache:
        if token_major_cache:
            gck, gcv = Guarded(sentinel_bf16((B, Lmax, Hkv, D))), Guarded(sentinel_bf16((B, Lmax, Hkv, D)))
            dk, dv = gck.t.permute(0, 2, 1, 3), gcv.t.permute(0, 2, 1, 3)
        else:
            gck, gcv = Guarded(sentinel_bf16((B, Hkv, Lmax, D))), Guarded(sentinel_bf16((B, Hkv, Lmax, D)))
            dk, dv = gck.t, gcv.t
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    lens_dev = torch.as_tensor(lens, dtype=torch.int32).cuda()
    l4l.l4l_attn_prefill(gq.t, gk.t, gv.t, go.t, lens_dev, scale, ws, cache_k=dk, cache_v=dv,
                         lse=glse.t if want_lse else None)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for g in (gq, gk, gv, go, glse, gck, gcv):
        assert g is None or g.margins_intact()
    return go.t, glse.t, dk, dv


def check_prefill(q, k, v, lens, scale, **kw):
    lens = np.asarray(lens, dtype=np.int32)
    B, S, Hq, D = q.shape
    Hkv = k.shape[2]
    ref, ref_lse = orc.prefill(q, k, v, lens, scale)
    o, lse, ck, cv = run_prefill(q, k, v, lens, scale, **kw)
    o_cpu, lse_cpu = o.cpu(), lse.cpu()
    valid = torch.arange(S).view(1, S) < torch.as_tensor(lens).view(B, 1)          # [B,S]
    if valid.any():
        assert_close_to_oracle(o_cpu[valid], ref[valid.numpy()], "prefill o")
        vl = valid.view(B, 1, S).expand(B, Hq, S)
        assert np.abs(lse_cpu[vl].double().numpy() - ref_lse[vl.numpy()]).max() <= 2e-3
    # rows past the end of a sequence are never written
    assert (o_cpu[~valid].view(torch.int16) == SENTINEL).all()
    assert (lse_cpu[~valid.view(B, 1, S).expand(B, Hq, S)] == -12345.0).all()
    if ck is not None:
        Lmax = ck.shape[2]
        ek, ev = orc.kv_append(sentinel_bf16((B, Hkv, Lmax, D)), sentinel_bf16((B, Hkv, Lmax, D)), k, v,
                               np.zeros(B, np.int32), lens)
        assert bits_equal(ck.contiguous(), ek) and bits_equal(cv.contiguous(), ev)
    return o


def rand_qkv(B, S, Hq, Hkv, D, seed, value_scale=1.0):
    g = torch.Generator().manual_seed(seed)
    mk = lambda H: (torch.randn(B, S, H, D, generator=g) * value_scale).to(torch.bfloat16)
    return mk(Hq), mk(Hkv), mk(Hkv)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(4, 2), (3, 3), (8, 2), (8, 1), (16, 1)])
def test_prefill_ragged_edge_lengths(D, Hq, Hkv):
    lens = [0, 1, 2, 63, 64, 65, 127, 128, 129, 200, 255, 256, 257, 300]
    S = 300
    q, k, v = rand_qkv(len(lens), S, Hq, Hkv, D, seed=300 + D + Hq)
    q, k, v = poison_padding(q, lens), poison_padding(k, lens), poison_padding(v, lens)
    check_prefill(q, k, v, lens, 1.0 / math.sqrt(D), Lmax=320)


def test_prefill_without_cache_and_without_lse():
    q, k, v = rand_qkv(2, 150, 4, 2, 128, seed=31)
    lens = np.array([150, 97], np.int32)
    ref, _ = orc.prefill(q, k, v, lens, 0.1)
    o, _, _, _ = run_prefill(q, k, v, lens, 0.1, with_cache=False, want_lse=False)
    assert_close_to_oracle(o[0].cpu(), ref[0], "no-cache prefill")
    assert_close_to_oracle(o[1, :97].cpu(), ref[1, :97], "no-cache prefill")


def test_prefill_token_major_cache_and_fused_qkv_views():
    B, S, Hq, Hkv, D = 2, 200, 8, 2, 128
    g = torch.Generator().manual_seed(33)
    qkv = torch.randn(B, S, Hq + 2 * Hkv, D, generator=g).to(torch.bfloat16)
    lens = np.array([200, 131], np.int32)
    q, k, v = qkv[:, :, :Hq].contiguous(), qkv[:, :, Hq:Hq + Hkv].contiguous(), qkv[:, :, Hq + Hkv:].contiguous()
    ref, _ = orc.prefill(q, k, v, lens, 0.09)
    dqkv = qkv.cuda()
    dq, dk, dv = dqkv[:, :, :Hq], dqkv[:, :, Hq:Hq + Hkv], dqkv[:, :, Hq + Hkv:]      # strided views
    o = torch.zeros(B, S, Hq, D, dtype=torch.bfloat16, device="cuda")
    ck = sentinel_bf16((B, 256, Hkv, D)).cuda()
    cv = sentinel_bf16((B, 256, Hkv, D)).cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill(dq, dk, dv, o, torch.as_tensor(lens).cuda(), 0.09, ws,
                         cache_k=ck.permute(0, 2, 1, 3), cache_v=cv.permute(0, 2, 1, 3))
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for b in range(B):
        assert_close_to_oracle(o[b, :lens[b]].cpu(), ref[b, :lens[b]], "fused-qkv prefill")
        assert bits_equal(ck[b, :lens[b]], k[b, :lens[b]]) and bits_equal(cv[b, :lens[b]], v[b, :lens[b]])
        assert (ck[b, lens[b]:].cpu().view(torch.int16) == SENTINEL).all()


def test_prefill_causality_and_determinism_on_gpu():
    B, S, Hq, Hkv, D = 1, 384, 4, 2, 128
    q, k, v = rand_qkv(B, S, Hq, Hkv, D, seed=35)
    lens = [S]
    o1, l1, _, _ = run_prefill(q, k, v, lens, 0.088)
    o1b, l1b, _, _ = run_prefill(q, k, v, lens, 0.088)
    assert bits_equal(o1, o1b) and torch.equal(l1, l1b)
    cut = 201
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    q2[:, cut:], k2[:, cut:], v2[:, cut:] = 3.0, -7.0, 11.0
    o2, _, _, _ = run_prefill(q2, k2, v2, lens, 0.088)
    assert bits_equal(o1[:, :cut], o2[:, :cut])
    assert not bits_equal(o1[:, cut:], o2[:, cut:])


def test_prefill_closed_forms_on_gpu():
    B, S, Hq, Hkv, D = 1, 260, 4, 2, 64
    g = torch.Generator().manual_seed(37)
    q = torch.randn(B, S, Hq, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, S, Hkv, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16).expand(B, S, Hkv, D).contiguous()
    o, _, _, _ = run_prefill(q, k, v, [S], 0.125)
    pm = (v.double().cumsum(dim=1) / torch.arange(1, S + 1).view(1, S, 1, 1)).repeat_interleave(Hq // Hkv, dim=2)
    assert (o.cpu().double() - pm).abs().max() <= 2e-2
    assert bits_equal(o[:, 0], v[:, 0].repeat_interleave(Hq // Hkv, dim=1))        # row 0 is V[0] exactly
    q1 = torch.ones(B, S, Hq, D).to(torch.bfloat16)
    k1 = torch.zeros(B, S, Hkv, D).to(torch.bfloat16)
    k1[:, 70] = 4.0
    o, _, _, _ = run_prefill(q1, k1, v, [S], 1.0)
    assert bits_equal(o[:, 70:], v[:, 70:71].repeat_interleave(Hq // Hkv, dim=2).expand(B, S - 70, Hq, D).contiguous())


def test_config_tiny_prefill():
    w = wl.WORKLOADS["tiny"]
    seq = wl.make_sequence(w)
    S = seq.S
    check_prefill(seq.q[:, :S].contiguous(), seq.k[:, :S].contiguous(), seq.v[:, :S].contiguous(), [S], w.scale,
                  Lmax=S + seq.T)


def test_config_layer8b_prefill_full_size():
    w = wl.WORKLOADS["layer8b"]
    seq = wl.make_sequence(w)
    S = seq.S
    check_prefill(seq.q[:, :S].contiguous(), seq.k[:, :S].contiguous(), seq.v[:, :S].contiguous(), [S], w.scale,
                  Lmax=S + seq.T)


def test_config_mha_small_prefill_full_size():
    w = wl.WORKLOADS["mha_small"]
    seq = wl.make_sequence(w)
    check_prefill(seq.q, seq.k, seq.v, [seq.S] * w.prefill_B, w.scale)


def test_config_long_prefill_full_size_sampled_rows():
    """B=4, S=8192 in the benchmark's launch configuration; the oracle evaluates a stratified sample of rows
    (the first block, every 64th row, the last 256 rows, random ones), the cache is compared in full."""
    w = wl.WORKLOADS["long_prefill"]
    seq = wl.make_sequence(w)
    B, S, Hq, Hkv, D = w.prefill_B, seq.S, w.Hq, w.Hkv, w.D
    dq, dk, dv = seq.q.cuda(), seq.k.cuda(), seq.v.cuda()
    o = sentinel_bf16((B, S, Hq, D)).cuda()
    lse = torch.empty(B, Hq, S, dtype=torch.float32, device="cuda")
    ck, cv = sentinel_bf16((B, Hkv, S, D)).cuda(), sentinel_bf16((B, Hkv, S, D)).cuda()
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    lens = torch.full((B,), S, dtype=torch.int32, device="cuda")
    l4l.l4l_attn_prefill(dq, dk, dv, o, lens, w.scale, ws, cache_k=ck, cache_v=cv, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert bits_equal(ck, seq.k.permute(0, 2, 1, 3).contiguous()) and bits_equal(cv, seq.v.permute(0, 2, 1, 3).contiguous())
    # Stratified sample, about 24 thousand rows (a few seconds of oracle time): rows 0..255 (first block, every
    # sub-tile and diagonal case), every 64th row (a row in each half of every 128-row sub-tile of every block), the
    # last 256 rows (the longest causal spans) and a few random ones; every query head of sequence 0, two random heads
    # of each other sequence.
    rng = np.random.default_rng(4)
    toks = sorted(set(list(range(256)) + list(range(0, S, 64)) + list(range(S - 256, S)) + [4095, 4096, 4097] +
                      rng.integers(0, S, 24).tolist()))
    rows = [(0, i, h) for i in toks for h in range(Hq)]
    for b in range(1, B):
        rows += [(b, i, h) for h in rng.choice(Hq, 2, replace=False).tolist() for i in toks]
    ref, ref_lse = orc.prefill_rows(seq.q, seq.k, seq.v, np.full(B, S, np.int32), w.scale, rows)
    idx = torch.as_tensor(rows)
    got = o.cpu()[idx[:, 0], idx[:, 1], idx[:, 2]]
    assert_close_to_oracle(got, ref, "long_prefill sampled rows")
    got_lse = lse.cpu()[idx[:, 0], idx[:, 2], idx[:, 1]].double().numpy()
    assert np.abs(got_lse - ref_lse).max() <= 2e-3
    # properties that hold at any size: every output finite, row 0 equals V[0] exactly
    assert torch.isfinite(o.float()).all()
    assert bits_equal(o[:, 0], seq.v[:, 0].repeat_interleave(Hq // Hkv, dim=1))
