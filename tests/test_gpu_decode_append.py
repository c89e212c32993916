"""l4l_attn_decode_append (cache update fused into decode) against the oracle's append followed by its decode."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from paper_2608_21836_b200 import workloads as wl
from helpers import Guarded, assert_close_to_oracle, bits_equal, nan_bf16

pytestmark = pytest.mark.gpu


def make_case(B, Hq, Hkv, D, Lmax, lens, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    kn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
    vn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
    kv_len = torch.tensor(lens, dtype=torch.int32)
    # everything from the newest token's slot on is poison: the slot itself must come from k_new / v_new
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= (kv_len.view(B, 1, 1, 1) - 1).clamp(min=0)
    nan = nan_bf16((1,))
    return q, torch.where(dead, nan, ck).contiguous(), torch.where(dead, nan, cv).contiguous(), kn, vn, kv_len


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4), (16, 1)])
def test_decode_append_ragged_edge_lengths(D, Hq, Hkv):
    lens = [0, 1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 191, 300, 320, 1000]
    B, Lmax = len(lens), 1024
    q, ck, cv, kn, vn, kv_len = make_case(B, Hq, Hkv, D, Lmax, lens, seed=600 + D + Hq)
    scale = 1.0 / math.sqrt(D)
    pos = (kv_len - 1).clamp(min=0).numpy()
    n_new = (kv_len > 0).to(torch.int32).numpy()
    ek, ev = orc.kv_append(ck, cv, kn, vn, pos, n_new)
    ek_t = torch.from_numpy(ek.view(np.int16)).view(torch.bfloat16)
    ev_t = torch.from_numpy(ev.view(np.int16)).view(torch.bfloat16)
    ref, ref_lse = orc.decode(q, ek_t, ev_t, kv_len.numpy(), scale)

    gk, gv = Guarded(ck), Guarded(cv)
    gq, gkn, gvn = Guarded(q), Guarded(kn), Guarded(vn)
    go = Guarded(nan_bf16((B, Hq, D)))
    lse = torch.full((B, Hq), float("nan"), device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    l4l.l4l_attn_decode_append(gq.t, go.t, gk.t, gv.t, gkn.t, gvn.t, kv_len.cuda(), Lmax, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for g in (gk, gv, gq, gkn, gvn, go):
        assert g.margins_intact()
    # the cache got exactly the new rows, nothing else changed
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)
    assert_close_to_oracle(go.t, ref, "decode_append o")
    got_lse = lse.cpu().double().numpy()
    fin = np.isfinite(ref_lse)
    assert np.array_equal(np.isneginf(got_lse), np.isneginf(ref_lse))
    assert np.abs(got_lse[fin] - ref_lse[fin]).max() <= 2e-3


def test_decode_append_steps_equal_prefill_rows_layer8b():
    """The 8B-shaped layer: 256 fused decode steps after a prompt of 2048 tokens; sampled steps against the
    oracle's causal-prefill rows, the whole cache against the sequence's K/V."""
    w = wl.WORKLOADS["layer8b"]
    seq = wl.make_sequence(w)
    B, S, T, Hq, Hkv, D = w.prefill_B, seq.S, seq.T, w.Hq, w.Hkv, w.D
    Lmax = S + T
    ck = nan_bf16((B, Hkv, Lmax, D)).cuda()
    cv = nan_bf16((B, Hkv, Lmax, D)).cuda()
    k_dev, v_dev, q_dev = seq.k.cuda(), seq.v.cuda(), seq.q.cuda()
    l4l.l4l_kv_append(ck, cv, k_dev[:, :S], v_dev[:, :S], torch.zeros(B, dtype=torch.int32, device="cuda"))
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    outs = torch.empty(B, T, Hq, D, dtype=torch.bfloat16, device="cuda")
    for t in range(T):
        n = torch.full((B,), S + t + 1, dtype=torch.int32, device="cuda")
        l4l.l4l_attn_decode_append(q_dev[:, S + t].contiguous(), outs[:, t], ck, cv, k_dev[:, S + t:S + t + 1],
                                   v_dev[:, S + t:S + t + 1], n, Lmax, w.scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert bits_equal(ck, seq.k.permute(0, 2, 1, 3).contiguous()) and bits_equal(cv, seq.v.permute(0, 2, 1, 3).contiguous())
    steps = [0, 1, 15, 16, 63, 64, 127, 128, 200, 255]
    rows = [(b, S + t, h) for b in range(B) for t in steps for h in range(Hq)]
    ref, _ = orc.prefill_rows(seq.q, seq.k, seq.v, np.full(B, S + T, np.int32), w.scale, rows)
    got = torch.stack([outs[b, t, h] for b in range(B) for t in steps for h in range(Hq)])
    assert_close_to_oracle(got, ref, "layer8b fused decode steps")


@pytest.mark.parametrize("B,Lmax", [(3, 512), (40, 512)])
def test_decode_append_length_beyond_the_host_bound_leaves_the_cache_alone(B, Lmax):
    """A sequence whose device length exceeds the host bound has no slot for its new token inside the bound: the
    fused step must not write it over a valid slot. It is treated as empty (o = 0, lse = -inf, nothing written);
    the other sequences of the batch are unaffected. Small batch: cluster kernel; 40 x 8 units: split kernel."""
    Hq, Hkv, D, bound = 16, 8, 128, 256
    lens = [200] * B
    lens[1] = 300                                            # > bound (but inside the cache)
    q, ck, cv, kn, vn, kv_len = make_case(B, Hq, Hkv, D, Lmax, lens, seed=640 + B)
    ck, cv = torch.nan_to_num(ck.float()).to(torch.bfloat16), torch.nan_to_num(cv.float()).to(torch.bfloat16)
    scale = 1.0 / math.sqrt(D)
    ok = torch.tensor([b != 1 for b in range(B)])
    pos = (kv_len - 1).numpy()
    ek, ev = orc.kv_append(ck, cv, kn, vn, pos, ok.to(torch.int32).numpy())
    ek_t = torch.from_numpy(ek.view(np.int16)).view(torch.bfloat16)
    ev_t = torch.from_numpy(ev.view(np.int16)).view(torch.bfloat16)
    ref, _ = orc.decode(q, ek_t, ev_t, torch.where(ok, kv_len, torch.zeros_like(kv_len)).numpy(), scale)
    dk, dv = ck.cuda(), cv.cuda()
    o = nan_bf16((B, Hq, D)).cuda()
    lse = torch.full((B, Hq), float("nan"), device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, bound)
    l4l.l4l_attn_decode_append(q.cuda(), o, dk, dv, kn.cuda(), vn.cuda(), kv_len.cuda(), bound, scale, ws, lse=lse)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert bits_equal(dk, ek) and bits_equal(dv, ev)         # sequence 1's cache untouched, the others got their row
    assert_close_to_oracle(o, ref, "decode_append with one over-long sequence")
    assert torch.isneginf(lse[1]).all() and torch.isfinite(lse[ok.cuda()]).all()
