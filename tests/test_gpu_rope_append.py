"""l4l_rope_kv_append (rotary embedding + optional RMS norm of q and k, fused with the cache update) against the
oracle, alone and followed by the attention calls that consume its outputs."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from paper_2608_21836_b200.workloads import make_rope_tables
from helpers import Guarded, assert_close_to_oracle, bits_equal

pytestmark = pytest.mark.gpu
SENTINEL = 0x4D4D


def sentinel_bf16(shape):
    return torch.full(shape, SENTINEL, dtype=torch.int16).view(torch.bfloat16)


def ordered(bits_u16: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> integers whose order is the order of the values (so a difference of 1 is one ulp)."""
    b = bits_u16.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def assert_bf16_close(gpu: torch.Tensor, want_bits: np.ndarray, what: str):
    """The GPU rotates in fp32 and rounds once; the oracle rounds the fp64 value. They may differ by one bf16 ulp
    where the exact value sits within fp32 rounding error of a tie (expected ~1e-4 of the elements)."""
    got = orc.bits(gpu.cpu())
    d = np.abs(ordered(got) - ordered(want_bits))
    assert d.max() <= 1, f"{what}: off by {d.max()} ulp"
    assert (d != 0).mean() <= 2e-3, f"{what}: {(d != 0).mean():.2e} of the elements differ"


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("norm", [False, True])
def test_rope_append_ragged(D, norm):
    B, T, Hq, Hkv, Lmax, n_pos = 5, 37, 8, 2, 96, 80
    g = torch.Generator().manual_seed(800 + D + norm)
    q = torch.randn(B, T, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    ck, cv = sentinel_bf16((B, Hkv, Lmax, D)), sentinel_bf16((B, Hkv, Lmax, D))
    pos = [0, 5, 60, 79, 43]                       # third runs past the table (80), fourth has one valid token
    n_new = [37, 1, 37, 20, 0]
    cos, sin = make_rope_tables(n_pos, D)
    qw = (torch.rand(D, generator=g) + 0.5) if norm else None
    kw = (torch.rand(D, generator=g) + 0.5) if norm else None
    eps = 1e-6 if norm else 0.0
    ref_q, ref_ck, ref_cv, _, _ = orc.rope_kv_append(q, k, v, ck, cv, pos, n_new, cos.numpy(), sin.numpy(),
                                                      None if qw is None else qw.numpy(),
                                                      None if kw is None else kw.numpy(), eps)
    gq, gk, gv, gck, gcv = Guarded(q), Guarded(k), Guarded(v), Guarded(ck), Guarded(cv)
    l4l.l4l_rope_kv_append(gq.t, gk.t, gv.t, gck.t, gcv.t, torch.tensor(pos, dtype=torch.int32).cuda(),
                           torch.tensor(n_new, dtype=torch.int32).cuda(), cos.cuda(), sin.cuda(),
                           None if qw is None else qw.cuda(), None if kw is None else kw.cuda(), eps)
    torch.cuda.synchronize()
    for x in (gq, gk, gv, gck, gcv):
        assert x.margins_intact()
    assert bits_equal(gk.t, k) and bits_equal(gv.t, v)                       # inputs are only read
    assert np.array_equal(orc.bits(gcv.t.cpu()), ref_cv)                     # v: bit for bit, other slots untouched
    assert_bf16_close(gq.t, ref_q, "q")
    assert_bf16_close(gck.t, ref_ck, "cache k")
    # slots and rows that must not be written are exactly as before
    untouched_k = ref_ck == SENTINEL
    assert (orc.bits(gck.t.cpu())[untouched_k] == SENTINEL).all()
    skipped = np.zeros((B, T), bool)
    for b in range(B):
        for t in range(T):
            skipped[b, t] = not (t < n_new[b] and pos[b] + t < min(Lmax, n_pos))
    assert np.array_equal(orc.bits(gq.t.cpu())[skipped], orc.bits(q)[skipped])


def test_rope_append_then_attention_matches_the_oracle_chain():
    """Prompt: rope + append at position 0, then attention over the cache (past = 0). Then three single-token
    steps: rope + append of one token, decode. The oracle chain is rope -> causal prefill / decode on ITS rounded
    values."""
    B, S, steps, Hq, Hkv, D, Lmax = 2, 300, 3, 8, 2, 128, 384
    g = torch.Generator().manual_seed(77)
    T = S + steps
    q = torch.randn(B, T, Hq, D, generator=g).to(torch.bfloat16)
    k = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(B, T, Hkv, D, generator=g).to(torch.bfloat16)
    qw, kw = torch.rand(D, generator=g) + 0.5, torch.rand(D, generator=g) + 0.5
    cos, sin = make_rope_tables(Lmax, D)
    scale = 1.0 / math.sqrt(D)
    lens = [S, 123]
    # ---- oracle: rotate everything it will ever need (positions b-dependent for the second sequence's steps)
    ck0 = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16)
    oq, ock, ocv, _, _ = orc.rope_kv_append(q[:, :S].contiguous(), k[:, :S].contiguous(), v[:, :S].contiguous(), ck0,
                                            ck0.clone(), [0, 0], lens, cos.numpy(), sin.numpy(), qw.numpy(), kw.numpy(),
                                            1e-6)
    ref_o, _ = orc.prefill_chunk(oq, ock, ocv, np.zeros(B, np.int32), np.array(lens, np.int32), scale)
    # ---- GPU
    dq, dk, dv = q.cuda(), k.cuda(), v.cuda()
    dck = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16, device="cuda")
    dcv = torch.zeros_like(dck)
    dcos, dsin, dqw, dkw = cos.cuda(), sin.cuda(), qw.cuda(), kw.cuda()
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    dlens = torch.tensor(lens, dtype=torch.int32, device="cuda")
    qp = dq[:, :S].clone()
    l4l.l4l_rope_kv_append(qp, dk[:, :S], dv[:, :S], dck, dcv, zero, dlens, dcos, dsin, dqw, dkw, 1e-6)
    out = torch.zeros(B, S, Hq, D, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, B, Hq, Hkv, D, S)
    l4l.l4l_attn_prefill_chunk(qp, out, dck, dcv, zero, dlens, scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for b in range(B):
        assert_close_to_oracle(out[b, :lens[b]].cpu(), ref_o[b, :lens[b]], f"rope + prefill, sequence {b}")
    # ---- decode steps
    wsd = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    cur = np.array(lens, np.int32)
    for s in range(steps):
        tok = S + s
        oq1, ock, ocv, _, _ = orc.rope_kv_append(q[:, tok:tok + 1].contiguous(), k[:, tok:tok + 1].contiguous(),
                                                 v[:, tok:tok + 1].contiguous(), ock, ocv, cur, None, cos.numpy(),
                                                 sin.numpy(), qw.numpy(), kw.numpy(), 1e-6)
        ref_d, _ = orc.decode(oq1[:, 0], ock, ocv, cur + 1, scale)
        q1 = dq[:, tok:tok + 1].clone()
        dcur = torch.tensor(cur, dtype=torch.int32, device="cuda")
        l4l.l4l_rope_kv_append(q1, dk[:, tok:tok + 1], dv[:, tok:tok + 1], dck, dcv, dcur, None, dcos, dsin, dqw, dkw,
                               1e-6)
        od = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
        l4l.l4l_attn_decode(q1[:, 0], od, dck, dcv, dcur + 1, int(cur.max()) + 1, scale, wsd)
        torch.cuda.synchronize()
        assert l4l.l4l_last_device_error(wsd) == 0
        assert_close_to_oracle(od.cpu(), ref_d, f"rope + decode step {s}")
        cur = cur + 1
    assert_bf16_close(dck, ock, "cache k after the steps")
    assert np.array_equal(orc.bits(dcv.cpu()), ocv)


def test_rope_append_rejects_bad_arguments():
    B, T, Hq, Hkv, D = 1, 4, 4, 2, 64
    q = torch.zeros(B, T, Hq, D, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(B, T, Hkv, D, dtype=torch.bfloat16, device="cuda")
    ck = torch.zeros(B, Hkv, 8, D, dtype=torch.bfloat16, device="cuda")
    cos, sin = make_rope_tables(8, D)
    pos = torch.zeros(B, dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        l4l.l4l_rope_kv_append(q, k, k.clone(), ck, ck.clone(), pos, None, cos.cuda()[:, :16].contiguous(), sin.cuda())
    with pytest.raises(TypeError):
        l4l.l4l_rope_kv_append(q, k, k.clone(), ck, ck.clone(), pos, None, cos, sin.cuda())     # host table
    with pytest.raises(l4l.L4LError):
        l4l.l4l_rope_kv_append(q, k, k.clone(), ck, ck.clone(), pos, None, cos.cuda(), sin.cuda(), eps=-1.0)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4), (16, 1)])
@pytest.mark.parametrize("norm", [False, True])
def test_decode_step_with_rope_and_append_in_one_launch(D, Hq, Hkv, norm):
    """l4l_attn_decode_rope_append against the oracle chain rope -> append -> decode, over several steps, with lengths
    that put the new token at the start, in the middle and at the end of tiles."""
    B, Lmax, steps = 6, 700, 3
    lens = np.array([1, 16, 17, 128, 129, 600], np.int32)        # kv_len INCLUDING the new token at the first step
    g = torch.Generator().manual_seed(900 + D + Hq + norm)
    ck = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, Lmax, D, generator=g).to(torch.bfloat16)
    cos, sin = make_rope_tables(Lmax, D)
    qw = (torch.rand(D, generator=g) + 0.5) if norm else None
    kw = (torch.rand(D, generator=g) + 0.5) if norm else None
    eps = 1e-6 if norm else 0.0
    scale = 1.0 / math.sqrt(D)
    dck, dcv = ck.cuda(), cv.cuda()
    ock, ocv = orc.bits(ck), orc.bits(cv)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    dcos, dsin = cos.cuda(), sin.cuda()
    for s in range(steps):
        q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
        kn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
        vn = torch.randn(B, 1, Hkv, D, generator=g).to(torch.bfloat16)
        cur = lens + s
        oq, ock, ocv, _, _ = orc.rope_kv_append(q.view(B, 1, Hq, D), kn, vn, ock, ocv, cur - 1, None, cos.numpy(),
                                                sin.numpy(), None if qw is None else qw.numpy(),
                                                None if kw is None else kw.numpy(), eps)
        ref, _ = orc.decode(oq[:, 0], ock, ocv, cur, scale)
        dq = q.cuda()
        q_before = dq.clone()
        o = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device="cuda")
        l4l.l4l_attn_decode_rope_append(dq, o, dck, dcv, kn.cuda(), vn.cuda(), torch.from_numpy(cur).cuda(), Lmax, scale,
                                        dcos, dsin, ws, q_weight=None if qw is None else qw.cuda(),
                                        k_weight=None if kw is None else kw.cuda(), eps=eps)
        torch.cuda.synchronize()
        assert l4l.l4l_last_device_error(ws) == 0
        assert bits_equal(dq, q_before)                                          # q is read only
        assert_close_to_oracle(o.cpu(), ref, f"rope + append + decode, step {s}")
    assert_bf16_close(dck, ock, "cache k after the fused steps")
    assert np.array_equal(orc.bits(dcv.cpu()), ocv)
