"""Parity of l4l_attn_decode / l4l_kv_append (CUDA, through the C ABI) with the fp64 oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from paper_2608_21836_b200 import workloads as wl
from helpers import Guarded, assert_close_to_oracle, bits_equal, nan_bf16

pytestmark = pytest.mark.gpu


def run_decode(q, ck, cv, kv_len, scale, max_kv_len=None, want_lse=True, ws_bytes=None, strided_cache=False):
    """q [B,Hq,D], caches [B,Hkv,Lmax,D] (CPU bf16), kv_len int32 [B] -> (o, lse, guards)."""
    B, Hq, D = q.shape
    Hkv, Lmax = ck.shape[1], ck.shape[2]
    gq = Guarded(q)
    if strided_cache:   # token-major storage [B, Lmax, Hkv, D] viewed as [B, Hkv, Lmax, D]
        gk, gv = Guarded(ck.permute(0, 2, 1, 3).contiguous()), Guarded(cv.permute(0, 2, 1, 3).contiguous())
        dk, dv = gk.t.permute(0, 2, 1, 3), gv.t.permute(0, 2, 1, 3)
    else:
        gk, gv = Guarded(ck), Guarded(cv)
        dk, dv = gk.t, gv.t
    go = Guarded(nan_bf16((B, Hq, D)))
    glse = Guarded(torch.full((B, Hq), float("nan")))
    lens = kv_len.to(torch.int32).cuda()
    max_kv_len = Lmax if max_kv_len is None else max_kv_len
    if ws_bytes is None:
        ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, max_kv_len)
    else:
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        l4l.l4l_workspace_init(ws)
    l4l.l4l_attn_decode(gq.t, go.t, dk, dv, lens, max_kv_len, scale, ws, lse=glse.t if want_lse else None)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    for g in (gq, gk, gv, go, glse):
        assert g.margins_intact()
    return go.t, glse.t


def check_decode(q, ck, cv, kv_len, scale, **kw):
    ref, ref_lse = orc.decode(q, ck, cv, kv_len.numpy(), scale)
    o, lse = run_decode(q, ck, cv, kv_len, scale, **kw)
    stats = assert_close_to_oracle(o, ref, "decode o")
    got_lse = lse.cpu().double().numpy()
    fin = np.isfinite(ref_lse)
    assert np.array_equal(np.isneginf(got_lse), np.isneginf(ref_lse))
    assert np.abs(got_lse[fin] - ref_lse[fin]).max() <= 2e-3
    return o, stats


def random_batch(B, Hq, Hkv, D, Lmax, lens, seed, value_scale=1.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(B, Hq, D, generator=g) * value_scale).to(torch.bfloat16)
    ck = (torch.randn(B, Hkv, Lmax, D, generator=g) * value_scale).to(torch.bfloat16)
    cv = (torch.randn(B, Hkv, Lmax, D, generator=g) * value_scale).to(torch.bfloat16)
    kv_len = torch.tensor(lens, dtype=torch.int32)
    dead = torch.arange(Lmax).view(1, 1, Lmax, 1) >= kv_len.view(B, 1, 1, 1)
    nan = nan_bf16((1,))
    return q, torch.where(dead, nan, ck).contiguous(), torch.where(dead, nan, cv).contiguous(), kv_len


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("Hq,Hkv", [(4, 2), (8, 8), (8, 2), (8, 1), (16, 1), (6, 2), (3, 1)])
def test_decode_ragged_edge_lengths(D, Hq, Hkv):
    lens = [0, 1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 191, 300, 320]
    q, ck, cv, kv_len = random_batch(len(lens), Hq, Hkv, D, 320, lens, seed=100 + D + Hq)
    check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(D))


@pytest.mark.parametrize("D", [64, 128])
def test_decode_many_splits_and_forced_large_chunks(D):
    # one long sequence on few heads: small chunks, many partials per (sequence, head)
    lens = [3000, 77]
    q, ck, cv, kv_len = random_batch(2, 4, 1, D, 3072, lens, seed=7)
    o1, _ = check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(D))
    # a workspace too small for the preferred split: the library must grow the chunks, not fail
    small = 256 + 128 * 1024 + 2 * 4 * 3 * (D + 1) * 4
    o2, _ = check_decode(q, ck, cv, kv_len, 1.0 / math.sqrt(D), ws_bytes=small)
    # and an upper bound far above the real lengths is only a hint
    o3, _ = check_decode(q, ck, cv, torch.tensor([100, 77], dtype=torch.int32), 1.0 / math.sqrt(D))


def test_decode_token_major_cache_layout():
    lens = [200, 64, 1, 131]
    q, ck, cv, kv_len = random_batch(4, 8, 2, 128, 256, lens, seed=9)
    check_decode(q, ck, cv, kv_len, 0.09, strided_cache=True)


def test_decode_is_deterministic():
    lens = [1000, 513, 2047, 64]
    q, ck, cv, kv_len = random_batch(4, 8, 2, 128, 2048, lens, seed=11)
    o1, l1 = run_decode(q, ck, cv, kv_len, 0.088)
    o2, l2 = run_decode(q, ck, cv, kv_len, 0.088)
    assert bits_equal(o1, o2) and torch.equal(l1, l2)


def test_decode_closed_forms_on_gpu():
    B, Hq, Hkv, D, L = 2, 4, 2, 64, 200
    g = torch.Generator().manual_seed(13)
    q = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    cv = torch.randn(B, Hkv, L, D, generator=g).to(torch.bfloat16)
    # identical keys -> mean of V
    ck = torch.randn(B, Hkv, 1, D, generator=g).to(torch.bfloat16).expand(B, Hkv, L, D).contiguous()
    kv_len = torch.tensor([L, 150], dtype=torch.int32)
    o, _ = run_decode(q, ck, cv, kv_len, 0.125)
    for b, n in enumerate(kv_len.tolist()):
        mean = cv[b, :, :n].double().mean(dim=1).repeat_interleave(Hq // Hkv, dim=0).numpy()
        assert np.abs(o[b].cpu().double().numpy() - mean).max() <= 2e-2
    # one dominant key -> its V row, exactly (weights underflow to 0 next to 1)
    q1 = torch.ones(B, Hq, D).to(torch.bfloat16)
    ck1 = torch.zeros(B, Hkv, L, D).to(torch.bfloat16)
    ck1[:, :, 37] = 4.0
    o, _ = run_decode(q1, ck1, cv, kv_len, 1.0)
    assert bits_equal(o, cv[:, :, 37].repeat_interleave(Hq // Hkv, dim=1).contiguous())


def test_config_batched_decode_full_size():
    w = wl.WORKLOADS["batched_decode"]
    db = wl.make_decode_batch(w)
    assert db.kv_len.min() >= 512 and db.kv_len.max() <= 4096
    check_decode(db.q, db.cache_k, db.cache_v, db.kv_len, w.scale)


def test_config_mha_small_decode_full_size():
    w = wl.WORKLOADS["mha_small"]
    db = wl.make_decode_batch(w)
    check_decode(db.q, db.cache_k, db.cache_v, db.kv_len, w.scale)


@pytest.mark.parametrize("name", ["tiny", "layer8b"])
def test_config_append_then_decode_steps_equal_prefill_rows(name):
    """Decode at step t must equal causal-prefill row S+t of the same sequence (oracle prefill rows)."""
    w = wl.WORKLOADS[name]
    seq = wl.make_sequence(w)
    B, S, T, Hq, Hkv, D = w.prefill_B, seq.S, seq.T, w.Hq, w.Hkv, w.D
    Lmax = S + T
    gk, gv = Guarded(nan_bf16((B, Hkv, Lmax, D))), Guarded(nan_bf16((B, Hkv, Lmax, D)))
    k_dev, v_dev, q_dev = seq.k.cuda(), seq.v.cuda(), seq.q.cuda()
    # the prompt's K/V enter the cache through the append entry point (T = S tokens at once)
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    l4l.l4l_kv_append(gk.t, gv.t, k_dev[:, :S], v_dev[:, :S], zero)
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, B, Hq, Hkv, D, Lmax)
    steps = list(range(T)) if name == "tiny" else [0, 1, 63, 64, 127, 200, 255]
    outs = torch.empty(B, T, Hq, D, dtype=torch.bfloat16, device="cuda")
    for t in range(T):
        pos = torch.full((B,), S + t, dtype=torch.int32, device="cuda")
        l4l.l4l_kv_append(gk.t, gv.t, k_dev[:, S + t:S + t + 1], v_dev[:, S + t:S + t + 1], pos)
        l4l.l4l_attn_decode(q_dev[:, S + t].contiguous(), outs[:, t], gk.t, gv.t, pos + 1, Lmax, w.scale, ws)
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0 and gk.margins_intact() and gv.margins_intact()
    # cache == the sequence's K/V, bit for bit
    assert bits_equal(gk.t, seq.k.permute(0, 2, 1, 3).contiguous())
    assert bits_equal(gv.t, seq.v.permute(0, 2, 1, 3).contiguous())
    rows = [(b, S + t, h) for b in range(B) for t in steps for h in range(Hq)]
    ref, _ = orc.prefill_rows(seq.q, seq.k, seq.v, np.full(B, S + T, np.int32), w.scale, rows)
    got = torch.stack([outs[b, t, h] for b in range(B) for t in steps for h in range(Hq)])
    assert_close_to_oracle(got, ref, f"{name} decode steps")


def test_decode_repeated_calls_on_one_workspace_stay_correct():
    """The ticket counters and partials live in the workspace across calls: alternate two different
    batches many times on ONE workspace (every merge path: sequences cut in 2, 3 and more pieces) and
    check each result against the oracle's."""
    D, Hq, Hkv, Lmax = 128, 32, 8, 4096
    rng = np.random.default_rng(77)
    batches = []
    for seed, B in ((1, 32), (2, 24)):
        lens = rng.integers(512, 4097, B).tolist()
        lens[0], lens[1] = 4096, 1                      # the longest possible and a trivial one
        q, ck, cv, kv_len = random_batch(B, Hq, Hkv, D, Lmax, lens, seed=900 + seed)
        ref, _ = orc.decode(q, ck, cv, kv_len.numpy(), 0.09)
        batches.append((q.cuda(), ck.cuda(), cv.cuda(), kv_len.cuda(), ref))
    ws = l4l.new_workspace(l4l.L4L_OP_DECODE, 32, Hq, Hkv, D, Lmax)
    for it in range(12):
        q, ck, cv, kv_len, ref = batches[it % 2]
        o = torch.zeros_like(q)
        l4l.l4l_attn_decode(q, o, ck, cv, kv_len, Lmax, 0.09, ws)
        if it in (0, 1, 6, 11):
            torch.cuda.synchronize()
            assert_close_to_oracle(o, ref, f"repeated decode, call {it}")
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
