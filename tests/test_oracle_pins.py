"""Pins of the CPU oracle against what softmax attention fixes by definition.

The paper prints no formula and no worked numeric example for attention, so nothing
here comes from a printed value; every pin is a closed form, an invariant, a special
case that reduces to a textbook/library routine, or brute force on tiny inputs. Each is
chosen so that a plausible slip in the oracle (dropped scale, wrong head mapping,
off-by-one causal bound, transposed operand, missing normalisation) fails at least one.
"""
import math
import struct

import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc


def bf16(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16)


def randn(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return bf16(torch.randn(shape, generator=g) * scale)


def f64(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.float64).numpy()


def full_lens(B, S):
    return np.full((B,), S, dtype=np.int32)


def cache_from(k: torch.Tensor) -> torch.Tensor:
    """[B, L, Hkv, D] token-major -> cache layout [B, Hkv, L, D]."""
    return k.permute(0, 2, 1, 3).contiguous()


# --------------------------------------------------------------------------- I5 brute force
def _bf16_bits_to_float(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", (bits & 0xFFFF) << 16))[0]


def brute_force_row(qrow, keys, vals, scale):
    """Independent evaluation in pure Python: no max subtraction, d-outer loop order,
    exact-sum accumulation with math.fsum."""
    n, D = len(keys), len(qrow)
    s = [0.0] * n
    for d in range(D):
        for j in range(n):
            s[j] += qrow[d] * keys[j][d]
    w = [math.exp(scale * sj) for sj in s]
    z = math.fsum(w)
    out = [math.fsum(w[j] * vals[j][d] for j in range(n)) / z for d in range(D)]
    return out, math.log(z)


@pytest.mark.parametrize("B,S,Hq,Hkv,D", [(2, 8, 4, 2, 8), (1, 5, 3, 1, 4), (2, 7, 2, 2, 6)])
def test_I5_bruteforce_prefill_and_decode(B, S, Hq, Hkv, D):
    q, k, v = randn((B, S, Hq, D), 1), randn((B, S, Hkv, D), 2), randn((B, S, Hkv, D), 3)
    scale = 0.37
    out, lse = orc.prefill(q, k, v, full_lens(B, S), scale)
    qb, kb, vb = orc.bits(q), orc.bits(k), orc.bits(v)
    G = Hq // Hkv
    for b in range(B):
        for i in range(S):
            for h in range(Hq):
                g = h // G
                qrow = [_bf16_bits_to_float(int(x)) for x in qb[b, i, h]]
                keys = [[_bf16_bits_to_float(int(x)) for x in kb[b, j, g]] for j in range(i + 1)]
                vals = [[_bf16_bits_to_float(int(x)) for x in vb[b, j, g]] for j in range(i + 1)]
                ref, ref_lse = brute_force_row(qrow, keys, vals, scale)
                np.testing.assert_allclose(out[b, i, h], ref, rtol=0, atol=1e-12)
                assert abs(lse[b, h, i] - ref_lse) < 1e-12
    # decode over the same data, all tokens visible
    dq = q[:, -1].contiguous()
    dout, dlse = orc.decode(dq, cache_from(k), cache_from(v), full_lens(B, S), scale)
    np.testing.assert_allclose(dout, out[:, -1], rtol=0, atol=1e-13)
    np.testing.assert_allclose(dlse, lse[:, :, -1], rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- I1 identical keys
def test_I1_identical_keys_give_prefix_mean_of_v():
    B, S, Hq, Hkv, D = 2, 33, 4, 2, 16
    q = randn((B, S, Hq, D), 4)
    k = randn((B, 1, Hkv, D), 5).expand(B, S, Hkv, D).contiguous()
    v = randn((B, S, Hkv, D), 6)
    out, lse = orc.prefill(q, k, v, full_lens(B, S), 0.25)
    vv = f64(v)
    counts = np.arange(1, S + 1, dtype=np.float64)[None, :, None, None]
    pm = np.cumsum(vv, axis=1) / counts                 # prefix mean  [B,S,Hkv,D]
    np.testing.assert_allclose(out, np.repeat(pm, Hq // Hkv, axis=2), rtol=0, atol=1e-13)
    # lse = common score + log(number of keys)
    s = 0.25 * np.einsum("bihd,bhd->bih", f64(q), np.repeat(f64(k)[:, 0], Hq // Hkv, axis=1))
    np.testing.assert_allclose(lse, (s + np.log(counts[..., 0])).transpose(0, 2, 1), rtol=0, atol=1e-12)
    dout, _ = orc.decode(q[:, -1].contiguous(), cache_from(k), cache_from(v), full_lens(B, S), 0.25)
    np.testing.assert_allclose(dout, np.repeat(vv.mean(axis=1), Hq // Hkv, axis=1), rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- I2 dominant key
def test_I2_single_dominant_score_returns_its_v_row():
    B, S, H, D = 1, 24, 2, 8
    q = bf16(torch.ones(B, S, H, D))
    k = bf16(torch.zeros(B, S, H, D))
    jstar = 5
    k[:, jstar] = 16.0                                   # score 16*8 = 128 above the rest
    v = randn((B, S, H, D), 7)
    out, _ = orc.prefill(q, k, v, full_lens(B, S), 1.0)
    vv = f64(v)
    for i in range(jstar, S):
        np.testing.assert_allclose(out[0, i], vv[0, jstar], rtol=0, atol=1e-30 + i * math.exp(-128) * 10)
    # before the dominant key is visible all scores tie: prefix mean
    np.testing.assert_allclose(out[0, jstar - 1], vv[0, :jstar].mean(axis=0), rtol=0, atol=1e-13)
    dout, _ = orc.decode(q[:, -1].contiguous(), cache_from(k), cache_from(v), full_lens(B, S), 1.0)
    np.testing.assert_allclose(dout[0], vv[0, jstar], rtol=0, atol=1e-30)


# --------------------------------------------------------------------------- I3 causality
def test_I3_future_tokens_do_not_change_earlier_rows():
    B, S, Hq, Hkv, D = 1, 20, 4, 2, 8
    q, k, v = randn((B, S, Hq, D), 8), randn((B, S, Hkv, D), 9), randn((B, S, Hkv, D), 10)
    out0, lse0 = orc.prefill(q, k, v, full_lens(B, S), 0.3)
    cut = 11
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    q2[:, cut:], k2[:, cut:], v2[:, cut:] = randn((B, S - cut, Hq, D), 11), 7.0, -3.0
    out1, lse1 = orc.prefill(q2, k2, v2, full_lens(B, S), 0.3)
    assert np.array_equal(out0[:, :cut], out1[:, :cut])
    assert np.array_equal(lse0[:, :, :cut], lse1[:, :, :cut])
    assert not np.array_equal(out0[:, cut:], out1[:, cut:])
    # the diagonal IS visible: changing token i's own k/v changes row i
    k3 = k.clone()
    k3[:, cut - 1] = 2.0
    out2, _ = orc.prefill(q, k3, v, full_lens(B, S), 0.3)
    assert np.array_equal(out0[:, : cut - 1], out2[:, : cut - 1])
    assert not np.array_equal(out0[:, cut - 1], out2[:, cut - 1])


def test_ragged_seq_len_ignores_padding_and_leaves_rows_undefined():
    B, S, Hq, Hkv, D = 2, 12, 2, 1, 8
    q, k, v = randn((B, S, Hq, D), 12), randn((B, S, Hkv, D), 13), randn((B, S, Hkv, D), 14)
    lens = np.array([7, 12], dtype=np.int32)
    out, lse = orc.prefill(q, k, v, lens, 0.5)
    full, _ = orc.prefill(q, k, v, full_lens(B, S), 0.5)
    assert np.array_equal(out[0, :7], full[0, :7]) and np.array_equal(out[1], full[1])
    assert np.isnan(out[0, 7:]).all() and np.isnan(lse[0, :, 7:]).all()


# --------------------------------------------------------------------------- I4 phase equivalence
def test_I4_decode_step_equals_prefill_row():
    B, L, Hq, Hkv, D = 2, 19, 4, 2, 8
    q, k, v = randn((B, L, Hq, D), 15), randn((B, L, Hkv, D), 16), randn((B, L, Hkv, D), 17)
    out, lse = orc.prefill(q, k, v, full_lens(B, L), 0.41)
    Lmax = 32
    ck = torch.zeros(B, Hkv, Lmax, D, dtype=torch.bfloat16)
    cv = torch.zeros_like(ck)
    ck[:, :, :L], cv[:, :, :L] = cache_from(k), cache_from(v)
    ck[:, :, L:], cv[:, :, L:] = float("nan"), float("nan")      # must never be read
    for t in (0, 1, 7, L - 1):
        dout, dlse = orc.decode(q[:, t].contiguous(), ck, cv, full_lens(B, t + 1), 0.41)
        np.testing.assert_allclose(dout, out[:, t], rtol=0, atol=1e-14)
        np.testing.assert_allclose(dlse, lse[:, :, t], rtol=0, atol=1e-14)


# --------------------------------------------------------------------------- I6, I7
def test_I6_first_row_is_v0_exactly_and_empty_is_zero():
    B, S, Hq, Hkv, D = 2, 4, 4, 2, 8
    q, k, v = randn((B, S, Hq, D), 18), randn((B, S, Hkv, D), 19), randn((B, S, Hkv, D), 20)
    out, lse = orc.prefill(q, k, v, full_lens(B, S), 0.7)
    assert np.array_equal(out[:, 0], np.repeat(f64(v)[:, 0], Hq // Hkv, axis=1))
    s00 = 0.7 * np.einsum("bhd,bhd->bh", f64(q)[:, 0], np.repeat(f64(k)[:, 0], Hq // Hkv, axis=1))
    np.testing.assert_allclose(lse[:, :, 0], s00, rtol=0, atol=1e-14)
    dout, _ = orc.decode(q[:, 0].contiguous(), cache_from(k), cache_from(v), full_lens(B, 1), 0.7)
    assert np.array_equal(dout, out[:, 0])
    dout0, dlse0 = orc.decode(q[:, 0].contiguous(), cache_from(k), cache_from(v), np.zeros(B, np.int32), 0.7)
    assert (dout0 == 0).all() and np.isneginf(dlse0).all()


def test_I7_zero_scale_gives_running_mean():
    B, S, Hq, Hkv, D = 1, 40, 2, 2, 4
    q, k, v = randn((B, S, Hq, D), 21), randn((B, S, Hkv, D), 22), randn((B, S, Hkv, D), 23)
    out, lse = orc.prefill(q, k, v, full_lens(B, S), 0.0)
    counts = np.arange(1, S + 1, dtype=np.float64)[None, :, None, None]
    np.testing.assert_allclose(out, np.cumsum(f64(v), axis=1) / counts, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse[0, 0], np.log(counts[0, :, 0, 0]), rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- I8 head mapping
def test_I8_gqa_equals_mha_with_consecutively_repeated_kv_heads():
    B, S, Hq, Hkv, D = 1, 16, 8, 2, 8
    G = Hq // Hkv
    q, k, v = randn((B, S, Hq, D), 24), randn((B, S, Hkv, D), 25), randn((B, S, Hkv, D), 26)
    out, lse = orc.prefill(q, k, v, full_lens(B, S), 0.35)
    kr, vr = k.repeat_interleave(G, dim=2), v.repeat_interleave(G, dim=2)
    out_mha, lse_mha = orc.prefill(q, kr, vr, full_lens(B, S), 0.35)
    assert np.array_equal(out, out_mha) and np.array_equal(lse, lse_mha)
    # the rejected convention (h % Hkv) would tile, not interleave: it must differ
    out_tiled, _ = orc.prefill(q, k.repeat(1, 1, G, 1), v.repeat(1, 1, G, 1), full_lens(B, S), 0.35)
    assert not np.array_equal(out, out_tiled)
    # decode uses the same mapping
    dout, _ = orc.decode(q[:, -1].contiguous(), cache_from(k), cache_from(v), full_lens(B, S), 0.35)
    dmha, _ = orc.decode(q[:, -1].contiguous(), cache_from(kr), cache_from(vr), full_lens(B, S), 0.35)
    assert np.array_equal(dout, dmha)


def test_kv_head_only_feeds_its_own_query_group():
    B, S, Hq, Hkv, D = 1, 9, 6, 3, 4
    G = Hq // Hkv
    q, k, v = randn((B, S, Hq, D), 27), randn((B, S, Hkv, D), 28), randn((B, S, Hkv, D), 29)
    out0, _ = orc.prefill(q, k, v, full_lens(B, S), 0.5)
    v2 = v.clone()
    v2[:, :, 1] += 1.0
    out1, _ = orc.prefill(q, k, v2, full_lens(B, S), 0.5)
    changed = [h for h in range(Hq) if not np.array_equal(out0[:, :, h], out1[:, :, h])]
    assert changed == list(range(G, 2 * G))


# --------------------------------------------------------------------------- I9, I10, I11
def test_I9_adding_a_constant_vector_to_every_key_changes_nothing():
    B, S, H, D = 1, 12, 2, 8
    # dyadic values so that k + c is exact in bf16
    g = torch.Generator().manual_seed(30)
    q = bf16(torch.randint(-8, 9, (B, S, H, D), generator=g) / 8.0)
    k = bf16(torch.randint(-8, 9, (B, S, H, D), generator=g) / 8.0)
    v = randn((B, S, H, D), 31)
    c = bf16(torch.randint(-8, 9, (1, 1, H, D), generator=g) / 4.0)
    out0, lse0 = orc.prefill(q, k, v, full_lens(B, S), 0.125)
    out1, lse1 = orc.prefill(q, bf16(k.float() + c.float()), v, full_lens(B, S), 0.125)
    np.testing.assert_allclose(out0, out1, rtol=0, atol=1e-13)
    shift = 0.125 * np.einsum("bihd,hd->bhi", f64(q), f64(c)[0, 0])
    np.testing.assert_allclose(lse1 - lse0, shift, rtol=0, atol=1e-12)


def test_I10_decode_is_invariant_to_a_joint_permutation_of_cache_tokens():
    B, L, Hq, Hkv, D = 2, 23, 4, 2, 8
    q = randn((B, Hq, D), 32)
    ck, cv = randn((B, Hkv, L, D), 33), randn((B, Hkv, L, D), 34)
    perm = torch.randperm(L, generator=torch.Generator().manual_seed(35))
    out0, lse0 = orc.decode(q, ck, cv, full_lens(B, L), 0.3)
    out1, lse1 = orc.decode(q, ck[:, :, perm].contiguous(), cv[:, :, perm].contiguous(), full_lens(B, L), 0.3)
    np.testing.assert_allclose(out0, out1, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse0, lse1, rtol=0, atol=1e-13)
    # permuting K alone is a different problem
    out2, _ = orc.decode(q, ck[:, :, perm].contiguous(), cv, full_lens(B, L), 0.3)
    assert np.abs(out2 - out0).max() > 1e-3


def test_I11_linear_in_v_and_constant_v_gives_constant():
    B, S, H, D = 1, 14, 2, 8
    q, k = randn((B, S, H, D), 36), randn((B, S, H, D), 37)
    g = torch.Generator().manual_seed(38)
    v1 = bf16(torch.randint(-16, 17, (B, S, H, D), generator=g) / 8.0)
    v2 = bf16(torch.randint(-16, 17, (B, S, H, D), generator=g) / 8.0)
    o1, _ = orc.prefill(q, k, v1, full_lens(B, S), 0.3)
    o2, _ = orc.prefill(q, k, v2, full_lens(B, S), 0.3)
    o12, _ = orc.prefill(q, k, bf16(2.0 * v1.float() - 0.5 * v2.float()), full_lens(B, S), 0.3)
    np.testing.assert_allclose(o12, 2.0 * o1 - 0.5 * o2, rtol=0, atol=1e-13)
    oc, _ = orc.prefill(q, k, bf16(torch.full((B, S, H, D), 1.75)), full_lens(B, S), 0.3)
    np.testing.assert_allclose(oc, 1.75, rtol=0, atol=1e-14)


# --------------------------------------------------------------------------- I12 split/merge
def test_I12_lse_merge_of_any_partition_equals_the_whole():
    B, L, Hq, Hkv, D = 1, 50, 4, 2, 8
    q = randn((B, Hq, D), 39)
    ck, cv = randn((B, Hkv, L, D), 40, 2.0), randn((B, Hkv, L, D), 41)
    whole, whole_lse = orc.decode(q, ck, cv, full_lens(B, L), 0.4)
    cuts = [0, 3, 4, 21, 50]
    parts = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        o, l = orc.decode(q, ck[:, :, a:b].contiguous(), cv[:, :, a:b].contiguous(), full_lens(B, b - a), 0.4)
        parts.append((o, l))
    lses = np.stack([l for _, l in parts])                # [C,B,Hq]
    m = lses.max(axis=0)
    w = np.exp(lses - m)
    merged = sum(w[c][..., None] * parts[c][0] for c in range(len(parts))) / w.sum(axis=0)[..., None]
    np.testing.assert_allclose(merged, whole, rtol=0, atol=1e-13)
    np.testing.assert_allclose(m + np.log(w.sum(axis=0)), whole_lse, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- I13 library routine
@pytest.mark.parametrize("B,S,Hq,Hkv,D", [(2, 37, 4, 2, 16), (1, 64, 6, 6, 8)])
def test_I13_matches_torch_sdpa_float64(B, S, Hq, Hkv, D):
    q, k, v = randn((B, S, Hq, D), 42), randn((B, S, Hkv, D), 43), randn((B, S, Hkv, D), 44)
    scale = 1.0 / math.sqrt(D)
    out, _ = orc.prefill(q, k, v, full_lens(B, S), scale)
    G = Hq // Hkv
    qq = q.double().permute(0, 2, 1, 3)
    kk = k.double().repeat_interleave(G, dim=2).permute(0, 2, 1, 3)
    vv = v.double().repeat_interleave(G, dim=2).permute(0, 2, 1, 3)
    ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, is_causal=True, scale=scale)
    np.testing.assert_allclose(out, ref.permute(0, 2, 1, 3).numpy(), rtol=0, atol=1e-12)
    dref = torch.nn.functional.scaled_dot_product_attention(qq[:, :, -1:], kk, vv, is_causal=False, scale=scale)
    dout, _ = orc.decode(q[:, -1].contiguous(), cache_from(k), cache_from(v), full_lens(B, S), scale)
    np.testing.assert_allclose(dout, dref[:, :, 0].numpy(), rtol=0, atol=1e-12)


def test_chunk_over_populated_cache_equals_rows_of_the_full_prefill():
    """Prefill of tokens [P, P+L) over a cache that holds tokens [0, P+L) must give rows P..P+L-1 of the causal
    prefill of the whole sequence, and with L = 1 it is decode; padding slots must not matter."""
    B, T, Hq, Hkv, D = 2, 29, 4, 2, 8
    q, k, v = randn((B, T, Hq, D), 50), randn((B, T, Hkv, D), 51), randn((B, T, Hkv, D), 52)
    full, full_lse = orc.prefill(q, k, v, full_lens(B, T), 0.33)
    Lmax = 40
    ck = torch.full((B, Hkv, Lmax, D), float("nan")).to(torch.bfloat16)
    cv = ck.clone()
    ck[:, :, :T], cv[:, :, :T] = cache_from(k), cache_from(v)
    past = np.array([11, 0], np.int32)
    qlen = np.array([T - 11, 17], np.int32)
    S = int(qlen.max())
    qc = torch.zeros(B, S, Hq, D, dtype=torch.bfloat16)
    for b in range(B):
        qc[b, :qlen[b]] = q[b, past[b]:past[b] + qlen[b]]
    # the second sequence's cache is cut at past+qlen: later slots are poison
    ck[1, :, 17:], cv[1, :, 17:] = float("nan"), float("nan")
    out, lse = orc.prefill_chunk(qc, ck, cv, past, qlen, 0.33)
    for b in range(B):
        sl = slice(past[b], past[b] + qlen[b])
        np.testing.assert_allclose(out[b, :qlen[b]], full[b, sl], rtol=0, atol=1e-14)
        np.testing.assert_allclose(lse[b, :, :qlen[b]], full_lse[b, :, sl], rtol=0, atol=1e-14)
        assert np.isnan(out[b, qlen[b]:]).all()
    # one new token over P cached ones is decode with kv_len = P + 1
    d_out, d_lse = orc.decode(q[:, 20].contiguous(), ck, cv, np.array([21, 17], np.int32), 0.33)
    c_out, c_lse = orc.prefill_chunk(q[:, 20:21].contiguous(), ck, cv, np.array([20, 16], np.int32),
                                     np.array([1, 1], np.int32), 0.33)
    np.testing.assert_allclose(c_out[:, 0], d_out, rtol=0, atol=1e-14)
    with pytest.raises(ValueError):
        orc.prefill_chunk(qc, ck, cv, np.array([30, 0], np.int32), qlen, 0.33)       # past + q_len > Lmax


def test_prefill_rows_is_the_same_function_as_prefill():
    B, S, Hq, Hkv, D = 2, 21, 4, 2, 8
    q, k, v = randn((B, S, Hq, D), 45), randn((B, S, Hkv, D), 46), randn((B, S, Hkv, D), 47)
    lens = np.array([21, 13], dtype=np.int32)
    out, lse = orc.prefill(q, k, v, lens, 0.2)
    rows = [(0, 0, 0), (0, 20, 3), (1, 12, 1), (1, 5, 2)]
    o, l = orc.prefill_rows(q, k, v, lens, 0.2, rows)
    for r, (b, i, h) in enumerate(rows):
        assert np.array_equal(o[r], out[b, i, h]) and l[r] == lse[b, h, i]
    with pytest.raises(ValueError):
        orc.prefill_rows(q, k, v, lens, 0.2, [(1, 13, 0)])


# --------------------------------------------------------------------------- cache copy
def test_kv_append_is_a_bit_exact_copy_and_touches_nothing_else():
    B, T, Hkv, D, Lmax = 3, 4, 2, 8, 16
    g = torch.Generator().manual_seed(48)
    # all 16-bit patterns are legal payload (NaNs, -0, denormals): use raw random bits
    def rawbits(shape):
        return torch.randint(0, 65536, shape, generator=g, dtype=torch.int32).to(torch.int16).view(torch.bfloat16)
    ck, cv = rawbits((B, Hkv, Lmax, D)), rawbits((B, Hkv, Lmax, D))
    kn, vn = rawbits((B, T, Hkv, D)), rawbits((B, T, Hkv, D))
    pos = np.array([0, 5, 12], dtype=np.int32)
    n_new = np.array([4, 0, 3], dtype=np.int32)
    ok, ov = orc.kv_append(ck, cv, kn, vn, pos, n_new)
    ek, ev = orc.bits(ck).copy(), orc.bits(cv).copy()
    knb, vnb = orc.bits(kn), orc.bits(vn)
    for b in range(B):
        n = int(n_new[b])
        ek[b, :, pos[b]:pos[b] + n] = knb[b, :n].transpose(1, 0, 2)
        ev[b, :, pos[b]:pos[b] + n] = vnb[b, :n].transpose(1, 0, 2)
    assert np.array_equal(ok, ek) and np.array_equal(ov, ev)
    with pytest.raises(ValueError):
        orc.kv_append(ck, cv, kn, vn, np.array([0, 5, 14], np.int32), n_new)


def test_oracle_reports_thread_count():
    assert orc.num_threads() >= 1


# --------------------------------------------------------------------------- rotary embedding + RMS norm + cache update
def _rope_inputs(B=2, T=7, Hq=4, Hkv=2, D=16, Lmax=24, n_pos=32, seed=90):
    from paper_2608_21836_b200.workloads import make_rope_tables

    q, k, v = randn((B, T, Hq, D), seed), randn((B, T, Hkv, D), seed + 1), randn((B, T, Hkv, D), seed + 2)
    ck = torch.full((B, Hkv, Lmax, D), 3.0).to(torch.bfloat16)
    cv = torch.full((B, Hkv, Lmax, D), 5.0).to(torch.bfloat16)
    cos, sin = make_rope_tables(n_pos, D)
    return q, k, v, ck, cv, cos.numpy(), sin.numpy()


def test_bf16_rounding_matches_the_library_conversion():
    """The oracle's fp64 -> bf16 rounding against torch's float32 -> bfloat16 (RNE), ties and extremes included."""
    g = torch.Generator().manual_seed(5)
    x = torch.randn(20000, generator=g) * torch.exp(torch.randn(20000, generator=g) * 8)
    ties = torch.tensor([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7), 1.0 + 2.0 ** -8 + 2.0 ** -20,
                         0.0, -0.0, 3.3895313892515355e38, float("inf"), 2.0 ** -130, 1e-40])
    x = torch.cat([x, ties])
    want = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.round_bf16(x.double().numpy())
    assert np.array_equal(got, want)
    # a value just above a tie in fp64 that fp32 cannot distinguish from the tie must round up
    assert orc.round_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81


def test_rope_is_a_complex_rotation_and_keeps_relative_position():
    q, k, v, ck, cv, cos, sin = _rope_inputs()
    B, T, Hq, D = q.shape
    pos = np.array([3, 0], np.int32)
    qb, ckb, cvb, q_ex, k_ex = orc.rope_kv_append(q, k, v, ck, cv, pos, None, cos, sin)
    H = D // 2
    # (x_i, x_{i+D/2}) as a complex number times e^{i P theta_i}, with numpy's complex product
    for b in range(B):
        for t in range(T):
            P = pos[b] + t
            z = f64(q)[b, t, :, :H] + 1j * f64(q)[b, t, :, H:]
            w = z * (cos[P].astype(np.float64) + 1j * sin[P].astype(np.float64))[None, :]
            np.testing.assert_allclose(q_ex[b, t, :, :H], w.real, rtol=0, atol=1e-14)
            np.testing.assert_allclose(q_ex[b, t, :, H:], w.imag, rtol=0, atol=1e-14)
    # a rotation keeps the length of every pair
    np.testing.assert_allclose(k_ex[..., :H] ** 2 + k_ex[..., H:] ** 2, f64(k)[..., :H] ** 2 + f64(k)[..., H:] ** 2,
                               rtol=1e-6, atol=0)        # tables are float32: cos^2 + sin^2 = 1 to ~1e-7
    # position 0 is the identity, bit for bit after rounding
    assert np.array_equal(qb[1, 0], orc.bits(q)[1, 0])
    # relative position: <rope(q, m), rope(k, n)> depends on m - n only (same vectors placed 5 positions later)
    q1, k1 = q[:1, :1].contiguous(), k[:1, :1].contiguous()
    dots = []
    for shift in (0, 5, 11):
        _, _, _, qe, _ = orc.rope_kv_append(q1, k1, v[:1, :1].contiguous(), ck[:1], cv[:1], [7 + shift], None, cos, sin)
        _, _, _, _, ke = orc.rope_kv_append(q1, k1, v[:1, :1].contiguous(), ck[:1], cv[:1], [2 + shift], None, cos, sin)
        dots.append(np.einsum("d,d->", qe[0, 0, 0], ke[0, 0, 0]))
    np.testing.assert_allclose(dots[1:], dots[0], rtol=0, atol=2e-5)


def test_rope_append_writes_the_right_slots_and_nothing_else():
    q, k, v, ck, cv, cos, sin = _rope_inputs()
    B, T, Hq, D = q.shape
    Lmax = ck.shape[2]
    pos = np.array([20, 1], np.int32)                    # sequence 0 runs off the cache after 4 tokens
    n_new = np.array([7, 3], np.int32)
    qb, ckb, cvb, q_ex, k_ex = orc.rope_kv_append(q, k, v, ck, cv, pos, n_new, cos, sin)
    vb, ck0, cv0 = orc.bits(v), orc.bits(ck), orc.bits(cv)
    for b in range(B):
        written = [pos[b] + t for t in range(n_new[b]) if pos[b] + t < Lmax]
        for slot in range(Lmax):
            if slot in written:
                t = slot - pos[b]
                assert np.array_equal(cvb[b, :, slot], vb[b, t])                 # v: exact copy
                assert np.array_equal(ckb[b, :, slot], orc.round_bf16(k_ex[b, t]))
            else:
                assert np.array_equal(ckb[b, :, slot], ck0[b, :, slot]) and np.array_equal(cvb[b, :, slot], cv0[b, :, slot])
        for t in range(T):
            if t < n_new[b] and pos[b] + t < Lmax:
                assert np.array_equal(qb[b, t], orc.round_bf16(q_ex[b, t]))
            else:
                assert np.array_equal(qb[b, t], orc.bits(q)[b, t]) and np.isnan(q_ex[b, t]).all()


def test_rms_norm_part_of_rope_has_unit_rms_scale_invariance_and_weight_linearity():
    q, k, v, ck, cv, cos, sin = _rope_inputs(D=32)
    D = q.shape[-1]
    ones = np.ones(D, np.float32)
    pos = np.array([0, 0], np.int32)
    # at position 0 the rotation is the identity, so the exact output is the normalised row
    _, _, _, qn, kn = orc.rope_kv_append(q[:, :1].contiguous(), k[:, :1].contiguous(), v[:, :1].contiguous(), ck, cv,
                                         pos, None, cos, sin, q_weight=ones, k_weight=ones, eps=0.0)
    np.testing.assert_allclose(np.sqrt((qn ** 2).mean(-1)), 1.0, rtol=1e-13)
    np.testing.assert_allclose(np.sqrt((kn ** 2).mean(-1)), 1.0, rtol=1e-13)
    # scaling the input by a power of two (exact in bf16) changes nothing when eps = 0
    _, _, _, qn4, _ = orc.rope_kv_append((q[:, :1] * 4).contiguous(), k[:, :1].contiguous(), v[:, :1].contiguous(), ck,
                                         cv, pos, None, cos, sin, q_weight=ones, k_weight=ones, eps=0.0)
    np.testing.assert_allclose(qn4, qn, rtol=1e-14)
    # the weight multiplies element-wise; k without a weight is left un-normalised
    w = np.linspace(0.5, 2.0, D).astype(np.float32)
    _, _, _, qw, kraw = orc.rope_kv_append(q[:, :1].contiguous(), k[:, :1].contiguous(), v[:, :1].contiguous(), ck, cv,
                                           pos, None, cos, sin, q_weight=w, k_weight=None, eps=0.0)
    np.testing.assert_allclose(qw, qn * w.astype(np.float64), rtol=1e-14)
    np.testing.assert_allclose(kraw, f64(k[:, :1]), rtol=0, atol=0)
    # eps enters under the root: a row of constant c gives c / sqrt(c^2 + eps)
    const = torch.full((1, 1, 1, D), 0.5).to(torch.bfloat16)
    _, _, _, qc, _ = orc.rope_kv_append(const, const, const, ck[:1, :1], cv[:1, :1], [0], None, cos, sin,
                                        q_weight=ones, eps=0.75)
    np.testing.assert_allclose(qc, 0.5 / math.sqrt(0.25 + 0.75), rtol=1e-14)


# --------------------------------------------------------------------------- paged cache = the cache its pages spell out
def test_paged_decode_is_decode_over_the_pages_laid_end_to_end():
    B, Hq, Hkv, D, page, n_per = 3, 4, 2, 8, 4, 5
    Lmax = page * n_per
    q = randn((B, Hq, D), 60)
    ck, cv = randn((B, Hkv, Lmax, D), 61), randn((B, Hkv, Lmax, D), 62)
    lens = np.array([Lmax, 7, 1], np.int32)
    want, want_lse = orc.decode(q, ck, cv, lens, 0.4)
    # scatter the contiguous caches into a shuffled pool with spare, poisoned pages
    rng = np.random.default_rng(3)
    n_pages = B * n_per + 4
    perm = rng.permutation(n_pages)[: B * n_per].reshape(B, n_per)
    pool_k = torch.full((n_pages, Hkv, page, D), float("nan")).to(torch.bfloat16)
    pool_v = pool_k.clone()
    for b in range(B):
        for i in range(n_per):
            pool_k[perm[b, i]] = ck[b, :, i * page:(i + 1) * page]
            pool_v[perm[b, i]] = cv[b, :, i * page:(i + 1) * page]
    got, got_lse = orc.decode_paged(q, pool_k, pool_v, perm, lens, 0.4)
    assert np.array_equal(got, want) and np.array_equal(got_lse, want_lse)
    assert np.array_equal(orc.gather_pages(pool_k, perm, Lmax), orc.bits(ck))
    # entries past a sequence's last token are never looked at
    perm2 = perm.copy()
    perm2[1, 2:] = -1
    perm2[2, 1:] = 10 ** 6
    got2, _ = orc.decode_paged(q, pool_k, pool_v, perm2, lens, 0.4)
    assert np.array_equal(got2, want)
    # appending through the table lands where the gather finds it
    k_new, v_new = randn((B, 3, Hkv, D), 63), randn((B, 3, Hkv, D), 64)
    pos = np.array([Lmax - 2, 7, 1], np.int32)                     # sequence 0: third token falls off its table
    pk2, pv2 = orc.kv_append_paged(pool_k, pool_v, perm, k_new, v_new, pos, None)
    ck2, cv2 = orc.kv_append(ck, cv, k_new, v_new, pos, np.array([2, 3, 3], np.int32))
    assert np.array_equal(orc.gather_pages(pk2, perm, Lmax), ck2)
    assert np.array_equal(orc.gather_pages(pv2, perm, Lmax), cv2)
    # a slot whose table entry names no page of the pool is dropped: the pools come back untouched for that sequence
    perm3 = perm.copy()
    perm3[1, 7 // page] = -1
    perm3[2, 1 // page] = n_pages
    pk3, pv3 = orc.kv_append_paged(pool_k, pool_v, perm3, k_new[:, :1], v_new[:, :1], pos, np.array([0, 1, 1], np.int32))
    assert np.array_equal(pk3, orc.bits(pool_k)) and np.array_equal(pv3, orc.bits(pool_v))


# --------------------------------------------------------------------------- fp8 (e4m3) cache
def test_e4m3_code_table_and_rounding_match_the_library_type():
    codes = torch.arange(256, dtype=torch.uint8)
    want = codes.view(torch.float8_e4m3fn).float().double().numpy()
    got = orc.e4m3_decode(codes)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan) and np.array_equal(got[~nan], want[~nan])
    assert got[0x7E] == 448.0 and got[0x08] == 2.0 ** -6 and got[0x01] == 2.0 ** -9
    g = torch.Generator().manual_seed(8)
    x = torch.randn(50000, generator=g) * torch.exp(torch.randn(50000, generator=g) * 3)
    x = x[x.abs() <= 448.0]
    ties = torch.tensor([1.0625, 1.1875, -3.25, 0.0009765625, 2.0 ** -10, 3 * 2.0 ** -10, 0.0, -0.0, 447.9, 448.0])
    x = torch.cat([x, ties])
    want_c = x.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(orc.e4m3_encode(x.numpy()), want_c)
    # saturation instead of overflow
    assert list(orc.e4m3_encode(np.array([449.0, 1e9, -1e9], np.float32))) == [0x7E, 0x7E, 0xFE]


def test_fp8_decode_equals_bf16_decode_on_values_both_formats_hold_exactly():
    """Every e4m3 value is a bf16 value, and so is its product with a power-of-two scale: decode over the codes
    must equal, bit for bit, decode over a bf16 cache holding the values the codes stand for."""
    B, Hq, Hkv, D, Lmax = 2, 4, 2, 8, 20
    g = torch.Generator().manual_seed(70)
    ck8 = torch.randint(0, 256, (B, Hkv, Lmax, D), generator=g, dtype=torch.uint8)
    cv8 = torch.randint(0, 256, (B, Hkv, Lmax, D), generator=g, dtype=torch.uint8)
    ck8[(ck8 & 0x7F) == 0x7F] = 0x10                      # no NaN codes
    cv8[(cv8 & 0x7F) == 0x7F] = 0x10
    ck8[(ck8 & 0x78) == 0x78] &= 0xB7                     # keep |k| <= 30 so that the scores stay moderate
    ks, vs = np.array([0.5, 2.0], np.float32), np.array([4.0, 0.25], np.float32)
    kv = torch.from_numpy(orc.e4m3_decode(ck8) * ks[None, :, None, None]).to(torch.bfloat16)
    vv = torch.from_numpy(orc.e4m3_decode(cv8) * vs[None, :, None, None]).to(torch.bfloat16)
    assert np.array_equal(f64(kv), orc.e4m3_decode(ck8) * ks[None, :, None, None])          # exact in bf16
    q = randn((B, Hq, D), 71, 0.25)
    lens = np.array([Lmax, 7], np.int32)
    want, want_lse = orc.decode(q, kv, vv, lens, 0.3)
    got, got_lse = orc.decode_fp8(q, ck8, cv8, lens, ks, vs, 0.3)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)
    np.testing.assert_allclose(got_lse, want_lse, rtol=0, atol=1e-13)


def test_fp8_append_quantises_by_division_and_touches_only_its_slots():
    B, T, Hkv, D, Lmax = 2, 3, 2, 8, 10
    k, v = randn((B, T, Hkv, D), 72, 3.0), randn((B, T, Hkv, D), 73, 100.0)
    ck8 = torch.full((B, Hkv, Lmax, D), 0x55, dtype=torch.uint8)
    cv8 = ck8.clone()
    ks, vs = np.array([0.37, 1.0], np.float32), np.array([0.9, 3.0], np.float32)
    gk, gv = orc.kv_append_fp8(ck8, cv8, k, v, [4, 8], [3, 3], ks, vs)      # sequence 1: third token falls off
    for b, slots in ((0, [4, 5, 6]), (1, [8, 9])):
        for t, s_ in enumerate(slots):
            for g_ in range(Hkv):
                wk = (k[b, t, g_].float() / float(ks[g_])).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
                assert np.array_equal(gk[b, g_, s_], wk)
                y = v[b, t, g_].float() / float(vs[g_])
                wv = y.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()    # the oracle saturates
                assert np.array_equal(gv[b, g_, s_], wv)
        others = [s_ for s_ in range(Lmax) if s_ not in slots]
        assert (gk[b][:, others] == 0x55).all() and (gv[b][:, others] == 0x55).all()


# --------------------------------------------------------------------------- gated linear recurrence (RG-LRU)
def _sig(z):
    return 1.0 / (1.0 + np.exp(-z))


def test_rglru_constant_gates_give_the_geometric_series():
    """With constant gate inputs a and b are constant: h_t = b (1 - a^t) / (1 - a) + a^t h_0."""
    B, T, W = 1, 50, 3
    gx_v, ga_v, x_v = 0.5, -1.0, 0.75                     # all exact in bf16
    ap = np.array([-2.0, 0.0, 1.5], np.float32)
    ones = torch.ones(B, T, W)
    y, st = orc.rglru(bf16(ones * x_v), bf16(ones * gx_v), bf16(ones * ga_v), ap, state=np.full((B, W), 0.3))
    a = np.exp(-8.0 * _sig(ga_v) * np.log1p(np.exp(ap.astype(np.float64))))
    b = np.sqrt(1 - a * a) * _sig(gx_v) * x_v
    t = np.arange(1, T + 1)[:, None]
    want = b * (1 - a ** t) / (1 - a) + a ** t * 0.3
    np.testing.assert_allclose(y[0], want, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(st[0], want[-1], rtol=1e-12)


def test_rglru_equals_the_unrolled_sum_and_brute_force():
    """h_t = sum_s (prod_{u=s+1..t} a_u) b_s + (prod_{u<=t} a_u) h_0, evaluated with cumulative products (a different
    route from the step-by-step recurrence), and a pure-Python loop on the first channel."""
    B, T, W = 2, 24, 5
    x, gx, ga = randn((B, T, W), 80), randn((B, T, W), 81), randn((B, T, W), 82)
    ap = np.linspace(-3, -1, W).astype(np.float32)        # a stays well away from 0: the division below is safe
    h0 = np.random.default_rng(0).normal(size=(B, W))
    y, st = orc.rglru(x, gx, ga, ap, state=h0)
    sp = np.log1p(np.exp(ap.astype(np.float64)))
    a = np.exp(-8.0 * _sig(f64(ga)) * sp)
    bterm = np.sqrt(1 - a * a) * _sig(f64(gx)) * f64(x)
    P = np.cumprod(a, axis=1)
    want = P * (h0[:, None, :] + np.cumsum(bterm / P, axis=1))
    np.testing.assert_allclose(y, want, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(st, want[:, -1], rtol=1e-9, atol=1e-12)
    h = h0[1, 0]
    for t in range(T):
        r = 1 / (1 + math.exp(-float(ga[1, t, 0])))
        i = 1 / (1 + math.exp(-float(gx[1, t, 0])))
        at = math.exp(-8 * r * math.log1p(math.exp(float(ap[0]))))
        h = at * h + math.sqrt(1 - at * at) * i * float(x[1, t, 0])
        assert abs(h - y[1, t, 0]) < 1e-13


def test_rglru_reset_ragged_and_chunking():
    B, T, W = 2, 30, 4
    x, gx, ga = randn((B, T, W), 83), randn((B, T, W), 84), randn((B, T, W), 85)
    ap = np.array([-1.0, 0.0, 0.5, 2.0], np.float32)
    pos = np.tile(np.arange(T, dtype=np.int32), (B, 1))
    pos[1, 12:] = np.arange(T - 12)                       # a second segment starts at t = 12 of sequence 1
    h0 = np.ones((B, W))
    y, st = orc.rglru(x, gx, ga, ap, state=h0, position=pos, seq_len=[T, 20])
    # a reset step forgets everything before it and passes the gated input through un-normalised
    np.testing.assert_allclose(y[:, 0], _sig(f64(gx))[:, 0] * f64(x)[:, 0], rtol=1e-14)
    np.testing.assert_allclose(y[1, 12], _sig(f64(gx))[1, 12] * f64(x)[1, 12], rtol=1e-14)
    y2, _ = orc.rglru(x[1:, 12:20].contiguous(), gx[1:, 12:20].contiguous(), ga[1:, 12:20].contiguous(), ap,
                      state=np.full((1, W), 123.0), position=pos[1:, 12:20])
    np.testing.assert_allclose(y[1, 12:20], y2[0], rtol=0, atol=0)
    assert np.isnan(y[1, 20:]).all()
    # the state after seq_len steps; processing in two chunks with the state carried over changes nothing
    np.testing.assert_allclose(st[1], y[1, 19], rtol=0, atol=0)
    ya, sa = orc.rglru(x[:, :11].contiguous(), gx[:, :11].contiguous(), ga[:, :11].contiguous(), ap, state=h0,
                       position=pos[:, :11])
    yb, sb = orc.rglru(x[:, 11:].contiguous(), gx[:, 11:].contiguous(), ga[:, 11:].contiguous(), ap, state=sa,
                       position=pos[:, 11:], seq_len=[T - 11, 9])
    np.testing.assert_allclose(np.concatenate([ya, yb], 1)[0], y[0], rtol=0, atol=0)
    np.testing.assert_allclose(sb, st, rtol=0, atol=0)
    # without positions there is no reset: step 0 uses the incoming state
    y3, _ = orc.rglru(x, gx, ga, ap, state=h0)
    assert not np.allclose(y3[:, 0], y[:, 0])


def test_rglru_keeps_unit_variance_for_white_inputs():
    """The sqrt(1 - a^2) factor is there so that white unit-variance inputs (gate fully open) give a state of unit
    variance whatever a is: a statistical pin of that factor."""
    B, T, W = 1, 20000, 3
    g = torch.Generator().manual_seed(86)
    x = torch.randn(B, T, W, generator=g).to(torch.bfloat16)
    gx = torch.full((B, T, W), 30.0).to(torch.bfloat16)    # sigmoid = 1 to 1e-13
    ga = torch.zeros(B, T, W).to(torch.bfloat16)           # r = 1/2
    y, _ = orc.rglru(x, gx, ga, np.array([-3.0, -1.0, 0.5], np.float32))
    var = (y[0, 2000:] ** 2).mean(axis=0)
    np.testing.assert_allclose(var, 1.0, rtol=0.12)
