"""l4l_kv_append must be an exact copy that touches nothing else (compared with the oracle's copy)."""
import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, bits_equal

pytestmark = pytest.mark.gpu


def rawbits(shape, g):
    return torch.randint(0, 65536, shape, generator=g, dtype=torch.int32).to(torch.int16).view(torch.bfloat16)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("token_major_cache", [False, True])
def test_append_bit_exact_ragged(D, token_major_cache):
    B, T, Hkv, Lmax = 5, 7, 3, 40
    g = torch.Generator().manual_seed(21 + D)
    ck, cv = rawbits((B, Hkv, Lmax, D), g), rawbits((B, Hkv, Lmax, D), g)
    kn, vn = rawbits((B, T, Hkv, D), g), rawbits((B, T, Hkv, D), g)
    pos = torch.tensor([0, 33, 12, 39, 5], dtype=torch.int32)
    n_new = torch.tensor([7, 7, 0, 1, 3], dtype=torch.int32)
    ek, ev = orc.kv_append(ck, cv, kn, vn, pos.numpy(), n_new.numpy())
    if token_major_cache:
        gk, gv = Guarded(ck.permute(0, 2, 1, 3).contiguous()), Guarded(cv.permute(0, 2, 1, 3).contiguous())
        dk, dv = gk.t.permute(0, 2, 1, 3), gv.t.permute(0, 2, 1, 3)
    else:
        gk, gv = Guarded(ck), Guarded(cv)
        dk, dv = gk.t, gv.t
    gkn, gvn = Guarded(kn), Guarded(vn)
    l4l.l4l_kv_append(dk, dv, gkn.t, gvn.t, pos.cuda(), n_new.cuda())
    torch.cuda.synchronize()
    assert bits_equal(dk.contiguous(), ek) and bits_equal(dv.contiguous(), ev)
    assert gk.margins_intact() and gv.margins_intact() and gkn.margins_intact() and gvn.margins_intact()


def test_append_out_of_range_slots_are_dropped_not_written():
    B, T, Hkv, D, Lmax = 2, 4, 2, 64, 8
    g = torch.Generator().manual_seed(23)
    ck, cv = rawbits((B, Hkv, Lmax, D), g), rawbits((B, Hkv, Lmax, D), g)
    kn, vn = rawbits((B, T, Hkv, D), g), rawbits((B, T, Hkv, D), g)
    gk, gv = Guarded(ck), Guarded(cv)
    pos = torch.tensor([6, -2], dtype=torch.int32)      # slots 6,7 valid, 8,9 dropped; -2,-1 dropped, 0,1 valid
    l4l.l4l_kv_append(gk.t, gv.t, kn.cuda(), vn.cuda(), pos.cuda())
    torch.cuda.synchronize()
    assert gk.margins_intact() and gv.margins_intact()
    ek, ev = ck.clone(), cv.clone()
    ek[0, :, 6:8], ev[0, :, 6:8] = kn[0, 0:2].transpose(0, 1), vn[0, 0:2].transpose(0, 1)
    ek[1, :, 0:2], ev[1, :, 0:2] = kn[1, 2:4].transpose(0, 1), vn[1, 2:4].transpose(0, 1)
    assert bits_equal(gk.t, ek) and bits_equal(gv.t, ev)
