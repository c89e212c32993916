"""l4l_rglru_scan (gated linear recurrence of the RecurrentGemma block) against the fp64 oracle.

Tolerance. y is rounded to bf16 (2^-9 relative) and the kernel uses hardware approximations (tanh.approx for the two
sigmoids: ~2.5e-4 absolute each; ex2.approx). An error d in the recurrence gate changes ln a by 8 softplus(a_param) d;
over the state's memory horizon (about 1 / |ln a| steps) that accumulates to a relative error of about d / r in the
carried state, i.e. below 1e-3 unless the gate is nearly closed. For the O(1) data used here the attention tolerances
(max-abs 2e-2, mean-abs 2e-3) hold with margin and are asserted tighter: max-abs 1e-2, mean-abs 1.5e-3."""
import numpy as np
import pytest
import torch

from oracle import l4l_oracle as orc
from paper_2608_21836_b200 import binding as l4l
from helpers import Guarded, nan_bf16

pytestmark = pytest.mark.gpu
SENTINEL = 0x4D4D


def make(B, T, W, seed):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(B, T, W, generator=g).to(torch.bfloat16)
    gx = (torch.randn(B, T, W, generator=g) * 2).to(torch.bfloat16)
    ga = (torch.randn(B, T, W, generator=g) * 2).to(torch.bfloat16)
    # a^8-style initialisation: a at r = 1 between 0.9 and 0.999  ->  softplus(a_param) = -ln(a) / 8
    a_max = torch.rand(W, generator=g) * 0.099 + 0.9
    sp = -torch.log(a_max) / 8
    a_param = torch.log(torch.expm1(sp))
    h0 = torch.randn(B, W, generator=g)
    return x, gx, ga, a_param.float(), h0.float()


def check(y_gpu, st_gpu, y_ref, st_ref, valid):
    got = y_gpu.float().cpu().double().numpy()
    err = np.abs(got - y_ref)[valid]
    assert np.isfinite(got[valid]).all()
    assert err.max() <= 1e-2, f"max-abs {err.max():.3g}"
    assert err.mean() <= 1.5e-3, f"mean-abs {err.mean():.3g}"
    assert torch.isfinite(st_gpu).all()
    serr = np.abs(st_gpu.cpu().double().numpy() - st_ref)
    assert serr.max() <= 5e-3, f"state max-abs {serr.max():.3g}"


@pytest.mark.parametrize("B,T,W", [(2, 300, 2560), (1, 1237, 200), (3, 65, 40), (1, 1, 64), (5, 1000, 96), (1, 16, 64), (2, 17, 128),
                                   (4, 300, 2560), (4, 600, 2560), (5, 520, 2440), (19, 530, 512)])
def test_rglru_matches_oracle(B, T, W):
    """Sequences of many tiles (eight warps hand the state on from tile to tile), of exactly one tile (the one-warp
    variant) and just past it; a second segment inside a sequence, ragged lengths, a channel count that does not fill
    the last strip; launches of 149 to 200 strips, which the library cuts into 32- or 16-channel strips (a warp
    then owns two or four consecutive time tiles)."""
    if (B, W) in ((4, 2560), (5, 2440), (19, 512)):                    # 160, 195 and 152 strips at 64 channels
        assert l4l.l4l_rglru_strip_channels(B, T, W) in (16, 32)
        assert l4l.l4l_rglru_strip_channels(4, 600, 2560) == 16 and l4l.l4l_rglru_strip_channels(4, 300, 2560) == 32
    x, gx, ga, ap, h0 = make(B, T, W, 1100 + T)
    pos = torch.arange(T, dtype=torch.int32).repeat(B, 1)
    if T > 40:
        pos[0, 37:] = torch.arange(T - 37, dtype=torch.int32)        # a second segment inside sequence 0
    lens = [T] + [max(1, T - 7 * i) for i in range(1, B)]
    # rows past a sequence's length are caller memory that may hold anything: NaN there must reach neither y nor the state
    dead = torch.arange(T).view(1, T, 1) >= torch.tensor(lens).view(B, 1, 1)
    nan = nan_bf16((1,))
    x, gx, ga = torch.where(dead, nan, x), torch.where(dead, nan, gx), torch.where(dead, nan, ga)
    y_ref, st_ref = orc.rglru(x, gx, ga, ap.numpy(), state=h0.double().numpy(), position=pos.numpy(), seq_len=lens)
    gy = Guarded(torch.full((B, T, W), SENTINEL, dtype=torch.int16).view(torch.bfloat16))
    gs = Guarded(h0)
    ws = l4l.new_rglru_workspace(B, T, W)
    l4l.l4l_rglru_scan(x.cuda(), gx.cuda(), ga.cuda(), ap.cuda(), gs.t, gy.t, ws, position=pos.cuda(),
                       seq_lens=torch.tensor(lens, dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    assert gy.margins_intact() and gs.margins_intact()
    valid = np.arange(T)[None, :, None] < np.array(lens)[:, None, None]
    valid = np.broadcast_to(valid, (B, T, W))
    check(gy.t, gs.t, y_ref, st_ref, valid)
    assert (gy.t.cpu().view(torch.int16).numpy()[~valid] == SENTINEL).all()          # rows past seq_len untouched


def test_rglru_chunks_carry_the_state():
    """A prompt of 200 steps, then single steps (the decode regime): same as one pass over all of it."""
    B, T, W = 2, 205, 128
    x, gx, ga, ap, h0 = make(B, T, W, 7)
    y_ref, st_ref = orc.rglru(x, gx, ga, ap.numpy(), state=np.zeros((B, W)),
                              position=np.tile(np.arange(T, dtype=np.int32), (B, 1)))
    dx, dgx, dga, dap = x.cuda(), gx.cuda(), ga.cuda(), ap.cuda()
    state = torch.zeros(B, W, device="cuda")
    y = torch.zeros(B, T, W, dtype=torch.bfloat16, device="cuda")
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, 1, 1, 1, 64, 1)
    pos = torch.arange(200, dtype=torch.int32, device="cuda").repeat(B, 1)
    y0 = torch.zeros(B, 200, W, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_rglru_scan(dx[:, :200].contiguous(), dgx[:, :200].contiguous(), dga[:, :200].contiguous(), dap, state, y0, ws,
                       position=pos)
    y[:, :200] = y0
    for t in range(200, T):
        y1 = torch.zeros(B, 1, W, dtype=torch.bfloat16, device="cuda")
        l4l.l4l_rglru_scan(dx[:, t:t + 1].contiguous(), dgx[:, t:t + 1].contiguous(), dga[:, t:t + 1].contiguous(), dap,
                           state, y1, ws)
        y[:, t] = y1[:, 0]
    torch.cuda.synchronize()
    assert l4l.l4l_last_device_error(ws) == 0
    check(y, state, y_ref, st_ref, np.ones((B, T, W), bool))


def test_rglru_rejects_bad_shapes():
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, 1, 1, 1, 64, 1)
    x = torch.zeros(1, 4, 12, dtype=torch.bfloat16, device="cuda")                  # W not a multiple of 8
    with pytest.raises(l4l.L4LError):
        l4l.l4l_rglru_scan(x, x.clone(), x.clone(), torch.zeros(12, device="cuda"), torch.zeros(1, 12, device="cuda"),
                           x.clone(), ws)


def test_rglru_empty_inputs_are_a_no_op():
    ws = l4l.new_workspace(l4l.L4L_OP_PREFILL, 1, 1, 1, 64, 1)
    state = torch.full((2, 64), 7.0, device="cuda")
    e = torch.zeros(2, 0, 64, dtype=torch.bfloat16, device="cuda")
    l4l.l4l_rglru_scan(e, e.clone(), e.clone(), torch.zeros(64, device="cuda"), state, e.clone(), ws)
    # all sequences of length 0: the state comes back unchanged
    x = torch.randn(2, 8, 64, device="cuda").to(torch.bfloat16)
    y = torch.full((2, 8, 64), 3.0, device="cuda").to(torch.bfloat16)
    l4l.l4l_rglru_scan(x, x.clone(), x.clone(), torch.zeros(64, device="cuda"), state, y, ws,
                       seq_lens=torch.zeros(2, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert (state == 7.0).all() and (y == 3.0).all() and l4l.l4l_last_device_error(ws) == 0
