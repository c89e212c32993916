"""Shared helpers of the GPU parity tests: guard-banded device buffers and the tolerance check."""
import numpy as np
import torch

MAX_ABS_TOL = 2e-2    # bf16 output vs fp64 oracle, stated by the benchmark spec
MEAN_ABS_TOL = 2e-3
NAN_BITS = 0x7FC0
GUARD_ELEMS = 4096


class Guarded:
    """A device copy of `t` with NaN-filled margins on both sides. An over-read that reaches the
    math poisons the result; `margins_intact()` shows an out-of-bounds write."""

    def __init__(self, t: torch.Tensor, fill_bits: int = NAN_BITS):
        assert t.is_contiguous()
        n = t.numel()
        if t.dtype == torch.bfloat16:
            buf = torch.full((n + 2 * GUARD_ELEMS,), fill_bits, dtype=torch.int16, device="cuda").view(torch.bfloat16)
        elif t.dtype == torch.float32:
            buf = torch.full((n + 2 * GUARD_ELEMS,), float("nan"), dtype=torch.float32, device="cuda")
        elif t.dtype == torch.uint8:                       # fp8 codes: 0x7F is the e4m3 NaN
            buf = torch.full((n + 2 * GUARD_ELEMS,), 0x7F, dtype=torch.uint8, device="cuda")
        else:
            raise TypeError(t.dtype)
        self.buf = buf
        self.t = buf[GUARD_ELEMS:GUARD_ELEMS + n].view(t.shape)
        self.t.copy_(t)
        self._ref = buf.clone()

    def margins_intact(self) -> bool:
        if self.buf.dtype == torch.uint8:
            a = self.buf
        else:
            a = self.buf.view(torch.int16) if self.buf.dtype == torch.bfloat16 else self.buf.view(torch.int32)
        b = self._ref.view(a.dtype)
        return bool(torch.equal(a[:GUARD_ELEMS], b[:GUARD_ELEMS]) and torch.equal(a[-GUARD_ELEMS:], b[-GUARD_ELEMS:]))


def nan_bf16(shape, device="cpu"):
    return torch.full(shape, NAN_BITS, dtype=torch.int16, device=device).view(torch.bfloat16)


def assert_close_to_oracle(gpu: torch.Tensor, ref: np.ndarray, what: str = ""):
    got = gpu.detach().float().cpu().double().numpy()
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values in the GPU output"
    err = np.abs(got - ref)
    assert err.max() <= MAX_ABS_TOL, f"{what}: max-abs error {err.max():.4g} > {MAX_ABS_TOL}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean-abs error {err.mean():.4g} > {MEAN_ABS_TOL}"
    return float(err.max()), float(err.mean())


def bits_equal(a: torch.Tensor, b) -> bool:
    a16 = a.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    if isinstance(b, torch.Tensor):
        b = b.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    return bool(np.array_equal(a16, b))
