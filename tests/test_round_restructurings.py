"""The two restructurings the whole-round entry points apply, checked on the CPU against the oracle's step-by-step
recurrences (Eq. parle_y, parle_z): they must be identities, not approximations.

1. z is touched every other inner step: z_{k+2} = alpha^2 z_k + (1 - alpha)(alpha y_{k+1} + y_{k+2}), with the
   schedule first step / (skip, two-step) pairs / one closing one-step update when L is even.
2. y is held as two 16-bit planes, the halves of (fp32 word + 0x8000): the upper one is y rounded to bf16 (nearest,
   ties away from zero), and ((upper << 16) | lower) - 0x8000 is the word again."""
import numpy as np
import pytest
import torch

from oracle import parle_oracle as po


def z_modes(L):
    """Mirror of the library's schedule: 0 = one-step, 1 = z untouched, 2 = two-step (first step: z formed from x)."""
    out = [0]
    rest = L - 1
    for idx in range(rest):
        if rest % 2 and idx == rest - 1:
            out.append(0)
        else:
            out.append(2 if idx % 2 else 1)
    return out


@pytest.mark.parametrize("L", [1, 2, 3, 4, 5, 6, 25])
def test_paired_z_schedule_reproduces_the_step_by_step_z(L):
    rng = np.random.default_rng(L)
    hp = po.Hyper(0.1, 0.1, 0.75, 2.0, 0.5)
    x = rng.standard_normal(64)
    lam = rng.uniform(0.1, 2.0, 64)
    y = x.copy(); z = x.copy()                      # oracle: reset, then L one-step updates
    ys = []
    for _ in range(L):
        y, z = po.inner_step(y, z, x, lam * y, hp)
        ys.append(y)
    zp = x.copy(); y_prev = x.copy()                # restructured: same y, z by the schedule
    for mode, y_new in zip(z_modes(L), ys):
        if mode == 0:
            zp = hp.alpha * zp + (1 - hp.alpha) * y_new
        elif mode == 2:
            zp = hp.alpha ** 2 * zp + (1 - hp.alpha) * (hp.alpha * y_prev + y_new)
        y_prev = y_new
    assert z_modes(L).count(1) == (L - 1) // 2
    np.testing.assert_allclose(zp, z, rtol=1e-14, atol=0)


def encode_planes(y):
    w = (y.view(np.uint32).astype(np.uint64) + 0x8000) & 0xFFFFFFFF
    return (w >> 16).astype(np.uint32), (w & 0xFFFF).astype(np.uint32)


def decode_planes(hi, lo):
    return ((((hi.astype(np.uint64) << 16) | lo) - 0x8000) & 0xFFFFFFFF).astype(np.uint32).view(np.float32)


def test_two_plane_y_round_trips_exactly_and_its_upper_plane_is_the_nearest_bf16():
    rng = np.random.default_rng(7)
    y = rng.standard_normal(1 << 20).astype(np.float32) * np.float32(0.05)
    bits = y.view(np.uint32).copy()
    bits[:4096] = (bits[:4096] & 0xFFFF0000) | 0x8000          # ties, half of them under an odd upper half
    bits[4096:8192] |= 0xFFFF                                   # rounds up with carry into the upper half
    bits[8192:8200] = [0, 0x80000000, 0x00008000, 0x00018000, 0x3F7FFFFF, 0xBF7F8000, 0x00000001, 0x7F000000]
    y = bits.view(np.float32)
    hi, lo = encode_planes(y)
    assert np.array_equal(decode_planes(hi, lo).view(np.uint32), bits)           # exact, ties included
    # the upper plane against the definition of rounding to the nearest bf16, worked out in fp64:
    # the two neighbours are the truncated word and the next one up in magnitude; ties go to the larger magnitude
    down = (bits & 0xFFFF0000).view(np.float32).astype(np.float64)
    up = ((bits & 0xFFFF0000) + 0x10000).astype(np.uint32).view(np.float32).astype(np.float64)
    v = y.astype(np.float64)
    want = np.where(np.abs(v - down) < np.abs(up - v), down, up)
    got = (hi << 16).astype(np.uint32).view(np.float32).astype(np.float64)
    assert np.array_equal(got, want)
    # it differs from torch's ties-to-even conversion on ties under an even upper half only
    rne = torch.from_numpy(y.copy()).to(torch.bfloat16).view(torch.int16).numpy().astype(np.uint32) & 0xFFFF
    differ = rne != hi
    tie_even = ((bits & 0xFFFF) == 0x8000) & ((bits >> 16) & 1 == 0)
    assert np.array_equal(differ, tie_even) and differ.sum() > 1000
