"""Pins for the oracle's per-tile quantizer (Algorithm 2, Stage 2; c_B = 127 / 448).

The oracle is held against torch's CPU casts and rounding (library routines the
oracle does not call) and against invariants that the definition fixes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_27875_b200 import workloads as wl

C = {oracle.FMT_INT8: 127.0, oracle.FMT_FP8_E4M3: 448.0, oracle.FMT_INT4: 7.0}


def _x(B=2, H=3, L=150, D=32, seed=0, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(B, H, L, D, generator=g) * scale).to(torch.bfloat16)


def _unpack_int4(codes):
    lo = (codes & 0xF).astype(np.int16)
    hi = (codes >> 4).astype(np.int16)
    lo[lo >= 8] -= 16
    hi[hi >= 8] -= 16
    out = np.empty(codes.shape[:-1] + (codes.shape[-1] * 2,), dtype=np.int16)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


def _torch_reference(x, fmt, bt):
    """Same definition through torch CPU ops: blockwise amax, fp32 divide,
    fp32 multiply, torch.round (half to even) / float8 cast."""
    B, H, L, D = x.shape
    nb = -(-L // bt)
    xf = x.float()
    pad = nb * bt - L
    xp = torch.nn.functional.pad(xf, (0, 0, 0, pad))
    amax = xp.reshape(B, H, nb, bt * D).abs().amax(-1)
    c = torch.tensor(C[fmt], dtype=torch.float32)
    scale = amax / c
    inv = c / amax
    y = xp.reshape(B, H, nb, bt, D) * inv[..., None, None]
    y = y.reshape(B, H, nb * bt, D)[:, :, :L]
    if fmt == oracle.FMT_FP8_E4M3:
        codes = y.clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    else:
        codes = torch.round(y).clamp(-C[fmt], C[fmt]).to(torch.int16).numpy()
    return codes, scale.numpy()


def test_e4m3_decode_matches_library_for_every_byte():
    b = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(b.copy()).view(torch.float8_e4m3fn).double().numpy()
    ok = ~np.isnan(ref)                       # 0x7F / 0xFF are NaN and never produced
    assert ok.sum() == 254
    np.testing.assert_array_equal(oracle.e4m3_decode(b)[ok], ref[ok])


def test_e4m3_encode_matches_library_cast():
    rng = np.random.default_rng(0)
    # dense sweep of the representable range + exact ties + subnormals + saturation edge
    ys = [rng.standard_normal(200000).astype(np.float32) * s for s in (1e-3, 0.02, 1, 30, 200)]
    grid = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()
    grid = np.sort(grid[~np.isnan(grid)])
    mids = ((grid[:-1].astype(np.float64) + grid[1:]) / 2).astype(np.float32)   # exact half-way points
    ys += [grid, mids, np.nextafter(mids, np.float32(1e9)), np.nextafter(mids, np.float32(-1e9)),
           np.array([0.0, -0.0, 448.0, -448.0, 447.9, 463.9, 2**-9, 2**-10, 2**-10 * 1.0001, 1e-30],
                    dtype=np.float32)]
    y = np.concatenate(ys).astype(np.float32)
    y = y[np.abs(y) <= 464.0]     # the library cast turns |y| >= 464 into NaN; the oracle saturates instead
    ref = torch.from_numpy(y.copy()).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    np.testing.assert_array_equal(oracle.e4m3_encode(y), ref)
    # saturation beyond the library's NaN threshold
    big = np.array([464.0, 1e4, -1e4, np.float32(3e38)], dtype=np.float32)
    np.testing.assert_array_equal(oracle.e4m3_encode(big), np.array([0x7E, 0x7E, 0xFE, 0x7E], dtype=np.uint8))


@pytest.mark.parametrize("fmt", [oracle.FMT_INT8, oracle.FMT_FP8_E4M3, oracle.FMT_INT4])
@pytest.mark.parametrize("L", [64, 150, 1])
def test_matches_torch_cpu_ops(fmt, L):
    x = _x(L=L, seed=L + fmt)
    codes, scales = oracle.quantize(wl.bits(x), fmt, 64)
    ref_codes, ref_scales = _torch_reference(x, fmt, 64)
    np.testing.assert_array_equal(scales, ref_scales)
    if fmt == oracle.FMT_INT8:
        np.testing.assert_array_equal(codes.view(np.int8).astype(np.int16), ref_codes)
    elif fmt == oracle.FMT_INT4:
        np.testing.assert_array_equal(_unpack_int4(codes), ref_codes)
    else:
        np.testing.assert_array_equal(codes, ref_codes)


@pytest.mark.parametrize("fmt", [oracle.FMT_INT8, oracle.FMT_FP8_E4M3, oracle.FMT_INT4])
def test_invariants(fmt):
    bt = 64
    x = _x(B=1, H=2, L=200, D=128, seed=3)
    codes, scales = oracle.quantize(wl.bits(x), fmt, bt)
    xf = x.double().numpy()
    if fmt == oracle.FMT_INT8:
        val = codes.view(np.int8).astype(np.float64)
    elif fmt == oracle.FMT_INT4:
        val = _unpack_int4(codes).astype(np.float64)
    else:
        val = oracle.e4m3_decode(codes)
    sc = np.repeat(scales.astype(np.float64), bt, axis=2)[:, :, :200, None]
    # every non-zero block reaches the top code; nothing exceeds it
    for n in range(scales.shape[2]):
        blk = np.abs(val[:, :, n * bt:(n + 1) * bt]).reshape(1, 2, -1).max(-1)
        np.testing.assert_array_equal(blk, C[fmt])
    # reconstruction error bound of a uniform grid (integers): half a step (+ fp32 slack)
    err = np.abs(xf - val * sc)
    if fmt != oracle.FMT_FP8_E4M3:
        assert (err <= sc * (0.5 + C[fmt] * 2.0 ** -22)).all()
    else:   # e4m3: relative half-ulp 2^-4 of the value's binade, absolute 2^-10 in the subnormal range
        assert (err <= np.maximum(np.abs(xf) * 2.0 ** -4 * 1.0001, sc * 2.0 ** -10 * 1.0001)).all()
    # odd symmetry: q(-x) = -q(x)
    codes_n, scales_n = oracle.quantize(wl.bits(-x), fmt, bt)
    np.testing.assert_array_equal(scales_n, scales)
    if fmt == oracle.FMT_INT8:
        np.testing.assert_array_equal(codes_n.view(np.int8), -codes.view(np.int8))
    elif fmt == oracle.FMT_INT4:
        np.testing.assert_array_equal(_unpack_int4(codes_n), -_unpack_int4(codes))
    else:
        np.testing.assert_array_equal(codes_n, codes ^ 0x80)
    # power-of-two scaling: same codes, doubled scale
    codes_2, scales_2 = oracle.quantize(wl.bits(x * 2), fmt, bt)
    np.testing.assert_array_equal(codes_2, codes)
    np.testing.assert_array_equal(scales_2, scales * 2)


def test_zero_block_and_packing():
    x = torch.zeros(1, 1, 70, 4, dtype=torch.bfloat16)
    x[0, 0, 64] = torch.tensor([7.0, -7.0, 1.0, -2.0])       # second block: scale 1, codes are the values
    codes, scales = oracle.quantize(wl.bits(x), oracle.FMT_INT4, 64)
    assert scales[0, 0, 0] == 0.0 and scales[0, 0, 1] == 1.0
    assert not codes[0, 0, :64].any()
    # even channel in the low nibble, two's complement
    np.testing.assert_array_equal(codes[0, 0, 64], np.array([0x7 | (0x9 << 4), 0x1 | (0xE << 4)], dtype=np.uint8))
    codes8, scales8 = oracle.quantize(wl.bits(x), oracle.FMT_INT8, 64)
    assert scales8[0, 0, 0] == 0.0 and not codes8[0, 0, :64].any()
    np.testing.assert_array_equal(codes8[0, 0, 64].view(np.int8), np.array([127, -127, 18, -36], dtype=np.int8))


def test_round_half_to_even_in_the_code():
    # block absmax 127 -> inv = 1: codes are rint(x) with ties to even
    x = torch.tensor([127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5], dtype=torch.bfloat16).reshape(1, 1, 1, 8)
    codes, scales = oracle.quantize(wl.bits(x), oracle.FMT_INT8, 64)
    assert scales[0, 0, 0] == 1.0
    np.testing.assert_array_equal(codes.view(np.int8).ravel(), np.array([127, 0, 2, 2, 0, -2, -2, 4], dtype=np.int8))
