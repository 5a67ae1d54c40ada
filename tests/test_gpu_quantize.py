"""GPU parity: hyq_quantize_blocks against the oracle, bit for bit (codes and fp32 scales)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import ensure_built, rand_bf16
from paper_2608_27875_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
FMTS = [wl.FMT_INT8, wl.FMT_FP8_E4M3, wl.FMT_INT4]


def _check(x, fmt, bt=64):
    ensure_built()
    codes, scales = api.hyq_quantize_blocks(x.cuda(), fmt, bt)
    torch.cuda.synchronize()
    ref_codes, ref_scales = oracle.quantize(wl.bits(x), fmt, bt)
    np.testing.assert_array_equal(scales.cpu().numpy().view(np.uint32), ref_scales.view(np.uint32))
    np.testing.assert_array_equal(codes.cpu().numpy(), ref_codes)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("shape", [(1, 2, 2048, 128), (2, 3, 1000, 128), (1, 1, 1, 128), (1, 5, 63, 128), (1, 2, 65, 128)])
def test_matches_oracle(fmt, shape):
    _check(rand_bf16(shape, seed=sum(shape) + fmt), fmt)


@pytest.mark.parametrize("bt", [32, 128])
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("shape", [(1, 2, 2048, 128), (2, 3, 1000, 128), (1, 1, 1, 128), (1, 5, 127, 128), (1, 2, 129, 128)])
def test_other_block_sizes_match_oracle(fmt, shape, bt):
    _check(rand_bf16(shape, seed=sum(shape) + fmt + bt), fmt, bt)


@pytest.mark.parametrize("fmt", FMTS)
def test_value_ranges_and_degenerate_tiles(fmt):
    x = rand_bf16((1, 4, 320, 128), seed=5)
    x[0, 0] *= 1e-3                     # tiny values
    x[0, 1] *= 3e4                      # large values
    x[0, 2, 64:128] = 0                 # an all-zero tile
    x[0, 2, 128:192] = -0.0
    x[0, 3, :, 7] *= 50                 # outlier channel
    x[0, 3, 200] = 1e-38                # subnormal-range bf16 values
    _check(x, fmt)


@pytest.mark.parametrize("fmt", FMTS)
def test_exact_ties_round_to_even(fmt):
    # tile absmax = c makes inv = 1: values k + 0.5 are exact ties
    c = {wl.FMT_INT8: 127.0, wl.FMT_FP8_E4M3: 448.0, wl.FMT_INT4: 7.0}[fmt]
    x = torch.zeros(1, 1, 64, 128)
    x[0, 0, 0, 0] = c
    ties = torch.arange(-6.5, 7.0, 1.0)
    x[0, 0, 1, : len(ties)] = ties
    x[0, 0, 2, :8] = torch.tensor([17.0, 18.0, 19.0, 21.0, 22.0, 23.0, 25.0, 27.0])   # e4m3 ties at step 2/4
    x[0, 0, 3, :6] = torch.tensor([0.0009765625, 0.0029296875, 0.001953125, 0.00390625, 2.0 ** -11, 3 * 2.0 ** -11])
    _check(x.to(torch.bfloat16), fmt)


@pytest.mark.parametrize("name", ["c0", "c1"])
def test_workload_tensors(name):
    w = wl.CONFIGS[name]
    Q, K, V = wl.make_inputs(w, heads=[0, w.Hkv - 1])
    for t, fmt in zip((Q, K, V), w.fmts):
        _check(t, fmt)
    _check(K, wl.FMT_INT4)
    _check(V, wl.FMT_FP8_E4M3)
