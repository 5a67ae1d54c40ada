"""GPU check of hyq_select_vertical_static, the selection entry point that brings its own scratch
memory for callers that cannot allocate any (a process whose memory pool already owns the GPU, a
latency-critical loop that must not trigger cudaMalloc).  It has to return exactly what
hyq_select_vertical returns, call after call, although every call reuses the same built-in array.
Collected last on purpose: a failure here must not hide the result of any other test."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from gpu_util import ensure_built, rand_bf16
from paper_2608_27875_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu


def _both(Q, K, window, k, n_tail=0):
    """Index sets from the workspace entry point and from the built-in-scratch entry point (raw C-ABI calls)."""
    lib = ensure_built()
    B, Hq, L, D = Q.shape
    Hkv = K.shape[1]
    need = ctypes.c_size_t(0)
    assert lib.hyq_select_vertical_workspace(B, Hq, Hkv, L, L, D, window, k, ctypes.byref(need)) == 0
    ws = torch.empty(need.value, dtype=torch.uint8, device="cuda")
    ref = torch.full((B, Hq, k), -1, dtype=torch.int32, device="cuda")
    got = torch.full((B, Hq, k), -2, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    assert lib.hyq_select_vertical(Q.data_ptr(), K.data_ptr(), B, Hq, Hkv, L, L, D, window, n_tail, k,
                                   ref.data_ptr(), ws.data_ptr(), ws.numel(), stream) == 0
    assert lib.hyq_select_vertical_static(Q.data_ptr(), K.data_ptr(), B, Hq, Hkv, L, L, D, window, n_tail, k,
                                          got.data_ptr(), stream) == 0
    torch.cuda.synchronize()
    return ref.cpu().numpy(), got.cpu().numpy()


def test_static_scratch_matches_workspace_entry_point_on_consecutive_calls():
    # two different problems back to back: the second call finds the first one's leftovers in the array
    cases = [((1, 8, 2, 3000), 256, 55), ((2, 4, 4, 700), 64, 9), ((1, 8, 2, 3000), 256, 55)]
    for n, ((B, Hq, Hkv, L), window, k) in enumerate(cases):
        Q = rand_bf16((B, Hq, L, 128), seed=100 + n).cuda()
        K = rand_bf16((B, Hkv, L, 128), seed=200 + n).cuda()
        ref, got = _both(Q, K, window, k)
        np.testing.assert_array_equal(got, ref)       # index sets are integers: equality, no tolerance
        assert (np.diff(got, axis=-1) > 0).all() and got.min() >= 0 and got.max() < L - window
        np.testing.assert_array_equal(got, oracle.select_vertical(wl.bits(Q.cpu()), wl.bits(K.cpu()), window, k))


def test_static_scratch_call_leaves_the_free_device_memory_unchanged():
    """The point of the entry point: with the output preallocated, a call (after the first one on the device,
    which looks up the array's address) takes nothing from the device's free memory and gives nothing back."""
    lib = ensure_built()
    B, Hq, Hkv, L, window, k = 1, 8, 2, 3000, 256, 55
    Q, K = rand_bf16((B, Hq, L, 128), seed=300).cuda(), rand_bf16((B, Hkv, L, 128), seed=301).cuda()
    out = torch.empty(B, Hq, k, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    call = lambda: lib.hyq_select_vertical_static(Q.data_ptr(), K.data_ptr(), B, Hq, Hkv, L, L, 128, window, 0, k,   # noqa: E731
                                                  out.data_ptr(), stream)
    assert call() == 0
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    assert call() == 0
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    np.testing.assert_array_equal(out.cpu().numpy(), oracle.select_vertical(wl.bits(Q.cpu()), wl.bits(K.cpu()), window, k))


def test_static_scratch_rejects_problems_beyond_its_fixed_size():
    lib = ensure_built()
    # 64 query heads x (70000 + 128) scores x 8 bytes > 8 MiB: refused on the host, before any launch
    rc = lib.hyq_select_vertical_static(0x1000, 0x2000, 1, 64, 8, 70256, 70256, 128, 256, 0, 100, 0x3000, None)
    assert rc == 3 and api.status_string(rc) == "workspace too small"
    # an empty problem needs no scratch at all
    assert lib.hyq_select_vertical_static(None, None, 1, 4, 2, 64, 64, 128, 64, 0, 8, None, None) == 0
