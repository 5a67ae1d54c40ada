"""The device-side failure path of the tensor-core attention kernel, exercised in the one harmless way: the test
hook makes the kernel's TMA producer leave out one K/V copy and shortens the bound of every barrier wait, so the
waits that depend on that copy run out.  Nothing faults, traps or spins without a limit: every role of every CTA
gives up after a bounded number of bounded waits, the CTA waits for its copies and MMAs in flight, frees its tensor
memory and returns; the host reads HYQ_ERR_TIMEOUT from the status word and the context stays usable."""
import pytest
import torch

from gpu_util import ensure_built, rand_bf16
from paper_2608_27875_b200 import api

pytestmark = pytest.mark.gpu
HYQ_ERR_TIMEOUT = 6


def _run(Q, K, V, fmts, idx, W, status):
    (qc, qs), (kc, ks), (vc, vs) = [api.hyq_quantize_blocks(t, f) for t, f in zip((Q, K, V), fmts)]
    out = api.hyq_hybrid_attention_prefill(Q, K, V, qc, kc, vc, qs, ks, vs, fmts, idx, W, impl=api.IMPL_TCGEN05,
                                           status_word=status)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("fmts", [(0, 0, 0), (2, 2, 1)])
@pytest.mark.parametrize("drop", [0, 3, 9])
def test_a_missing_copy_ends_in_a_timeout_status_and_the_next_call_is_fine(fmts, drop):
    ensure_built()
    B, Hq, Hkv, L, W, k = 1, 4, 2, 2048, 128, 32
    Q, K, V = (rand_bf16((B, h, L, 128), seed=900 + n).cuda() for n, h in enumerate((Hq, Hkv, Hkv)))
    idx = api.hyq_select_vertical(Q, K, W, k)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    good = _run(Q, K, V, fmts, idx, W, status)
    assert int(status.item()) == 0
    try:
        api.hyq_test_set_attention_hooks(wait_limit_clocks=200_000, drop_load_position=drop)     # ~0.1 ms per wait
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        _run(Q, K, V, fmts, idx, W, status)
        t1.record()
        torch.cuda.synchronize()
        assert int(status.item()) == HYQ_ERR_TIMEOUT
        assert api.status_string(HYQ_ERR_TIMEOUT) == "bounded device wait expired"
        assert t0.elapsed_time(t1) < 2000.0          # a handful of bounded waits per CTA, not seconds
    finally:
        api.hyq_test_set_attention_hooks(0, -1)
    # the context is intact: the same call, without the hook, gives the same result as before
    status.zero_()
    again = _run(Q, K, V, fmts, idx, W, status)
    assert int(status.item()) == 0
    assert torch.equal(again, good)


def test_hook_arguments_are_checked():
    lib = ensure_built()
    assert lib.hyq_test_set_attention_hooks(-1, -1) == 1
    assert lib.hyq_test_set_attention_hooks(0, -2) == 1
    assert lib.hyq_test_set_attention_hooks(0, -1) == 0
