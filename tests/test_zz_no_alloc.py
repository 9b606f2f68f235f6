"""The pooler + head entry point for callers that cannot allocate device memory
(mt_kernel_pooler_head_static) must give what mt_kernel_pooler_head gives with a
caller-provided scratch buffer.  Collected last on purpose: a run that stops at the
first failure has then already gone through every other test."""
import numpy as np
import pytest
import torch

from paper_2107_05377_b200 import binding as mt
from gpu_util import rand_bf16, to_dev_bf16

pytestmark = pytest.mark.gpu


def _inputs(B, S, H, C, tag):
    hb, _ = rand_bf16(61, f"h{tag}", (B * S, H), 1.0)
    pwb, _ = rand_bf16(62, f"pw{tag}", (H, H), 0.05)
    pbb, _ = rand_bf16(63, f"pb{tag}", (H,), 0.1)
    cwb, _ = rand_bf16(64, f"cw{tag}", (C, H), 0.05)
    cbb, _ = rand_bf16(65, f"cb{tag}", (C,), 0.1)
    return [to_dev_bf16(a) for a in (hb, pwb, pbb, cwb, cbb)]


def test_static_scratch_entry_matches_the_scratch_argument_entry_twice_in_a_row():
    # two calls in a row with different shapes: the second one finds the first one's features in the
    # shared array and must not be disturbed by them
    for B, S, H, C in ((32, 128, 768, 3), (9, 16, 1024, 1)):
        args = _inputs(B, S, H, C, f"{B}.{H}")
        want = torch.full((B, C + 2), -5.0, dtype=torch.float32, device="cuda")
        scratch = torch.empty(B, H, dtype=torch.float32, device="cuda")
        mt.mt_kernel_pooler_head(*args, scratch, want, B, S, col0=1)
        got = torch.full((B, C + 2), -5.0, dtype=torch.float32, device="cuda")
        mt.mt_kernel_pooler_head_static(*args, got, B, S, col0=1)
        torch.cuda.synchronize()
        assert float((got - want).abs().max()) <= 1e-4      # the tolerance of the pooler/head parity test
        assert torch.equal(got, want)                        # same kernels, same order: in fact identical
        assert torch.all(got[:, 0] == -5.0) and torch.all(got[:, C + 1] == -5.0)


def test_static_scratch_entry_rejects_what_does_not_fit():
    B, S, H, C = 4, 8, 768, 2
    args = _inputs(B, S, H, C, "reject")
    logits = torch.zeros(B, C, dtype=torch.float32, device="cuda")
    too_many = mt.STATIC_POOLER_MAX_FLOATS // H + 1          # batch * hidden beyond the built-in array
    with pytest.raises(mt.MTError) as e:
        mt.mt_kernel_pooler_head_static(*args, logits, too_many, S)
    assert e.value.code == -2
    torch.cuda.synchronize()
    assert torch.all(logits == 0), "a rejected call must not launch anything"
