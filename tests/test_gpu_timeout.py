"""The time-out path of the kernels' pipeline waits, without hanging anything: the bounded mbarrier wait that every
tensor-core kernel of the path uses is run on a barrier that nothing completes, with a limit of a few
milliseconds; the wait gives up, the other role leaves through the CTA's abort flag, the status word reports it,
and the context keeps working."""
import numpy as np
import pytest
import torch

from paper_2107_05377_b200 import binding as mt

pytestmark = pytest.mark.gpu

MT_FLAG_WAIT_TIMEOUT = 0x8


def probe(limit_ns, arrive):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(2, dtype=torch.int64, device="cuda")
    ok = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    mt.mt_debug_wait_probe(limit_ns, arrive, status, waited, ok)
    torch.cuda.synchronize()
    return int(status.item()), waited.cpu().numpy(), ok.cpu().numpy()


def test_a_wait_that_nothing_completes_gives_up_and_reports_it():
    limit = 3_000_000   # 3 ms (the kernels' own limit is 4 s)
    status, waited, ok = probe(limit, arrive=False)
    assert status == MT_FLAG_WAIT_TIMEOUT
    assert list(ok) == [0, 0]
    # warp 0 waited for its limit (the clock is read every 256 polls: a little more, never less)
    assert limit <= waited[0] <= 20 * limit
    # warp 1's own limit was 64 times longer: it left because warp 0 raised the abort flag
    assert waited[1] < 32 * limit
    # a barrier that is complete: no waiting to speak of, no flag
    status, waited, ok = probe(limit, arrive=True)
    assert status == 0 and list(ok) == [1, 1]
    assert waited.max() < limit
    # the status word is sticky across calls that share it, and the context is alive: an ordinary kernel still runs
    x = torch.randn(8, 768, device="cuda")
    g = torch.ones(768, device="cuda").to(torch.bfloat16)
    b = torch.zeros(768, device="cuda").to(torch.bfloat16)
    y = torch.empty(8, 768, dtype=torch.bfloat16, device="cuda")
    mt.mt_kernel_layernorm(x, g, b, y, 1e-12)
    torch.cuda.synchronize()
    want = torch.nn.functional.layer_norm(x, (768,), eps=1e-12)
    assert float((y.float() - want).abs().max()) < 3e-2


def test_probe_rejects_limits_outside_its_range():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(2, dtype=torch.int64, device="cuda")
    ok = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(mt.MTError):
        mt.mt_debug_wait_probe(10_000_000_000, False, status, waited, ok)   # 10 s: refused on the host
    with pytest.raises(mt.MTError):
        mt.mt_debug_wait_probe(10, False, status, waited, ok)
