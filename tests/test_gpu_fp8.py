"""The 8-bit (E4M3) path on the GPU against its oracle: the row-wise quantiser bit for bit (its decisions are
taken in fp32 on both sides), the tcgen05 kind::f8f6f4 GEMM on operands quantised by the ORACLE (products of
E4M3 values are exact in fp32, so only the accumulation order separates the two), and the quantised forward."""
import numpy as np
import pytest
import torch

from oracle import fp8_oracle as f8
from oracle import mt_oracle as orc
from paper_2107_05377_b200 import binding as mt
from paper_2107_05377_b200 import synth
from gpu_util import cached_weights, dev_batch, dev_bf16_to_f64, rand_bf16, rel_l2, task_triples, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols,std", [(1, 768, 1.0), (37, 768, 0.02), (300, 3072, 3.0), (129, 1024, 1.0), (64, 4096, 0.3)])
def test_quantiser_matches_the_oracle_bit_for_bit(rows, cols, std):
    xb, x = rand_bf16(41, f"q{rows}.{cols}", (rows, cols), std)
    if rows > 4:
        xb[3] = 0                     # a row of zeros
        x[3] = 0.0
        xb[4, 5:9] = 0x8000           # negative zeros keep their sign bit
        x[4, 5:9] = -0.0
    q = torch.full((rows + 2, cols), 0x55, dtype=torch.uint8, device="cuda")
    scale = torch.full((rows + 2,), -1.0, dtype=torch.float32, device="cuda")
    mt.mt_kernel_quantize_rows(to_dev_bf16(xb), q[:rows], scale[:rows])
    torch.cuda.synchronize()
    want_q, want_s = f8.quantize_rows(x)
    assert np.array_equal(scale[:rows].cpu().numpy(), want_s)
    assert np.array_equal(q[:rows].cpu().numpy(), want_q)
    assert torch.all(q[rows:] == 0x55) and torch.all(scale[rows:] == -1.0), "rows beyond the matrix were written"


@pytest.mark.parametrize("M,N,K,epi", [
    (64, 768, 768, 2),        # fewer rows than a tile, residual epilogue (128-wide tiles)
    (200, 2304, 768, 0),      # ragged last tile, Q/K/V shape
    (2409, 3072, 768, 1),     # FFN up + GELU at the valid-token count of the 32 x 128 batch
    (2409, 768, 3072, 2),     # FFN down + residual
    (520, 4096, 1024, 1),     # BERT-large width
    (1000, 1024, 4096, 2),
])
def test_fp8_linear_matches_the_oracle_on_oracle_quantised_operands(M, N, K, epi):
    xb, x = rand_bf16(51, f"x{M}.{N}.{K}", (M, K), 1.0)
    wb, w = rand_bf16(52, f"w{M}.{N}.{K}", (N, K), 0.05)
    bb, b = rand_bf16(53, f"b{M}.{N}.{K}", (N,), 0.5)
    r32 = (synth.standard_normal(54, f"r{M}.{N}.{K}", M * N).astype(np.float32)).reshape(M, N)
    xq, sx = f8.quantize_rows(x)
    wq, sw = f8.quantize_rows(w)
    out_dtype = torch.float32 if epi == 2 else torch.bfloat16
    y = torch.full((M + 8, N), float("nan"), dtype=out_dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mt.mt_kernel_linear_fp8(torch.from_numpy(xq).cuda(), torch.from_numpy(sx).cuda(), torch.from_numpy(wq).cuda(),
                            torch.from_numpy(sw).cuda(), to_dev_bf16(bb), torch.from_numpy(r32).cuda() if epi == 2 else None,
                            y[:M], epi, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = f8.dequantize_rows(xq, sx) @ f8.dequantize_rows(wq, sw).T + b
    if epi == 1:
        want = orc.gelu(want)
    if epi == 2:
        want = want + r32.astype(np.float64)
    got = y[:M].float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    assert torch.isnan(y[M:].float()).all(), "rows beyond M were written"
    if epi == 2:   # fp32 out: fp32 accumulation and the two fp32 scale products
        assert rel_l2(got, want) <= 1e-5
    else:          # one bf16 rounding of the output
        assert rel_l2(got, want) <= 3e-3
        assert np.max(np.abs(got - want)) <= float(np.max(np.abs(want))) * 2.0 ** -8 + 1e-3
    # and the quantisation itself costs what two E4M3 operands cost, no more
    exact = orc.linear(x, w, b)
    if epi == 0:
        assert rel_l2(got, exact) <= 0.06
