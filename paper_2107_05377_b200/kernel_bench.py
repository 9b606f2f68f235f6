"""Micro-benchmark of the single steps of the path, each called through the C ABI.

    python -m paper_2107_05377_b200.kernel_bench linear --m 4096 --n 2304 --k 768 --epilogue 0
    python -m paper_2107_05377_b200.kernel_bench linear_ln --m 4096 --n 768 --k 3072   # residual GEMM + LayerNorm, one launch
    python -m paper_2107_05377_b200.kernel_bench attention --batch 32 --seq 128 --heads 12
    python -m paper_2107_05377_b200.kernel_bench layernorm --rows 4096 --hidden 768
    python -m paper_2107_05377_b200.kernel_bench embed --batch 256 --seq 128
    python -m paper_2107_05377_b200.kernel_bench linear_fp8 --m 4096 --n 2304 --k 768            # E4M3 operands
    python -m paper_2107_05377_b200.kernel_bench suite          # the shapes of the 32 x 128 workload

Times `--iters` launches between CUDA events on the launching stream after `--warmup` launches; with
`--flush` a buffer larger than L2 is written before every launch (each launch timed on its own).
Prints one JSON line per case with the achieved TFLOP/s or GB/s of the algorithmic work.  Inputs are
random; nothing is checked here (the parity tests do that).  This is also the command the ncu
summaries under profiles/ were captured from.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as mt

L2_FLUSH_BYTES = 256 << 20
USE_GRAPH = False
CTA_PAIR = False
TENSOR_MEMORY = True


def _time(fn, iters, warmup, flush):
    stream = torch.cuda.current_stream()
    buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda") if flush else None
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if USE_GRAPH and not flush:
        # the launches are recorded once into a CUDA graph and replayed, so that the host's launch
        # rate does not bound the measurement of short kernels
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(iters):
                fn()
        graph.replay()
        torch.cuda.synchronize()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        graph.replay()
        end.record()
        torch.cuda.synchronize()
        return start.elapsed_time(end) / iters
    if not flush:
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(stream)
        for _ in range(iters):
            fn()
        end.record(stream)
        torch.cuda.synchronize()
        return start.elapsed_time(end) / iters
    total = 0.0
    for i in range(iters):
        buf.fill_(i & 0xFF)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(stream)
        fn()
        end.record(stream)
        torch.cuda.synchronize()
        total += start.elapsed_time(end)
    return total / iters


def bench_linear(m, n, k, epilogue, iters, warmup, flush):
    x = torch.randn(m, k, device="cuda").to(torch.bfloat16)
    w = (0.02 * torch.randn(n, k, device="cuda")).to(torch.bfloat16)
    b = (0.02 * torch.randn(n, device="cuda")).to(torch.bfloat16)
    r = torch.randn(m, n, device="cuda") if epilogue == 2 else None
    y = torch.empty(m, n, device="cuda", dtype=torch.float32 if epilogue == 2 else torch.bfloat16)
    ms = _time(lambda: mt.mt_kernel_linear(x, w, b, r, y, epilogue, cta_pair=CTA_PAIR), iters, warmup, flush)
    flops = 2.0 * m * n * k
    bytes_ = 2.0 * (m * k + n * k) + (8.0 if epilogue == 2 else 2.0) * m * n
    return {"kernel": "linear", "M": m, "N": n, "K": k, "epilogue": epilogue, "us": 1e3 * ms,
            "tflops": flops / ms / 1e9, "min_gbytes_per_s": bytes_ / ms / 1e6}


def bench_linear_fp8(m, n, k, epilogue, iters, warmup, flush):
    """The 8-bit GEMM on operands quantised by the library's own row-wise kernel (timed: the GEMM alone)."""
    x = torch.randn(m, k, device="cuda").to(torch.bfloat16)
    w = (0.02 * torch.randn(n, k, device="cuda")).to(torch.bfloat16)
    b = (0.02 * torch.randn(n, device="cuda")).to(torch.bfloat16)
    r = torch.randn(m, n, device="cuda") if epilogue == 2 else None
    y = torch.empty(m, n, device="cuda", dtype=torch.float32 if epilogue == 2 else torch.bfloat16)
    xq, wq = torch.empty(m, k, device="cuda", dtype=torch.uint8), torch.empty(n, k, device="cuda", dtype=torch.uint8)
    sx, sw = torch.empty(m, device="cuda"), torch.empty(n, device="cuda")
    mt.mt_kernel_quantize_rows(x, xq, sx)
    mt.mt_kernel_quantize_rows(w, wq, sw)
    ms = _time(lambda: mt.mt_kernel_linear_fp8(xq, sx, wq, sw, b, r, y, epilogue), iters, warmup, flush)
    ms_q = _time(lambda: mt.mt_kernel_quantize_rows(x, xq, sx), iters, warmup, flush)
    return {"kernel": "linear_fp8", "M": m, "N": n, "K": k, "epilogue": epilogue, "us": 1e3 * ms,
            "tflops": 2.0 * m * n * k / ms / 1e9, "quantize_rows_us": 1e3 * ms_q}


def bench_linear_ln(m, n, k, iters, warmup, flush, tile_cols=128):
    x = torch.randn(m, k, device="cuda").to(torch.bfloat16)
    w = (0.02 * torch.randn(n, k, device="cuda")).to(torch.bfloat16)
    b = (0.02 * torch.randn(n, device="cuda")).to(torch.bfloat16)
    g = torch.ones(n, device="cuda", dtype=torch.bfloat16)
    be = torch.zeros(n, device="cuda", dtype=torch.bfloat16)
    r = torch.randn(m, n, device="cuda")
    y = torch.empty(m, n, device="cuda", dtype=torch.bfloat16)
    y32 = torch.empty(m, n, device="cuda")
    ms = _time(lambda: mt.mt_kernel_linear_layernorm(x, w, b, r, g, be, y, y32, 1e-12, tile_cols=tile_cols), iters, warmup, flush)
    flops = 2.0 * m * n * k
    bytes_ = 2.0 * (m * k + n * k) + (4.0 + 2.0 + 4.0) * m * n
    return {"kernel": "linear_ln", "tile_cols": tile_cols, "M": m, "N": n, "K": k, "us": 1e3 * ms, "tflops": flops / ms / 1e9,
            "min_gbytes_per_s": bytes_ / ms / 1e6}


def bench_attention(batch, seq, heads, len_lo, iters, warmup, flush):
    hidden = heads * 64
    qkv = torch.randn(batch * seq, 3 * hidden, device="cuda").to(torch.bfloat16)
    lengths = torch.randint(len_lo, seq + 1, (batch,), device="cuda", dtype=torch.int32)
    ctx = torch.empty(batch * seq, hidden, device="cuda", dtype=torch.bfloat16)
    ms = _time(lambda: mt.mt_kernel_attention(qkv, lengths, ctx, batch, seq, heads, tensor_memory=TENSOR_MEMORY and seq <= 512), iters, warmup, flush)
    bytes_ = 2.0 * 4 * batch * seq * hidden
    n = lengths.double()
    flops = float((4.0 * hidden * n * n).sum())
    return {"kernel": "attention", "batch": batch, "seq": seq, "heads": heads, "us": 1e3 * ms,
            "gbytes_per_s": bytes_ / ms / 1e6, "valid_tflops": flops / ms / 1e9}


def bench_embed(batch, seq, hidden, iters, warmup, flush):
    vocab = 30522
    tok = torch.randint(1000, vocab, (batch, seq), device="cuda", dtype=torch.int32)
    seg = torch.randint(0, 2, (batch, seq), device="cuda", dtype=torch.int32)
    lens = torch.full((batch,), seq, device="cuda", dtype=torch.int32)
    word = (0.02 * torch.randn(vocab, hidden, device="cuda")).to(torch.bfloat16)
    pos = (0.02 * torch.randn(512, hidden, device="cuda")).to(torch.bfloat16)
    typ = (0.02 * torch.randn(2, hidden, device="cuda")).to(torch.bfloat16)
    g = torch.ones(hidden, device="cuda", dtype=torch.bfloat16)
    b = torch.zeros(hidden, device="cuda", dtype=torch.bfloat16)
    h0 = torch.empty(batch * seq, hidden, device="cuda", dtype=torch.bfloat16)
    h32 = torch.empty(batch * seq, hidden, device="cuda")
    ms = _time(lambda: mt.mt_kernel_embed(tok, seg, lens, word, pos, typ, g, b, h0, 1e-12, h0_f32=h32), iters, warmup, flush)
    # per token: one word row and one position row read (bf16), the bf16 and the fp32 state written
    return {"kernel": "embed", "batch": batch, "seq": seq, "hidden": hidden, "us": 1e3 * ms,
            "gbytes_per_s": 10.0 * batch * seq * hidden / ms / 1e6}


def bench_layernorm(rows, hidden, iters, warmup, flush):
    x = torch.randn(rows, hidden, device="cuda")
    g = torch.ones(hidden, device="cuda", dtype=torch.bfloat16)
    b = torch.zeros(hidden, device="cuda", dtype=torch.bfloat16)
    y = torch.empty(rows, hidden, device="cuda", dtype=torch.bfloat16)
    y32 = torch.empty(rows, hidden, device="cuda")
    ms = _time(lambda: mt.mt_kernel_layernorm(x, g, b, y, 1e-12, y_f32=y32), iters, warmup, flush)
    return {"kernel": "layernorm", "rows": rows, "hidden": hidden, "us": 1e3 * ms,
            "gbytes_per_s": 10.0 * rows * hidden / ms / 1e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["linear", "linear_fp8", "linear_ln", "attention", "layernorm", "embed", "suite"])
    ap.add_argument("--m", type=int, default=4096)
    ap.add_argument("--n", type=int, default=2304)
    ap.add_argument("--k", type=int, default=768)
    ap.add_argument("--epilogue", type=int, default=0)
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--seq", type=int, default=128)
    ap.add_argument("--heads", type=int, default=12)
    ap.add_argument("--len-lo", type=int, default=16)
    ap.add_argument("--rows", type=int, default=4096)
    ap.add_argument("--hidden", type=int, default=768)
    ap.add_argument("--iters", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--flush", action="store_true")
    ap.add_argument("--graph", action="store_true", help="replay the launches from a CUDA graph")
    ap.add_argument("--tile-cols", type=int, default=128, help="linear_ln: accumulator tile width, 128 or 256")
    ap.add_argument("--block-n", type=int, default=0, help="linear: force the tile width (0 = automatic)")
    ap.add_argument("--pair", action="store_true", help="linear: pairs of CTAs on 256-row tiles (cta_group::2)")
    ap.add_argument("--mma-sync", action="store_true", help="attention: the mma.sync kernel also where seq <= 128")
    a = ap.parse_args()
    global USE_GRAPH, CTA_PAIR, TENSOR_MEMORY
    USE_GRAPH = a.graph
    CTA_PAIR = a.pair
    TENSOR_MEMORY = not a.mma_sync
    mt.lib().mt_kernel_linear_force_block_n(a.block_n)
    torch.manual_seed(0)
    if a.kernel == "linear":
        print(json.dumps(bench_linear(a.m, a.n, a.k, a.epilogue, a.iters, a.warmup, a.flush)))
    elif a.kernel == "linear_fp8":
        print(json.dumps(bench_linear_fp8(a.m, a.n, a.k, a.epilogue, a.iters, a.warmup, a.flush)))
    elif a.kernel == "linear_ln":
        print(json.dumps(bench_linear_ln(a.m, a.n, a.k, a.iters, a.warmup, a.flush, a.tile_cols)))
    elif a.kernel == "attention":
        print(json.dumps(bench_attention(a.batch, a.seq, a.heads, a.len_lo, a.iters, a.warmup, a.flush)))
    elif a.kernel == "layernorm":
        print(json.dumps(bench_layernorm(a.rows, a.hidden, a.iters, a.warmup, a.flush)))
    elif a.kernel == "embed":
        print(json.dumps(bench_embed(a.batch, a.seq, a.hidden, a.iters, a.warmup, a.flush)))
    else:
        for m in (2409, 4096, 24576):   # the valid tokens of the 32 x 128 batch, its padded rows, six layers of them
            for (n, k, e) in ((2304, 768, 0), (768, 768, 2), (3072, 768, 1), (768, 3072, 2)):
                print(json.dumps(bench_linear(m, n, k, e, a.iters, a.warmup, a.flush)))
            for (n, k) in ((768, 768), (768, 3072)):
                print(json.dumps(bench_linear_ln(m, n, k, a.iters, a.warmup, a.flush)))
            for (n, k, e) in ((2304, 768, 0), (3072, 768, 1), (768, 3072, 2)):
                print(json.dumps(bench_linear_fp8(m, n, k, e, a.iters, a.warmup, a.flush)))
        print(json.dumps(bench_linear(8192, 8192, 8192, 0, 10, 2, a.flush)))
        print(json.dumps(bench_linear_fp8(8192, 8192, 8192, 0, 10, 2, a.flush)))
        print(json.dumps(bench_attention(32, 128, 12, 16, a.iters, a.warmup, a.flush)))
        print(json.dumps(bench_attention(16, 512, 12, 128, a.iters, a.warmup, a.flush)))
        print(json.dumps(bench_layernorm(4096, 768, a.iters, a.warmup, a.flush)))


if __name__ == "__main__":
    main()
