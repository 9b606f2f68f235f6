"""Per-kernel parity: each step of the path, called through the C ABI on the GPU,
against the matching fp64 oracle function on the same seeded bf16 inputs."""
import numpy as np
import pytest
import torch

from oracle import mt_oracle as orc
from paper_2107_05377_b200 import binding as mt
from paper_2107_05377_b200 import synth
from gpu_util import dev_bf16_to_f64, rand_bf16, rel_l2, to_dev_bf16

pytestmark = pytest.mark.gpu

# One bf16 rounding of the output (2^-9 relative) on top of fp32 accumulation.
OUT_REL_L2 = 3e-3


def bf16_round_tol(want):
    """max-abs bound for a result rounded once to bf16: half an ulp of the largest value + slack."""
    return float(np.max(np.abs(want))) * 2.0 ** -8 + 1e-3


@pytest.mark.parametrize("M,N,K,epi", [
    (64, 768, 768, 0),        # fewer rows than one tile
    (128, 128, 64, 0),        # a single tile, a single k-block
    (200, 768, 768, 2),       # ragged last tile, residual
    (333, 2304, 768, 0),      # wide tile (N=2304 uses 256-wide tiles), ragged
    (4096, 2304, 768, 0),     # QKV projection of the 32 x 128 batch
    (4096, 768, 768, 2),      # attention output + residual
    (4096, 3072, 768, 1),     # FFN up + GELU
    (4096, 768, 3072, 2),     # FFN down + residual
    (1000, 1024, 4096, 2),    # BERT-large width
    (520, 4096, 1024, 1),
])
@pytest.mark.parametrize("pair", [False, True], ids=["single_cta", "cta_pair"])
def test_linear_matches_oracle(M, N, K, epi, pair):
    xb, x = rand_bf16(11, f"x{M}.{N}.{K}", (M, K), 1.0)
    wb, w = rand_bf16(12, f"w{M}.{N}.{K}", (N, K), 0.05)
    bb, b = rand_bf16(13, f"b{M}.{N}.{K}", (N,), 0.5)
    r32 = (synth.standard_normal(14, f"r{M}.{N}.{K}", M * N).astype(np.float32)).reshape(M, N)   # fp32 residual
    out_dtype = torch.float32 if epi == 2 else torch.bfloat16
    y = torch.full((M + 8, N), float("nan"), dtype=out_dtype, device="cuda")   # 8 guard rows
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mt.mt_kernel_linear(to_dev_bf16(xb), to_dev_bf16(wb), to_dev_bf16(bb),
                        torch.from_numpy(r32).cuda() if epi == 2 else None, y[:M], epi, status=status, cta_pair=pair)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = orc.linear(x, w, b)
    if epi == 1:
        want = orc.gelu(want)
    if epi == 2:
        want = want + r32.astype(np.float64)
    got = y[:M].float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    assert torch.isnan(y[M:].float()).all(), "rows beyond M were written"
    if epi == 2:   # fp32 out: only fp32 accumulation error over K terms
        assert rel_l2(got, want) <= 1e-5
        assert np.max(np.abs(got - want)) <= 1e-4 * max(1.0, float(np.max(np.abs(want))))
    else:
        assert rel_l2(got, want) <= OUT_REL_L2
        assert np.max(np.abs(got - want)) <= bf16_round_tol(want)


@pytest.mark.parametrize("M,N,K", [
    (40, 768, 768),           # fewer rows than one tile: a single cluster of six CTAs
    (333, 768, 768),          # ragged last row block
    (2409, 768, 3072),        # FFN down + LayerNorm at the valid-token count of the 32 x 128 batch
    (4096, 768, 768),         # more row blocks than clusters fit the GPU at once: several tiles per cluster
    (700, 1024, 4096),        # BERT-large width: clusters of eight
    (7227, 768, 768),         # three layers' worth of valid tokens: several tiles per cluster
])
@pytest.mark.parametrize("tile_cols", [128, 256])
def test_linear_layernorm_cluster_matches_oracle_and_separate_kernels(M, N, K, tile_cols):
    """Residual GEMM + LayerNorm in one cluster launch (row statistics through distributed shared memory):
    against the oracle's linear + residual + layer_norm, and bit for bit against the plain residual GEMM
    followed by the LayerNorm kernel, which sums the row statistics in the same order."""
    xb, x = rand_bf16(21, f"x{M}.{N}.{K}", (M, K), 1.0)
    wb, w = rand_bf16(22, f"w{M}.{N}.{K}", (N, K), 0.05)
    bb, b = rand_bf16(23, f"b{M}.{N}.{K}", (N,), 0.5)
    gb, g = rand_bf16(24, f"g{N}", (N,), 0.3, mean=1.0)
    beb, be = rand_bf16(25, f"be{N}", (N,), 0.2)
    r32 = (synth.standard_normal(26, f"r{M}.{N}.{K}", M * N).astype(np.float32)).reshape(M, N)
    g_dev = to_dev_bf16(gb)
    res = torch.from_numpy(r32).cuda()
    y = torch.full((M + 8, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    y32 = torch.full((M + 8, N), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    xd, wd, bd, bed = to_dev_bf16(xb), to_dev_bf16(wb), to_dev_bf16(bb), to_dev_bf16(beb)
    mt.mt_kernel_linear_layernorm(xd, wd, bd, res, g_dev, bed, y[:M], y32[:M], 1e-12, status=status, tile_cols=tile_cols)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.isnan(y[M:].float()).all() and torch.isnan(y32[M:]).all(), "rows beyond M were written"
    want = orc.layer_norm(orc.linear(x, w, b) + r32.astype(np.float64), g, be, 1e-12)
    got32 = y32[:M].cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got32))
    assert rel_l2(got32, want) <= 1e-5
    got = y[:M].float().cpu().numpy().astype(np.float64)
    assert rel_l2(got, want) <= OUT_REL_L2
    assert np.max(np.abs(got - want)) <= bf16_round_tol(want)
    u = torch.empty(M, N, dtype=torch.float32, device="cuda")
    z = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    z32 = torch.empty(M, N, dtype=torch.float32, device="cuda")
    mt.mt_kernel_linear(xd, wd, bd, res, u, 2)
    mt.mt_kernel_layernorm(u, g_dev, bed, z, 1e-12, y_f32=z32)
    torch.cuda.synchronize()
    assert torch.equal(z32, y32[:M]) and torch.equal(z, y[:M])


def oracle_attention_from_qkv(qkv, lengths, B, S, heads):
    H = heads * 64
    ctx = np.zeros((B * S, H))
    for b in range(B):
        n = int(lengths[b])
        if n == 0:
            continue
        blk = qkv[b * S:b * S + n]
        for a in range(heads):
            q, k, v = (blk[:, i * H + a * 64:i * H + (a + 1) * 64] for i in range(3))
            ctx[b * S:b * S + n, a * 64:(a + 1) * 64] = orc.softmax_rows(q @ k.T / 8.0) @ v
    return ctx


@pytest.mark.parametrize("B,S,heads,lengths,tensor_memory", [
    (2, 32, 12, [32, 32], False),
    (4, 128, 12, [128, 37, 1, 64], False),
    (3, 100, 2, [100, 65, 9], False),       # seq not a multiple of the tile
    (2, 512, 16, [512, 300], False),
    (1, 1, 1, [1], False),
    (2, 32, 12, [32, 32], True),
    (6, 128, 12, [128, 37, 1, 64, 65, 127], True),
    (3, 100, 2, [100, 65, 9], True),        # the 128-row tile reaches into the next sequence and past the buffer
    (1, 1, 1, [1], True),
    (5, 128, 16, [0, 128, 0, 16, 113], True),   # a length of 0 is clamped to 1, as by every kernel of the path
    (5, 128, 16, [0, 128, 0, 16, 113], False),
    (2, 512, 16, [512, 300], True),           # more than 128 tokens: tiles of 128 queries walk tiles of 128 keys
    (3, 200, 2, [200, 129, 64], True),        # seq not a multiple of the tile; one key in the second tile
    (5, 384, 12, [1, 128, 257, 384, 0], True),
])
def test_attention_matches_oracle(B, S, heads, lengths, tensor_memory):
    H = heads * 64
    qb, qkv = rand_bf16(21, f"qkv{B}.{S}.{heads}", (B * S, 3 * H), 1.5)
    # poison the padded rows of the input: they must not leak into valid rows
    qkv_dev = to_dev_bf16(qb)
    lens = torch.tensor(lengths, dtype=torch.int32, device="cuda")
    lengths = [max(n, 1) for n in lengths]
    for b, n in enumerate(lengths):
        qkv_dev[b * S + n:(b + 1) * S] = float("nan")
    ctx = torch.full((B * S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mt.mt_kernel_attention(qkv_dev, lens, ctx, B, S, heads, tensor_memory=tensor_memory, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = dev_bf16_to_f64(ctx)
    want = oracle_attention_from_qkv(qkv, lengths, B, S, heads)
    assert np.all(np.isfinite(got))
    for b, n in enumerate(lengths):
        assert np.all(got[b * S + n:(b + 1) * S] == 0), "padded query rows must be written as zero"
    # probabilities are rounded to bf16 before the second product: 2^-9 relative per term
    assert rel_l2(got, want) <= 5e-3
    assert np.max(np.abs(got - want)) <= 2e-2 * max(1.0, float(np.max(np.abs(want))))


@pytest.mark.parametrize("rows,H", [(1, 768), (8, 768), (4099, 768), (1000, 1024)])
def test_layernorm_matches_oracle(rows, H):
    x32 = (0.7 + 2.0 * synth.standard_normal(31, f"ln{rows}", rows * H)).astype(np.float32).reshape(rows, H)
    gb, g = rand_bf16(32, f"g{H}", (H,), 0.2, mean=1.0)
    bb, b = rand_bf16(33, f"b{H}", (H,), 0.2)
    y = torch.empty(rows, H, dtype=torch.bfloat16, device="cuda")
    y32 = torch.empty(rows, H, dtype=torch.float32, device="cuda")
    mt.mt_kernel_layernorm(torch.from_numpy(x32).cuda(), to_dev_bf16(gb), to_dev_bf16(bb), y, 1e-12, y_f32=y32)
    torch.cuda.synchronize()
    want = orc.layer_norm(x32.astype(np.float64), g, b, 1e-12)
    got = dev_bf16_to_f64(y)
    assert rel_l2(got, want) <= OUT_REL_L2
    assert np.max(np.abs(got - want)) <= bf16_round_tol(want)
    got32 = y32.cpu().numpy().astype(np.float64)
    assert rel_l2(got32, want) <= 1e-5
    assert torch.equal(y32.to(torch.bfloat16), y), "the bf16 copy is the rounding of the fp32 copy"
    y_only = torch.empty_like(y)
    mt.mt_kernel_layernorm(torch.from_numpy(x32).cuda(), to_dev_bf16(gb), to_dev_bf16(bb), y_only, 1e-12)
    torch.cuda.synchronize()
    assert torch.equal(y_only, y)


@pytest.mark.parametrize("M,N,K,splits", [
    (1, 768, 3072, 4),       # a first-token tail of a single sequence
    (32, 768, 3072, 4),      # the first-token tail of the 32 x 128 batch
    (100, 768, 3072, 4),     # ragged
    (128, 768, 3072, 4),     # batch 1
    (512, 768, 3072, 4),     # batch 4: four row blocks
    (300, 1024, 4096, 4),    # BERT-large width
    (77, 768, 768, 2),
])
@pytest.mark.parametrize("block_n", [0, 64, 128])
def test_split_k_projection_and_its_layernorm(M, N, K, splits, block_n):
    """The FFN-down projection of launches of few rows: partial sums over ranges of K, then one kernel that adds the
    ranges in order, the bias and the residual and normalises the row."""
    xb, x = rand_bf16(71, f"x{M}.{N}.{K}", (M, K), 1.0)
    wb, w = rand_bf16(72, f"w{M}.{N}.{K}", (N, K), 0.05)
    bb, b = rand_bf16(73, f"b{M}.{N}.{K}", (N,), 0.5)
    gb, g = rand_bf16(74, f"g{N}", (N,), 0.2, mean=1.0)
    eb, e = rand_bf16(75, f"e{N}", (N,), 0.2)
    r32 = (synth.standard_normal(76, f"r{M}.{N}.{K}", M * N).astype(np.float32)).reshape(M, N)
    pitch = (M + 127) // 128 * 128
    part = torch.full((splits * pitch + 8, N), float("nan"), dtype=torch.float32, device="cuda")   # 8 guard rows
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lib = mt.lib()
    lib.mt_kernel_linear_force_block_n(block_n)
    try:
        mt.mt_kernel_linear_partial(to_dev_bf16(xb), to_dev_bf16(wb), part, splits, pitch, status=status)
        torch.cuda.synchronize()
    finally:
        lib.mt_kernel_linear_force_block_n(0)
    assert int(status.item()) == 0
    assert torch.isnan(part[splits * pitch:]).all(), "rows beyond the last range were written"
    got = part.cpu().numpy()
    ks = K // splits
    for s in range(splits):
        want_s = x[:, s * ks:(s + 1) * ks] @ w[:, s * ks:(s + 1) * ks].T          # this range of K alone, fp64
        got_s = got[s * pitch:s * pitch + M].astype(np.float64)
        assert np.all(np.isfinite(got_s))
        assert rel_l2(got_s, want_s) <= 1e-5, s
    # the rows put together and normalised, against the oracle's residual sub-layer
    y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    y32 = torch.empty(M, N, dtype=torch.float32, device="cuda")
    r_dev = torch.from_numpy(r32).cuda()
    mt.mt_kernel_layernorm_partial(part, splits, pitch, r_dev, to_dev_bf16(bb), to_dev_bf16(gb), to_dev_bf16(eb), y, 1e-12,
                                   y_f32=y32)
    torch.cuda.synchronize()
    want = orc.layer_norm(r32.astype(np.float64) + orc.linear(x, w, b), g, e, 1e-12)
    assert rel_l2(dev_bf16_to_f64(y), want) <= OUT_REL_L2
    assert rel_l2(y32.cpu().numpy().astype(np.float64), want) <= 2e-5
    # the order of the additions is part of the definition: residual + ((p0 + p1 + ...) + bias) in fp32, formed on
    # the host from the kernel's own partial sums, must normalise to the same bits
    acc = got[0:M].copy()
    for s in range(1, splits):
        acc = acc + got[s * pitch:s * pitch + M]
    x_host = r32 + (acc + b.astype(np.float32))
    y_ref = torch.empty_like(y)
    mt.mt_kernel_layernorm(torch.from_numpy(x_host.astype(np.float32)).cuda(), to_dev_bf16(gb), to_dev_bf16(eb), y_ref,
                           1e-12)
    torch.cuda.synchronize()
    assert torch.equal(y_ref, y)
    # and the unsplit kernels give the same result to fp32 rounding of the sum over K
    u = torch.empty(M, N, dtype=torch.float32, device="cuda")
    mt.mt_kernel_linear(to_dev_bf16(xb), to_dev_bf16(wb), to_dev_bf16(bb), r_dev, u, 2, status=status)
    y_plain = torch.empty(M, N, dtype=torch.float32, device="cuda")
    mt.mt_kernel_layernorm(u, to_dev_bf16(gb), to_dev_bf16(eb), torch.empty_like(y), 1e-12, y_f32=y_plain)
    torch.cuda.synchronize()
    assert rel_l2(y32.cpu().numpy().astype(np.float64), y_plain.cpu().numpy().astype(np.float64)) <= 2e-5


@pytest.mark.parametrize("H", [768, 1024])
def test_embed_matches_oracle_and_flags_bad_ids(H):
    B, S, V = 3, 40, 500
    wb, w = rand_bf16(41, f"word{H}", (V, H), 0.02)
    pb, p = rand_bf16(42, f"pos{H}", (64, H), 0.02)
    tb, t = rand_bf16(43, f"type{H}", (2, H), 0.02)
    gb, g = rand_bf16(44, f"eg{H}", (H,), 0.2, mean=1.0)
    bb, b = rand_bf16(45, f"eb{H}", (H,), 0.2)
    rng = np.random.default_rng(5)
    tok = rng.integers(0, V, (B, S)).astype(np.int32)
    seg = rng.integers(0, 2, (B, S)).astype(np.int32)
    lens = np.array([40, 17, 1], dtype=np.int32)
    out = torch.empty(B * S, H, dtype=torch.bfloat16, device="cuda")
    out32 = torch.empty(B * S, H, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = [to_dev_bf16(a) for a in (wb, pb, tb, gb, bb)]
    mt.mt_kernel_embed(torch.from_numpy(tok).cuda(), torch.from_numpy(seg).cuda(), torch.from_numpy(lens).cuda(),
                       *args, out, 1e-12, h0_f32=out32, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out32.to(torch.bfloat16), out)
    emb = {"word": w, "pos": p, "type": t, "ln_g": g, "ln_b": b}
    got = dev_bf16_to_f64(out).reshape(B, S, H)
    for i in range(B):
        want = orc.embed(tok[i], seg[i], emb, 1e-12)   # every position, padded ones included
        assert rel_l2(got[i], want) <= OUT_REL_L2
        assert np.max(np.abs(got[i] - want)) <= bf16_round_tol(want)
    # out-of-range ids are clamped and reported, never dereferenced
    tok[0, 0], seg[1, 1], lens[2] = V + 7, 5, 0
    mt.mt_kernel_embed(torch.from_numpy(tok).cuda(), torch.from_numpy(seg).cuda(), torch.from_numpy(lens).cuda(),
                       *args, out, 1e-12, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == (mt.FLAG_BAD_TOKEN | mt.FLAG_BAD_SEGMENT | mt.FLAG_BAD_LENGTH)
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("B,S,H,C", [(2, 32, 768, 2), (32, 128, 768, 3), (9, 16, 1024, 1), (1, 8, 768, 1)])
def test_pooler_head_matches_oracle(B, S, H, C):
    hb, h = rand_bf16(51, f"h{B}.{S}.{H}", (B * S, H), 1.0)
    pwb, pw = rand_bf16(52, f"pw{H}", (H, H), 0.05)
    pbb, pb = rand_bf16(53, f"pb{H}", (H,), 0.1)
    cwb, cw = rand_bf16(54, f"cw{H}.{C}", (C, H), 0.05)
    cbb, cb = rand_bf16(55, f"cb{C}", (C,), 0.1)
    logits = torch.full((B, C + 3), -77.0, dtype=torch.float32, device="cuda")
    scratch = torch.empty(B, H, dtype=torch.float32, device="cuda")
    mt.mt_kernel_pooler_head(to_dev_bf16(hb), to_dev_bf16(pwb), to_dev_bf16(pbb), to_dev_bf16(cwb), to_dev_bf16(cbb),
                             scratch, logits, B, S, col0=2)
    torch.cuda.synchronize()
    got = logits.cpu().numpy().astype(np.float64)
    tw = {"pool_w": pw, "pool_b": pb, "cls_w": cw, "cls_b": cb}
    for i in range(B):
        want = orc.pooler_head(h[i * S:(i + 1) * S], tw)
        assert np.max(np.abs(got[i, 2:2 + C] - want)) <= 1e-4
    assert np.all(got[:, :2] == -77.0) and np.all(got[:, 2 + C:] == -77.0), "other tasks' columns must be untouched"


def test_gelu_epilogue_stays_within_its_stated_fit_error():
    """The FFN-up epilogue evaluates the exact-form GELU x * Phi(x) through a fitted sigmoid argument whose
    stated largest absolute error is 2.6e-5; the result is then rounded once to bf16.  Pre-activations on a
    grid over [-8, 8] are produced exactly (one non-zero weight of 1 per output, zero bias)."""
    M, N, K = 128, 128, 64
    grid = np.linspace(-8.0, 8.0, M * K, dtype=np.float32).reshape(M, K)
    xb = synth.f32_to_bf16_bits(grid)
    x = synth.bf16_bits_to_f64(xb)
    w = np.zeros((N, K), dtype=np.float32)
    w[np.arange(N), np.arange(N) % K] = 1.0          # output n of row m is x[m, n % 64]
    y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    mt.mt_kernel_linear(to_dev_bf16(xb), to_dev_bf16(synth.f32_to_bf16_bits(w)),
                        to_dev_bf16(synth.f32_to_bf16_bits(np.zeros(N, dtype=np.float32))), None, y, 1)
    torch.cuda.synchronize()
    got = dev_bf16_to_f64(y)
    want = orc.gelu(x[:, np.arange(N) % K])
    half_ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want), 1e-30))) - 8)
    assert np.all(np.abs(got - want) <= 2.6e-5 + half_ulp + 1e-9)
