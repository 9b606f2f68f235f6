"""Pins for the fp64 oracle: closed forms, invariants, brute force on tiny
shapes written in a different loop order, and the layer totals the paper prints
in Tables 2 and 4.  None of these call the CUDA path."""
import math
import os
import re

import numpy as np
import pytest

from oracle import mt_oracle as orc
from paper_2107_05377_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# helpers: a tiny random model in float64 (not bf16: the oracle is dtype-blind)
# ---------------------------------------------------------------------------

def tiny_layer(rng, H, F, random_affine=True):
    L = {}
    for name, shape in {"wq": (H, H), "wk": (H, H), "wv": (H, H), "wo": (H, H), "w1": (F, H), "w2": (H, F)}.items():
        L[name] = rng.normal(0, 0.5, shape)
    for name, n in {"bq": H, "bk": H, "bv": H, "bo": H, "b1": F, "b2": H}.items():
        L[name] = rng.normal(0, 0.5, n)
    for name in ("ln1", "ln2"):
        L[name + "_g"] = rng.normal(1, 0.3, H) if random_affine else np.ones(H)
        L[name + "_b"] = rng.normal(0, 0.3, H) if random_affine else np.zeros(H)
    return L


def tiny_model(rng, H=8, F=16, vocab=20, max_pos=12, trunk=4, tasks=((2, 1, 2), (4, 2, 3), (0, 1, 1), (3, 0, 2))):
    emb = {"word": rng.normal(0, 1, (vocab, H)), "pos": rng.normal(0, 1, (max_pos, H)),
           "type": rng.normal(0, 1, (2, H)), "ln_g": rng.normal(1, 0.2, H), "ln_b": rng.normal(0, 0.2, H)}
    w = {"emb": emb, "trunk": [tiny_layer(rng, H, F) for _ in range(trunk)], "tasks": []}
    for (_, y, c) in tasks:
        w["tasks"].append({"layers": [tiny_layer(rng, H, F) for _ in range(y)],
                           "pool_w": rng.normal(0, 0.5, (H, H)), "pool_b": rng.normal(0, 0.5, H),
                           "cls_w": rng.normal(0, 0.5, (c, H)), "cls_b": rng.normal(0, 0.5, c)})
    return w, list(tasks)


# ---------------------------------------------------------------------------
# softmax
# ---------------------------------------------------------------------------

def test_softmax_rows_sum_to_one_and_closed_forms():
    rng = np.random.default_rng(0)
    s = rng.normal(0, 30, (7, 13))
    p = orc.softmax_rows(s)
    assert np.all(np.abs(p.sum(-1) - 1) <= 1e-15 * 4)
    assert np.all(p >= 0)
    # one key: weight is exactly 1
    assert orc.softmax_rows(np.array([[123.456]]))[0, 0] == 1.0
    # equal scores: uniform
    assert np.array_equal(orc.softmax_rows(np.full((2, 5), -3.25)), np.full((2, 5), 0.2))
    # two keys: logistic closed form
    a, b = 0.7, -1.9
    p2 = orc.softmax_rows(np.array([[a, b]]))[0]
    assert abs(p2[0] - 1 / (1 + math.exp(b - a))) < 1e-16 * 4
    assert abs(p2[1] - 1 / (1 + math.exp(a - b))) < 1e-16 * 4
    # shift invariance and no overflow at large magnitude
    big = orc.softmax_rows(np.array([[1000.0, 1001.0, 999.0]]))
    small = orc.softmax_rows(np.array([[0.0, 1.0, -1.0]]))
    assert np.allclose(big, small, rtol=0, atol=1e-15)


# ---------------------------------------------------------------------------
# LayerNorm
# ---------------------------------------------------------------------------

def test_layer_norm_hand_example():
    # x = [1,2,3,4]: mean 2.5, biased variance 1.25
    x = np.array([[1.0, 2.0, 3.0, 4.0]])
    g = np.array([1.0, 2.0, 3.0, 4.0])
    b = np.array([0.1, 0.2, 0.3, 0.4])
    y = orc.layer_norm(x, g, b, 0.0)[0]
    r = 1.0 / math.sqrt(1.25)
    want = [1 * (-1.5 * r) + 0.1, 2 * (-0.5 * r) + 0.2, 3 * (0.5 * r) + 0.3, 4 * (1.5 * r) + 0.4]
    assert np.allclose(y, want, rtol=0, atol=1e-15)
    assert abs(-1.5 * r - (-1.3416407864998738)) < 1e-15  # the printed decimal of 1.5/sqrt(1.25)


def test_layer_norm_moments_and_constant_row():
    rng = np.random.default_rng(1)
    x = rng.normal(3, 5, (11, 768))
    eps = 1e-12
    y = orc.layer_norm(x, np.ones(768), np.zeros(768), eps)
    assert np.all(np.abs(y.mean(-1)) < 1e-14)
    var_in = x.var(-1)  # numpy's default is the biased estimator
    assert np.allclose(y.var(-1), var_in / (var_in + eps), rtol=1e-13, atol=0)
    # an unbiased-variance mistake would give 767/768 here
    assert np.all(np.abs(y.var(-1) - 1) < 1e-9)
    beta = rng.normal(0, 1, 768)
    const = orc.layer_norm(np.full((2, 768), 4.5), rng.normal(1, 1, 768), beta, eps)
    assert np.array_equal(const, np.broadcast_to(beta, (2, 768)))
    # eps really is inside the square root: variance 1 row, eps = 3 -> scale 1/2
    row = np.array([[-1.0, 1.0, -1.0, 1.0]])
    assert np.allclose(orc.layer_norm(row, np.ones(4), np.zeros(4), 3.0), row / 2, rtol=0, atol=1e-16)


# ---------------------------------------------------------------------------
# GELU
# ---------------------------------------------------------------------------

def test_gelu_identities_and_values():
    x = np.linspace(-8, 8, 3201)
    g = orc.gelu(x)
    assert orc.gelu(np.array([0.0]))[0] == 0.0
    assert np.allclose(g - orc.gelu(-x), x, rtol=0, atol=2e-15)          # Phi(x) + Phi(-x) = 1
    assert np.all(np.diff(g[x >= 0]) > 0)                                 # increasing on x >= 0
    assert abs(orc.gelu(np.array([30.0]))[0] - 30.0) < 1e-12
    assert abs(orc.gelu(np.array([-30.0]))[0]) < 1e-12
    # Phi(1) and Phi(2) from standard normal tables
    assert abs(orc.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15
    assert abs(orc.gelu(np.array([-1.0]))[0] + 0.15865525393145707) < 1e-15
    assert abs(orc.gelu(np.array([2.0]))[0] - 2 * 0.9772498680518208) < 1e-15
    # the tanh approximation differs from the exact form by ~1e-4 at x = 2: make sure we are the exact one
    t = 0.5 * 2.0 * (1 + math.tanh(math.sqrt(2 / math.pi) * (2.0 + 0.044715 * 8.0)))
    assert abs(orc.gelu(np.array([2.0]))[0] - t) > 5e-5
    for v in (-2.5, -0.3, 0.9, 3.1):
        assert abs(orc.gelu(np.array([v]))[0] - v * 0.5 * (1 + math.erf(v / math.sqrt(2)))) < 1e-15


# ---------------------------------------------------------------------------
# linear and attention: scalar loops in another order, and closed forms
# ---------------------------------------------------------------------------

def test_linear_is_x_wT_plus_b_scalar_loops():
    rng = np.random.default_rng(2)
    x, w, b = rng.normal(size=(3, 8)), rng.normal(size=(5, 8)), rng.normal(size=5)
    y = orc.linear(x, w, b)
    assert y.shape == (3, 5)
    for i in range(3):
        for o in range(5):
            acc = b[o]
            for k in range(8):
                acc += x[i, k] * w[o, k]
            assert abs(y[i, o] - acc) < 1e-13


def brute_attention(h, L, heads):
    """head-major scalar loops: for each head, for each query, explicit exp/sum."""
    n, H = len(h), len(h[0])
    dh = H // heads
    ctx = [[0.0] * H for _ in range(n)]

    def proj(i, o, w, b):
        return b[o] + sum(h[i][k] * w[o][k] for k in range(H))

    for a in range(heads):
        for i in range(n):
            qi = [proj(i, a * dh + c, L["wq"], L["bq"]) for c in range(dh)]
            sc = []
            for j in range(n):
                kj = [proj(j, a * dh + c, L["wk"], L["bk"]) for c in range(dh)]
                sc.append(sum(qi[c] * kj[c] for c in range(dh)) / math.sqrt(dh))
            m = max(sc)
            ex = [math.exp(s - m) for s in sc]
            z = sum(ex)
            for c in range(dh):
                ctx[i][a * dh + c] = sum(ex[j] / z * proj(j, a * dh + c, L["wv"], L["bv"]) for j in range(n))
    return np.array(ctx)


def test_attention_brute_force_tiny():
    rng = np.random.default_rng(3)
    H, F, S, heads = 8, 16, 3, 2
    L = tiny_layer(rng, H, F)
    h = rng.normal(size=(S, H))
    got = orc.attention(h, L, heads)
    want = brute_attention(h.tolist(), {k: v.tolist() for k, v in L.items()}, heads)
    assert np.allclose(got, want, rtol=0, atol=1e-13)


def test_attention_closed_forms():
    rng = np.random.default_rng(4)
    n = 4
    # (a) zero query/key projections: all scores equal, context = mean of V rows
    L = tiny_layer(rng, 8, 16)
    for k in ("wq", "wk"):
        L[k] = np.zeros((8, 8))
    L["bq"] = np.zeros(8)
    h = rng.normal(size=(5, 8))
    v = h @ L["wv"].T + L["bv"]
    assert np.allclose(orc.attention(h, L, 2), np.broadcast_to(v.mean(0), (5, 8)), rtol=0, atol=1e-14)
    # (b) one head, h = I, keys = I, values = I: context rows are the softmax rows of wq^T / sqrt(n)
    A = rng.normal(size=(n, n))
    L1 = {"wq": A, "wk": np.eye(n), "wv": np.eye(n), "bq": np.zeros(n), "bk": np.zeros(n), "bv": np.zeros(n)}
    ctx = orc.attention(np.eye(n), L1, 1)
    for i in range(n):
        e = [math.exp(A[j, i] / 2.0) for j in range(n)]
        for j in range(n):
            assert abs(ctx[i, j] - e[j] / sum(e)) < 1e-15
    # (c) a single valid token attends to itself only: context = its value row
    one = orc.attention(h[:1], L, 2)
    assert np.allclose(one, h[:1] @ L["wv"].T + L["bv"], rtol=0, atol=1e-15)


# ---------------------------------------------------------------------------
# whole layer
# ---------------------------------------------------------------------------

def brute_layer(h, L, heads, eps):
    """Token-major scalar evaluation of the post-LN encoder layer."""
    n, H = h.shape
    F = len(L["b1"])
    ctx = brute_attention(h.tolist(), {k: np.asarray(v).tolist() for k, v in L.items()}, heads)

    def ln(row, g, b):
        m = sum(row) / len(row)
        v = sum((r - m) ** 2 for r in row) / len(row)
        return [g[i] * (row[i] - m) / math.sqrt(v + eps) + b[i] for i in range(len(row))]

    out = []
    for i in range(n):
        u = [h[i, o] + L["bo"][o] + sum(ctx[i, k] * L["wo"][o, k] for k in range(H)) for o in range(H)]
        h1 = ln(u, L["ln1_g"], L["ln1_b"])
        f = []
        for o in range(F):
            z = L["b1"][o] + sum(h1[k] * L["w1"][o, k] for k in range(H))
            f.append(0.5 * z * (1 + math.erf(z / math.sqrt(2))))
        u2 = [h1[o] + L["b2"][o] + sum(f[k] * L["w2"][o, k] for k in range(F)) for o in range(H)]
        out.append(ln(u2, L["ln2_g"], L["ln2_b"]))
    return np.array(out)


def test_encoder_layer_brute_force_tiny():
    rng = np.random.default_rng(5)
    H, F, S, heads, eps = 8, 16, 3, 2, 1e-12
    L = tiny_layer(rng, H, F)
    h = rng.normal(size=(S, H))
    assert np.allclose(orc.encoder_layer(h, L, heads, eps), brute_layer(h, L, heads, eps), rtol=0, atol=1e-12)


def test_encoder_layer_zero_projections_reduce_to_layernorms():
    rng = np.random.default_rng(6)
    H, F, eps = 16, 32, 1e-12
    L = tiny_layer(rng, H, F, random_affine=False)
    for k in ("wo", "w2"):
        L[k] = np.zeros_like(L[k])
    for k in ("bo", "b2"):
        L[k] = np.zeros_like(L[k])
    h = rng.normal(2, 3, (6, H))
    want = (h - h.mean(-1, keepdims=True)) / h.std(-1, keepdims=True)   # LN(LN(h)) = LN(h) up to O(eps)
    assert np.allclose(orc.encoder_layer(h, L, 4, eps), want, rtol=0, atol=1e-10)
    # residual + bias paths alone: value projection and FFN-up zeroed
    L = tiny_layer(rng, H, F, random_affine=True)
    L["wv"], L["bv"] = np.zeros((H, H)), np.zeros(H)
    L["w1"], L["b1"] = np.zeros((F, H)), np.zeros(F)

    def ln(x, g, b):
        return g * (x - x.mean(-1, keepdims=True)) / np.sqrt(x.var(-1, keepdims=True) + eps) + b

    h1 = ln(h + L["bo"], L["ln1_g"], L["ln1_b"])
    assert np.allclose(orc.encoder_layer(h, L, 4, eps), ln(h1 + L["b2"], L["ln2_g"], L["ln2_b"]), rtol=0, atol=1e-12)


# ---------------------------------------------------------------------------
# embeddings, pooler, head
# ---------------------------------------------------------------------------

def test_embed_indices_scalar():
    rng = np.random.default_rng(7)
    w, _ = tiny_model(rng)
    tok = np.array([5, 19, 0, 7, 7])
    seg = np.array([0, 0, 1, 1, 0])
    got = orc.embed(tok, seg, w["emb"], 1e-12)
    for i in range(5):
        e = w["emb"]["word"][tok[i]] + w["emb"]["pos"][i] + w["emb"]["type"][seg[i]]
        want = w["emb"]["ln_g"] * (e - e.mean()) / math.sqrt(e.var() + 1e-12) + w["emb"]["ln_b"]
        assert np.allclose(got[i], want, rtol=0, atol=1e-13)


def test_pooler_head_row0_tanh_scalar():
    rng = np.random.default_rng(8)
    w, tasks = tiny_model(rng)
    tw = w["tasks"][1]
    g = rng.normal(size=(4, 8))
    got = orc.pooler_head(g, tw)
    pooled = [math.tanh(tw["pool_b"][o] + sum(g[0, k] * tw["pool_w"][o, k] for k in range(8))) for o in range(8)]
    want = [tw["cls_b"][c] + sum(pooled[k] * tw["cls_w"][c, k] for k in range(8)) for c in range(3)]
    assert np.allclose(got, want, rtol=0, atol=1e-14)
    g2 = g.copy()
    g2[1:] += 5.0
    assert np.array_equal(orc.pooler_head(g2, tw), got)
    assert orc.pooler_head(g, w["tasks"][2]).shape == (1,)  # 1-wide regression head, raw output


def test_token_head_is_one_linear_map_per_token_scalar():
    """Token-level head: logits[i, c] = b_c + sum_k g[i, k] W_c[c, k] for every token i, by scalar loops;
    a token's logits depend on that token's state alone; no pooler weights are involved."""
    rng = np.random.default_rng(18)
    w, tasks = tiny_model(rng)
    tw = w["tasks"][1]
    g = rng.normal(size=(5, 8))
    got = orc.token_head(g, tw)
    assert got.shape == (5, 3)
    for i in range(5):
        for c in range(3):
            want = tw["cls_b"][c] + sum(g[i, k] * tw["cls_w"][c, k] for k in range(8))
            assert abs(got[i, c] - want) <= 1e-14
    g2 = g.copy()
    g2[3] += 1.0
    again = orc.token_head(g2, tw)
    assert np.array_equal(np.delete(again, 3, axis=0), np.delete(got, 3, axis=0)) and not np.array_equal(again[3], got[3])
    tw2 = dict(tw)
    tw2["pool_w"] = tw["pool_w"] + 1.0
    tw2["pool_b"] = tw["pool_b"] - 1.0
    assert np.array_equal(orc.token_head(g, tw2), got)
    # zero weight matrix: every token gets the bias
    tw3 = dict(tw)
    tw3["cls_w"] = np.zeros_like(tw["cls_w"])
    assert np.array_equal(orc.token_head(g, tw3), np.tile(tw["cls_b"], (5, 1)))


def test_token_level_tasks_in_the_merged_tree():
    """A tree that mixes sequence-level and token-level tasks: merged == stand-alone for both kinds, the
    token-level task's logits are its final state through the linear head, padding and task masking
    leave them untouched, and the two kinds of output have separate column spaces."""
    rng = np.random.default_rng(19)
    tasks = ((2, 1, 2, 0), (4, 2, 3, 1), (0, 1, 1), (3, 0, 2, 1))
    w, _ = tiny_model(rng, tasks=tuple(t[:3] for t in tasks))
    tok, seg, lens = _inputs(rng, 3, 10, 20, [10, 4, 1])
    for b in range(3):
        hid = {}
        mt = orc.forward_sequence_mt(tok[b], seg[b], lens[b], w, tasks, 2, 1e-12, hidden_out=hid)
        for t in range(4):
            st = orc.forward_sequence_st(tok[b], seg[b], lens[b], w, t, tasks, 2, 1e-12)
            want_shape = (lens[b], tasks[t][2]) if orc.head_kind(tasks[t]) == 1 else (tasks[t][2],)
            assert mt[t].shape == want_shape
            assert np.max(np.abs(mt[t] - st)) <= 1e-12
        final1 = hid[("task", 1, 2)]
        assert np.array_equal(mt[1], final1 @ w["tasks"][1]["cls_w"].T + w["tasks"][1]["cls_b"])
        assert np.array_equal(mt[3], hid[("trunk", 3)] @ w["tasks"][3]["cls_w"].T + w["tasks"][3]["cls_b"])
    tl = []
    logits = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12, token_logits_out=tl)
    assert logits.shape == (3, 3) and tl[0].shape == (3, 10, 5)     # sequence-level: 2 + 1; token-level: 3 + 2
    assert np.all(np.isnan(tl[0][1, 4:])) and np.all(np.isfinite(tl[0][1, :4])) and np.all(np.isfinite(logits))
    # padding invariance: more padded positions with arbitrary ids behind them change nothing
    tok2 = np.concatenate([tok, rng.integers(1, 20, (3, 2))], axis=1)
    seg2 = np.concatenate([seg, np.ones((3, 2), dtype=np.int64)], axis=1)
    tl2 = []
    logits2 = orc.forward_batch_mt(tok2, seg2, lens, w, tasks, 2, 1e-12, token_logits_out=tl2)
    assert np.array_equal(logits2, logits) and np.array_equal(tl2[0][:, :10], tl[0], equal_nan=True)
    # masking: an active task's outputs do not depend on the others
    tl3 = []
    part = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12, task_mask=0b1010, token_logits_out=tl3)
    assert np.all(np.isnan(part)) and np.array_equal(tl3[0], tl[0], equal_nan=True)
    tl4 = []
    part = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12, task_mask=0b0011, token_logits_out=tl4)
    assert np.array_equal(part[:, :2], logits[:, :2]) and np.all(np.isnan(part[:, 2:]))
    assert np.array_equal(tl4[0][..., :3], tl[0][..., :3], equal_nan=True) and np.all(np.isnan(tl4[0][..., 3:]))


# ---------------------------------------------------------------------------
# the merged tree: the paper's claims
# ---------------------------------------------------------------------------

def _inputs(rng, B, S, vocab, lens):
    tok = rng.integers(1, vocab, (B, S))
    seg = (np.arange(S)[None, :] >= (np.asarray(lens)[:, None] + 1) // 2).astype(np.int64)
    return tok, seg, np.asarray(lens)


def test_merged_equals_standalone_students():
    """Merging only shares the frozen layers' evaluation (Section 3.3): every
    task's output equals that of its stand-alone student."""
    rng = np.random.default_rng(9)
    w, tasks = tiny_model(rng)
    tok, seg, lens = _inputs(rng, 3, 10, 20, [10, 4, 1])
    for b in range(3):
        mt = orc.forward_sequence_mt(tok[b], seg[b], lens[b], w, tasks, 2, 1e-12)
        for t in range(len(tasks)):
            st = orc.forward_sequence_st(tok[b], seg[b], lens[b], w, t, tasks, 2, 1e-12)
            assert mt[t].shape == (tasks[t][2],)
            assert np.max(np.abs(mt[t] - st)) <= 1e-12


def test_modularity_and_masking():
    """Changing one task leaves the others untouched (Sections 1 and 5.1), and
    a task's output does not depend on which other tasks are active."""
    rng = np.random.default_rng(10)
    w, tasks = tiny_model(rng)
    tok, seg, lens = _inputs(rng, 2, 9, 20, [9, 5])
    base = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12)
    w2 = dict(w)
    w2["tasks"] = list(w["tasks"])
    w2["tasks"][1] = tiny_model(np.random.default_rng(99))[0]["tasks"][1]
    changed = orc.forward_batch_mt(tok, seg, lens, w2, tasks, 2, 1e-12)
    offs = np.concatenate([[0], np.cumsum([c for _, _, c in tasks])])
    for t in range(len(tasks)):
        cols = slice(offs[t], offs[t + 1])
        if t == 1:
            assert np.max(np.abs(base[:, cols] - changed[:, cols])) > 1e-3
        else:
            assert np.array_equal(base[:, cols], changed[:, cols])
    for mask in (0b0001, 0b0100, 0b1010, 0b0111):
        part = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12, task_mask=mask)
        for t in range(len(tasks)):
            cols = slice(offs[t], offs[t + 1])
            if (mask >> t) & 1:
                assert np.array_equal(part[:, cols], base[:, cols])
            else:
                assert np.all(np.isnan(part[:, cols]))
    with pytest.raises(ValueError):
        orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12, task_mask=0)


def test_padding_invariance_and_batch_permutation():
    rng = np.random.default_rng(11)
    w, tasks = tiny_model(rng)
    tok, seg, lens = _inputs(rng, 3, 6, 20, [6, 3, 2])
    base = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12)
    # pad to 12 with arbitrary ids/segments after the valid part
    tok2 = np.concatenate([tok, rng.integers(0, 20, (3, 6))], axis=1)
    seg2 = np.concatenate([seg, rng.integers(0, 2, (3, 6))], axis=1)
    for b in range(3):   # also scribble over the padded tail inside the original width
        tok2[b, lens[b]:] = rng.integers(0, 20, 12 - lens[b])
    assert np.array_equal(orc.forward_batch_mt(tok2, seg2, lens, w, tasks, 2, 1e-12), base)
    perm = [2, 0, 1]
    assert np.array_equal(orc.forward_batch_mt(tok[perm], seg[perm], lens[perm], w, tasks, 2, 1e-12), base[perm])
    sub = orc.forward_batch_mt(tok, seg, lens, w, tasks, 2, 1e-12, rows=[1])
    assert np.array_equal(sub[1], base[1]) and np.all(np.isnan(sub[[0, 2]]))


def test_hidden_snapshots_are_fork_states():
    rng = np.random.default_rng(12)
    w, tasks = tiny_model(rng)
    tok, seg, lens = _inputs(rng, 1, 7, 20, [7])
    hid = {}
    orc.forward_sequence_mt(tok[0], seg[0], 7, w, tasks, 2, 1e-12, hidden_out=hid)
    h = orc.embed(tok[0], seg[0], w["emb"], 1e-12)
    assert np.array_equal(hid[("trunk", 0)], h)
    for l in range(1, 5):
        h = orc.encoder_layer(h, w["trunk"][l - 1], 2, 1e-12)
        assert np.array_equal(hid[("trunk", l)], h)
    g = orc.encoder_layer(hid[("trunk", 4)], w["tasks"][1]["layers"][0], 2, 1e-12)
    assert np.array_equal(hid[("task", 1, 1)], g)


def read_paper_layer_counts():
    rows = []
    with open(os.path.join(GOLDEN, "paper_layer_counts.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, total, pairs = [p.strip() for p in line.split("|")]
            xy = [(int(a), int(b)) for a, b in re.findall(r"\((\d+),(\d+)\)", pairs)]
            rows.append((name, int(total), xy))
    return rows


@pytest.mark.parametrize("name,total,xy", read_paper_layer_counts())
def test_executed_layers_match_paper_tables(name, total, xy):
    """Tables 2 and 4 print the number of transformer layers evaluated for all
    eight tasks; the merged evaluation must run exactly that many."""
    assert len(xy) == 8
    tasks = [(x, y, 2) for x, y in xy]
    assert orc.overhead_layers(tasks) == total
    rng = np.random.default_rng(13)
    w, _ = tiny_model(rng, trunk=12, tasks=tasks)
    tok, seg, lens = _inputs(rng, 1, 3, 20, [3])
    c = orc.LayerCounter()
    orc.forward_sequence_mt(tok[0], seg[0], 3, w, tasks, 2, 1e-12, counter=c)
    assert c.count == total
    # the stand-alone students together cost sum(x + y): sharing is the saving
    c2 = orc.LayerCounter()
    for t in range(8):
        orc.forward_sequence_st(tok[0], seg[0], 3, w, t, tasks, 2, 1e-12, counter=c2)
    assert c2.count == sum(x + y for x, y in xy)


def test_trunk_stops_at_deepest_active_fork():
    rng = np.random.default_rng(14)
    w, tasks = tiny_model(rng)   # forks at 2, 4, 0, 3
    tok, seg, lens = _inputs(rng, 1, 4, 20, [4])
    for mask, want in ((0b0100, 0 + 1), (0b0001, 2 + 1), (0b1001, 3 + 1 + 0), (0b1111, 4 + 1 + 2 + 1 + 0)):
        c = orc.LayerCounter()
        orc.forward_sequence_mt(tok[0], seg[0], 4, w, tasks, 2, 1e-12, task_mask=mask, counter=c)
        assert c.count == want == orc.overhead_layers(tasks, mask)


# ---------------------------------------------------------------------------
# the seeded generator (no method arithmetic, but both sides depend on it)
# ---------------------------------------------------------------------------

def test_synth_bf16_and_statistics():
    x = np.array([1.0, 1.00390625, 1.005859375, -2.5, 0.0, 3.0e-5], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f64(bits)
    assert back[0] == 1.0 and back[3] == -2.5 and back[4] == 0.0
    assert back[1] == 1.0            # exactly half-way between 1.0 and 1.0078125: ties to even
    assert back[2] == 1.0078125      # above half-way: rounds up
    z = synth.standard_normal(0, "probe", 200000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    assert abs(np.mean(z ** 3)) < 0.03 and abs(np.mean(z ** 4) - 3) < 0.06
    assert np.array_equal(z[:10], synth.standard_normal(0, "probe", 10))
    assert not np.array_equal(z[:10], synth.standard_normal(1, "probe", 10))
    assert not np.array_equal(z[:10], synth.standard_normal(0, "probe2", 10))


def test_synth_batches_follow_the_recipe():
    cfg = synth.config_glue8()
    assert [t.fork_depth for t in cfg.tasks] == [7, 7, 6, 6, 5, 7, 4, 8]
    b = synth.batch_glue8(cfg)
    assert b.token_ids.shape == (32, 128) and b.lengths.min() >= 16 and b.lengths.max() <= 128
    valid = np.arange(128)[None, :] < b.lengths[:, None]
    assert np.all(b.token_ids[valid] >= 1000) and np.all(b.token_ids[valid] < 30522)
    assert np.all(b.token_ids[~valid] == 0) and np.all(b.segment_ids[~valid] == 0)
    for i in range(32):
        n = b.lengths[i]
        assert np.all(b.segment_ids[i, :(n + 1) // 2] == 0) and np.all(b.segment_ids[i, (n + 1) // 2:n] == 1)
    t = synth.batch_tiny(synth.config_tiny())
    assert np.all(t.lengths == 32) and np.all(t.segment_ids[:, :16] == 0) and np.all(t.segment_ids[:, 16:] == 1)
