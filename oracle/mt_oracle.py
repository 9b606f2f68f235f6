"""fp64 CPU oracle of the merged multi-task BERT forward pass.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the CUDA path, imports
nothing from it, and must never be called from the product path: only tests,
the smoke check and the benchmark's CPU-baseline leg use it.

What it computes (paper Section 3.3 and Fig. 1(c)): several single-task
student models, each made of ``x`` frozen bottom layers of the pre-trained
encoder plus ``y`` task-specific layers (Table 2's ``(x, y)`` notation), are
merged into one graph in which the frozen layers are evaluated once and shared.
Each task reads the trunk state after its own depth ("different tasks may be
fed with representations from different layers", Section 5.1), runs its own
layers, and emits its own output; one request yields every task's output
(Section 5.2).  The encoder itself is the 12-layer uncased BERT of Section 3:
the paper cites it and prints no formula, so the layer below is the published
post-LayerNorm transformer encoder layer with learned absolute positions,
erf-GELU, biased-variance LayerNorm, a tanh pooler on position 0 and a linear
head.  Readings taken where the paper is silent:

* padded keys are excluded from the softmax (weight exactly 0) and padded rows
  are never computed, so the oracle works on the ``n`` valid rows only;
* the pooler reads row 0 whatever token sits there; heads return raw logits
  (the regression task is a 1-wide head with no activation);
* ``fork_depth`` 0 forks off the embedding output; ``branch_layers`` 0 pools
  the trunk state directly; the trunk runs to the deepest fork among the
  *active* tasks only.

All arithmetic is float64 with no intermediate rounding.  Weights arrive as
float64 arrays (bf16 values widened exactly by the caller), ``W`` stored
``[out, in]`` so a linear map is ``x @ W.T + b``.

Pins (tests/test_oracle_pins.py): softmax rows sum to 1 / closed forms;
LayerNorm moments and a hand-computed row; GELU identities; linear+attention
against independently ordered scalar loops on tiny shapes; layer with zeroed
output projections reduces to LN(LN(h)); padding invariance; batch
permutation; merged == stand-alone per task; modularity; task masking; and the
executed-layer counts printed in the paper's Tables 2 and 4.
End-to-end logits for given inputs are printed nowhere in the paper:
PARITY UNPINNED for whole-model values beyond the composition of those parts.
"""
from __future__ import annotations

from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf  # library primitive: the error function


# ---------------------------------------------------------------------------
# elementary pieces
# ---------------------------------------------------------------------------

def layer_norm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    """LN over the last axis: gamma * (x - mean) / sqrt(var + eps) + beta with
    the biased variance (divide by the width)."""
    x = np.asarray(x, dtype=np.float64)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return gamma * ((x - mu) / np.sqrt(var + eps)) + beta


def gelu(x: np.ndarray) -> np.ndarray:
    """Exact GELU: x * Phi(x) with Phi the standard normal CDF."""
    x = np.asarray(x, dtype=np.float64)
    return x * 0.5 * (1.0 + erf(x / np.sqrt(2.0)))


def softmax_rows(s: np.ndarray) -> np.ndarray:
    """Row-wise softmax with the row maximum subtracted first."""
    s = np.asarray(s, dtype=np.float64)
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def linear(x: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """y = x W^T + b, W stored [out, in]."""
    return x @ w.T + b


def attention(h: np.ndarray, layer: Dict[str, np.ndarray], heads: int) -> np.ndarray:
    """Multi-head self-attention context over the valid rows ``h`` [n, H]
    (no key beyond n exists here, which is the padding mask)."""
    n, H = h.shape
    dh = H // heads
    q = linear(h, layer["wq"], layer["bq"])
    k = linear(h, layer["wk"], layer["bk"])
    v = linear(h, layer["wv"], layer["bv"])
    ctx = np.empty((n, H), dtype=np.float64)
    for a in range(heads):
        cols = slice(a * dh, (a + 1) * dh)
        scores = (q[:, cols] @ k[:, cols].T) / np.sqrt(float(dh))
        ctx[:, cols] = softmax_rows(scores) @ v[:, cols]
    return ctx


def encoder_layer(h: np.ndarray, layer: Dict[str, np.ndarray], heads: int, eps: float) -> np.ndarray:
    """One post-LN transformer encoder layer on valid rows [n, H]."""
    ctx = attention(h, layer, heads)
    h1 = layer_norm(h + linear(ctx, layer["wo"], layer["bo"]), layer["ln1_g"], layer["ln1_b"], eps)
    f = gelu(linear(h1, layer["w1"], layer["b1"]))
    return layer_norm(h1 + linear(f, layer["w2"], layer["b2"]), layer["ln2_g"], layer["ln2_b"], eps)


def embed(tokens: np.ndarray, segments: np.ndarray, emb: Dict[str, np.ndarray], eps: float) -> np.ndarray:
    """h0_i = LN(E_word[tok_i] + E_pos[i] + E_type[seg_i]) for the rows given."""
    n = len(tokens)
    e = emb["word"][tokens] + emb["pos"][np.arange(n)] + emb["type"][segments]
    return layer_norm(e, emb["ln_g"], emb["ln_b"], eps)


def pooler_head(g: np.ndarray, task_w: Dict[str, np.ndarray]) -> np.ndarray:
    """logits = W_c tanh(W_p g_0 + b_p) + b_c on row 0 of the final state."""
    pooled = np.tanh(linear(g[0], task_w["pool_w"], task_w["pool_b"]))
    return linear(pooled, task_w["cls_w"], task_w["cls_b"])


def token_head(g: np.ndarray, task_w: Dict[str, np.ndarray]) -> np.ndarray:
    """Token-level task (the production system of Appendix E serves token-level tasks beside the
    sequence-level ones and gives no formula for their output layer): the plain reading, one linear
    map on every token's final state, logits_i = W_c g_i + b_c, no pooler.  Returns [n, C]."""
    return linear(g, task_w["cls_w"], task_w["cls_b"])


# ---------------------------------------------------------------------------
# the merged tree (Fig. 1(c)) and the stand-alone students (Fig. 1(b))
# ---------------------------------------------------------------------------

# (fork_depth x, branch_layers y, num_classes) or, with a head kind, (x, y, num_classes, kind):
# kind 0 = sequence-level head (pooler on the first token + linear), kind 1 = token-level head.
TaskTriple = Tuple[int, ...]


def head_kind(task: TaskTriple) -> int:
    return int(task[3]) if len(task) > 3 else 0


def active_tasks(n_tasks: int, task_mask: Optional[int]) -> List[int]:
    if task_mask is None:
        return list(range(n_tasks))
    return [t for t in range(n_tasks) if (task_mask >> t) & 1]


def overhead_layers(tasks: Sequence[TaskTriple], task_mask: Optional[int] = None) -> int:
    """Transformer layers the merged model evaluates: the shared trunk up to
    the deepest fork plus every task's own layers (Table 2's "Layers" column,
    e.g. 7 + 2 x 8)."""
    act = active_tasks(len(tasks), task_mask)
    return max(tasks[t][0] for t in act) + sum(tasks[t][1] for t in act)


class LayerCounter:
    """Counts encoder_layer evaluations so tests can compare with the paper."""

    def __init__(self) -> None:
        self.count = 0


def forward_sequence_mt(tokens: np.ndarray, segments: np.ndarray, n: int, weights: Dict,
                        tasks: Sequence[TaskTriple], heads: int, eps: float,
                        task_mask: Optional[int] = None, hidden_out: Optional[Dict] = None,
                        counter: Optional[LayerCounter] = None, layer_fn=None) -> Dict[int, np.ndarray]:
    """Merged multi-task forward of ONE sequence with ``n`` valid tokens.

    The trunk is evaluated once up to D = max fork depth over the active
    tasks; the state after each depth some active task forks at is kept; then
    each active task runs its branch from its fork state.  Returns
    {task: logits[C_t]}.  ``hidden_out`` (if given) receives
    ("trunk", depth) -> [n, H] for every depth 0..D and ("task", t, j) ->
    [n, H] after branch layer j (1-based) of task t.  ``layer_fn`` replaces encoder_layer (same
    signature) for variants of the layer arithmetic, such as the reduced-precision one."""
    layer_fn = layer_fn or encoder_layer
    act = active_tasks(len(tasks), task_mask)
    if not act:
        raise ValueError("task_mask selects no task")
    tok = np.asarray(tokens[:n], dtype=np.int64)
    seg = np.asarray(segments[:n], dtype=np.int64)
    depth = max(tasks[t][0] for t in act)
    fork_depths = {tasks[t][0] for t in act}

    h = embed(tok, seg, weights["emb"], eps)
    forks = {}
    if 0 in fork_depths:
        forks[0] = h
    if hidden_out is not None:
        hidden_out[("trunk", 0)] = h
    for l in range(1, depth + 1):
        h = layer_fn(h, weights["trunk"][l - 1], heads, eps)
        if counter is not None:
            counter.count += 1
        if l in fork_depths:
            forks[l] = h
        if hidden_out is not None:
            hidden_out[("trunk", l)] = h

    out = {}
    for t in act:
        x, y = tasks[t][0], tasks[t][1]
        g = forks[x]
        for j in range(1, y + 1):
            g = layer_fn(g, weights["tasks"][t]["layers"][j - 1], heads, eps)
            if counter is not None:
                counter.count += 1
            if hidden_out is not None:
                hidden_out[("task", t, j)] = g
        out[t] = token_head(g, weights["tasks"][t]) if head_kind(tasks[t]) == 1 else pooler_head(g, weights["tasks"][t])
    return out


def forward_sequence_st(tokens: np.ndarray, segments: np.ndarray, n: int, weights: Dict,
                        task: int, tasks: Sequence[TaskTriple], heads: int, eps: float,
                        counter: Optional[LayerCounter] = None) -> np.ndarray:
    """The stand-alone student of ``task`` run by itself: its x frozen layers,
    then its y task layers, then its head.  Deliberately written as its own
    straight-line loop, sharing no state with the merged evaluation."""
    x, y = tasks[task][0], tasks[task][1]
    g = embed(np.asarray(tokens[:n], dtype=np.int64), np.asarray(segments[:n], dtype=np.int64),
              weights["emb"], eps)
    chain = [weights["trunk"][l] for l in range(x)] + [weights["tasks"][task]["layers"][j] for j in range(y)]
    for layer in chain:
        g = encoder_layer(g, layer, heads, eps)
        if counter is not None:
            counter.count += 1
    if head_kind(tasks[task]) == 1:
        return token_head(g, weights["tasks"][task])
    return pooler_head(g, weights["tasks"][task])


def forward_batch_mt(token_ids: np.ndarray, segment_ids: np.ndarray, lengths: np.ndarray, weights: Dict,
                     tasks: Sequence[TaskTriple], heads: int, eps: float,
                     task_mask: Optional[int] = None, rows: Optional[Iterable[int]] = None,
                     hidden_out: Optional[List[Dict]] = None,
                     token_logits_out: Optional[List[np.ndarray]] = None, layer_fn=None) -> np.ndarray:
    """Merged forward of a padded batch.  Returns float64 logits
    [B, sum C_t over the sequence-level tasks]; task t occupies columns
    [off_t, off_t + C_t); columns of inactive tasks and rows not in ``rows``
    are NaN.  Token-level tasks have columns of their own, counted over the
    token-level tasks only, in a [B, S, sum C_t] array appended to
    ``token_logits_out`` (NaN at positions >= length, for inactive tasks and
    for rows not selected).  Sequences are independent, so ``rows`` selects an
    exact subset."""
    B, S = token_ids.shape
    seq_c = [0 if head_kind(t) == 1 else t[2] for t in tasks]
    tok_c = [t[2] if head_kind(t) == 1 else 0 for t in tasks]
    offs = np.concatenate([[0], np.cumsum(seq_c)]).astype(int)
    tok_offs = np.concatenate([[0], np.cumsum(tok_c)]).astype(int)
    logits = np.full((B, offs[-1]), np.nan, dtype=np.float64)
    token_logits = np.full((B, S, tok_offs[-1]), np.nan, dtype=np.float64)
    for b in (range(B) if rows is None else rows):
        hid = {} if hidden_out is not None else None
        res = forward_sequence_mt(token_ids[b], segment_ids[b], int(lengths[b]), weights, tasks, heads, eps,
                                  task_mask=task_mask, hidden_out=hid, layer_fn=layer_fn)
        for t, lg in res.items():
            if head_kind(tasks[t]) == 1:
                token_logits[b, :lg.shape[0], tok_offs[t]:tok_offs[t + 1]] = lg
            else:
                logits[b, offs[t]:offs[t + 1]] = lg
        if hidden_out is not None:
            hidden_out.append(hid)
    if token_logits_out is not None:
        token_logits_out.append(token_logits)
    return logits
