"""Seeded synthetic weights and inputs for the merged multi-task BERT tree.

This module holds no arithmetic of the method itself: it only draws random
numbers, rounds them to bf16, names tensors and packs them into the weight
blob that ``mt_load_weights`` accepts.  Both the CUDA path and the fp64 test
oracle are fed from here, so that they see exactly the same values.

Every element is a pure function of ``(seed, tensor name, flat index)`` through
a counter-based generator (a splitmix64-style finaliser followed by the
Box-Muller transform), so any tensor can be regenerated in isolation.

The paper serves eight GLUE tasks on top of 12-layer uncased BERT-base
(Section 3; Table 2's ``(x, y)`` = (frozen layers, task layers) notation).
Neither GLUE nor the pre-trained checkpoint is used here: weights are
N(0, 0.02) rounded to bf16 and token ids are uniform, with the shapes of that
set-up.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------
# configuration
# --------------------------------------------------------------------------


@dataclass(frozen=True)
class TaskSpec:
    """One task of the tree: forks after trunk layer ``fork_depth`` (0 = the
    embedding output), runs ``branch_layers`` task-specific layers, and ends in
    a pooler plus a linear head with ``num_classes`` outputs - or, with
    ``token_level``, in a linear head applied to every token's final state."""

    fork_depth: int
    branch_layers: int
    num_classes: int
    token_level: bool = False


@dataclass(frozen=True)
class TreeConfig:
    hidden: int = 768
    heads: int = 12
    ffn: int = 3072
    trunk_layers: int = 12
    vocab_size: int = 30522
    max_position: int = 512
    type_vocab: int = 2
    ln_eps: float = 1e-12
    tasks: Tuple[TaskSpec, ...] = field(default_factory=tuple)

    @property
    def n_tasks(self) -> int:
        return len(self.tasks)

    @property
    def logit_offsets(self) -> List[int]:
        """First column of every task in its output array: sequence-level tasks are counted among
        themselves ([B, total_classes]), token-level tasks among themselves ([B, S, total_token_classes])."""
        offs, acc, acc_tok = [], 0, 0
        for t in self.tasks:
            if t.token_level:
                offs.append(acc_tok)
                acc_tok += t.num_classes
            else:
                offs.append(acc)
                acc += t.num_classes
        return offs

    @property
    def total_classes(self) -> int:
        return sum(t.num_classes for t in self.tasks if not t.token_level)

    @property
    def total_token_classes(self) -> int:
        return sum(t.num_classes for t in self.tasks if t.token_level)


def _tasks(depths: Sequence[int], branches: Sequence[int], classes: Sequence[int]) -> Tuple[TaskSpec, ...]:
    return tuple(TaskSpec(int(d), int(k), int(c)) for d, k, c in zip(depths, branches, classes))


def config_tiny() -> TreeConfig:
    """Two tasks fork at trunk layer 4 of a 4-layer trunk, one branch layer each."""
    return TreeConfig(trunk_layers=4, tasks=_tasks([4, 4], [1, 1], [2, 3]))


def config_glue8() -> TreeConfig:
    """Eight tasks on a 12-layer BERT-base trunk; task t fine-tuned L_t top
    layers, so it forks after trunk layer 12 - L_t, L = {5,5,6,6,7,5,8,4}."""
    L = [5, 5, 6, 6, 7, 5, 8, 4]
    return TreeConfig(tasks=_tasks([12 - x for x in L], [2, 1, 3, 2, 2, 1, 3, 2], [2, 2, 2, 3, 2, 2, 2, 1]))


def config_large8() -> TreeConfig:
    """BERT-large width: 24-layer trunk, H=1024, 16 heads, FFN 4096."""
    return TreeConfig(hidden=1024, heads=16, ffn=4096, trunk_layers=24,
                      tasks=_tasks([18, 17, 16, 15, 14, 13, 12, 16], [2] * 8, [2, 2, 2, 3, 2, 2, 2, 3]))


# The (x, y) = (frozen layers, task layers) lists of the merged models whose layer totals the paper prints
# (Table 2; Table 4 for c = 2, 3), tasks in the order QNLI RTE QQP MNLI SST-2 MRPC CoLA STS-B.  The
# "KD-n" rows print only "7 + n x 8"; the per-task x is taken from the bracketed rows, where it is fixed
# before distillation.
PAPER_TREES = {
    "full fine-tuning, 8 models": [(0, 12)] * 8,
    "ours (KD-1)": [(2, 1), (7, 1), (2, 1), (4, 1), (6, 1), (7, 1), (4, 1), (4, 1)],
    "ours (KD-2)": [(2, 2), (7, 2), (2, 2), (4, 2), (6, 2), (7, 2), (4, 2), (4, 2)],
    "ours (KD-3)": [(2, 3), (7, 3), (2, 3), (4, 3), (6, 3), (7, 3), (4, 3), (4, 3)],
    "ours (w/o KD)": [(2, 10), (7, 5), (2, 10), (4, 8), (6, 6), (7, 5), (4, 8), (4, 8)],
    "ours (mixed, c = 1)": [(2, 3), (7, 5), (2, 1), (4, 3), (6, 2), (7, 3), (4, 8), (4, 1)],
    "ours (c = 2)": [(2, 2), (7, 1), (2, 1), (4, 2), (6, 2), (7, 1), (4, 3), (4, 1)],
    "ours (c = 3)": [(2, 1), (7, 1), (2, 1), (4, 2), (6, 1), (7, 1), (4, 3), (4, 1)],
}
GLUE_CLASSES = [2, 2, 2, 3, 2, 2, 2, 1]


def config_paper_tree(name: str) -> TreeConfig:
    """One of the paper's merged models as a tree over a BERT-base trunk that is as deep as its deepest fork."""
    xy = PAPER_TREES[name]
    return TreeConfig(trunk_layers=max(x for x, _ in xy),
                      tasks=_tasks([x for x, _ in xy], [y for _, y in xy], GLUE_CLASSES))


def config_production21() -> TreeConfig:
    """Shaped like the production model of Appendix E: 21 tasks on a BERT-base trunk, 8 shared layers and
    32 task layers in all (eleven branches of 2 layers, ten of 1).  Every third task is token-level (9
    tags, as a slot-filling or entity task would have), the others are sequence-level with 2-4 classes."""
    branches = [2 if t % 2 == 0 else 1 for t in range(21)]
    classes = [9 if t % 3 == 2 else 2 + t % 3 for t in range(21)]
    tasks = tuple(TaskSpec(8, branches[t], classes[t], token_level=(t % 3 == 2)) for t in range(21))
    return TreeConfig(tasks=tasks)


def config_single_task(base: TreeConfig, task: int) -> TreeConfig:
    """The stand-alone single-task model of ``task``: same trunk prefix, its
    branch alone (Fig. 1(b): one student before merging)."""
    return TreeConfig(hidden=base.hidden, heads=base.heads, ffn=base.ffn, trunk_layers=base.trunk_layers,
                      vocab_size=base.vocab_size, max_position=base.max_position, type_vocab=base.type_vocab,
                      ln_eps=base.ln_eps, tasks=(base.tasks[task],))


def config_full_depth_single(base: TreeConfig, num_classes: int) -> TreeConfig:
    """A conventional fully fine-tuned single-task model: every layer is the task's own, nothing
    is shared - (x, y) = (0, 12) in Table 2's notation; its "12 x 8" baseline is eight of these.
    No frozen trunk layer is loaded."""
    return TreeConfig(hidden=base.hidden, heads=base.heads, ffn=base.ffn, trunk_layers=0,
                      vocab_size=base.vocab_size, max_position=base.max_position, type_vocab=base.type_vocab,
                      ln_eps=base.ln_eps, tasks=(TaskSpec(0, base.trunk_layers, num_classes),))


# --------------------------------------------------------------------------
# counter-based random numbers
# --------------------------------------------------------------------------

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wraps modulo 2^64)."""
    z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
    return z ^ (z >> np.uint64(31))


def name_id(name: str) -> int:
    """FNV-1a 64-bit hash of a tensor name."""
    h = 0xCBF29CE484222325
    for ch in name.encode():
        h = ((h ^ ch) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def _stream_key(seed: int, name: str) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix64(np.array([(seed * 0x2545F4914F6CDD1D + name_id(name)) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    return k[0]


def raw_u64(seed: int, name: str, start: int, count: int) -> np.ndarray:
    """``count`` 64-bit draws of stream ``(seed, name)`` starting at index ``start``."""
    key = _stream_key(seed, name)
    with np.errstate(over="ignore"):
        ctr = np.arange(start, start + count, dtype=np.uint64)
        return _mix64(key ^ _mix64(ctr))


def uniform01(seed: int, name: str, start: int, count: int) -> np.ndarray:
    """Doubles in (0, 1): top 53 bits, offset by half an ulp so 0 never occurs."""
    r = raw_u64(seed, name, start, count)
    return ((r >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def standard_normal(seed: int, name: str, count: int) -> np.ndarray:
    """Box-Muller: draws 2i and 2i+1 of the stream give normals 2i (cosine
    branch) and 2i+1 (sine branch)."""
    pairs = (count + 1) // 2
    u = uniform01(seed, name, 0, 2 * pairs)
    r = np.sqrt(-2.0 * np.log(u[0::2]))
    theta = 2.0 * np.pi * u[1::2]
    z = np.empty(2 * pairs, dtype=np.float64)
    z[0::2] = r * np.cos(theta)
    z[1::2] = r * np.sin(theta)
    return z[:count]


def randint(seed: int, name: str, count: int, lo: int, hi_inclusive: int) -> np.ndarray:
    span = np.uint64(hi_inclusive - lo + 1)
    return (raw_u64(seed, name, 0, count) % span).astype(np.int64) + lo


# --------------------------------------------------------------------------
# bf16
# --------------------------------------------------------------------------


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))
    return (b >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# weights
# --------------------------------------------------------------------------

LAYER_TENSORS = ("wq", "wk", "wv", "bq", "bk", "bv", "wo", "bo", "ln1_g", "ln1_b",
                 "w1", "b1", "w2", "b2", "ln2_g", "ln2_b")


def layer_shapes(cfg: TreeConfig) -> Dict[str, Tuple[int, ...]]:
    H, F = cfg.hidden, cfg.ffn
    return {"wq": (H, H), "wk": (H, H), "wv": (H, H), "bq": (H,), "bk": (H,), "bv": (H,),
            "wo": (H, H), "bo": (H,), "ln1_g": (H,), "ln1_b": (H,),
            "w1": (F, H), "b1": (F,), "w2": (H, F), "b2": (H,), "ln2_g": (H,), "ln2_b": (H,)}


def _gen(seed: int, name: str, shape: Tuple[int, ...], std: float, mean: float = 0.0) -> np.ndarray:
    n = int(np.prod(shape))
    x = mean + std * standard_normal(seed, name, n)
    return f32_to_bf16_bits(x.astype(np.float32)).reshape(shape)


def _const(shape: Tuple[int, ...], value: float) -> np.ndarray:
    return f32_to_bf16_bits(np.full(shape, value, dtype=np.float32))


def make_layer(cfg: TreeConfig, seed: int, prefix: str, random_affine: bool) -> Dict[str, np.ndarray]:
    out = {}
    for name, shape in layer_shapes(cfg).items():
        full = f"{prefix}.{name}"
        if name.endswith("_g"):
            out[name] = _gen(seed, full, shape, 0.1, 1.0) if random_affine else _const(shape, 1.0)
        elif name.endswith("_b") and name.startswith("ln"):
            out[name] = _gen(seed, full, shape, 0.1) if random_affine else _const(shape, 0.0)
        else:
            out[name] = _gen(seed, full, shape, 0.02)
    return out


def make_task_weights(cfg: TreeConfig, task: int, seed: int, random_affine: bool = False) -> Dict:
    """Branch layers, pooler and head of one task (bf16 bit patterns)."""
    spec = cfg.tasks[task]
    H = cfg.hidden
    p = f"task{task}"
    return {
        "layers": [make_layer(cfg, seed, f"{p}.layer{j}", random_affine) for j in range(spec.branch_layers)],
        "pool_w": _gen(seed, f"{p}.pool_w", (H, H), 0.02),
        "pool_b": _gen(seed, f"{p}.pool_b", (H,), 0.02),
        "cls_w": _gen(seed, f"{p}.cls_w", (spec.num_classes, H), 0.02),
        "cls_b": _gen(seed, f"{p}.cls_b", (spec.num_classes,), 0.02),
    }


def make_weights(cfg: TreeConfig, seed: int = 0, random_affine: bool = False) -> Dict:
    """All tensors of the tree as bf16 bit patterns (uint16 arrays).

    Matrices, biases and embedding tables are N(0, 0.02).  LayerNorm gamma is 1
    and beta 0 unless ``random_affine`` (then gamma ~ N(1, 0.1), beta ~ N(0, 0.1)).
    The trunk does not depend on the task list, so a single-task configuration
    built from the same seed shares the merged tree's trunk (the frozen layers
    of every student are the pre-trained ones, Section 3.2-3.3)."""
    H = cfg.hidden
    emb = {
        "word": _gen(seed, "emb.word", (cfg.vocab_size, H), 0.02),
        "pos": _gen(seed, "emb.pos", (cfg.max_position, H), 0.02),
        "type": _gen(seed, "emb.type", (cfg.type_vocab, H), 0.02),
        "ln_g": _gen(seed, "emb.ln_g", (H,), 0.1, 1.0) if random_affine else _const((H,), 1.0),
        "ln_b": _gen(seed, "emb.ln_b", (H,), 0.1) if random_affine else _const((H,), 0.0),
    }
    trunk = [make_layer(cfg, seed, f"trunk.layer{l}", random_affine) for l in range(cfg.trunk_layers)]
    tasks = [make_task_weights(cfg, t, seed, random_affine) for t in range(cfg.n_tasks)]
    return {"emb": emb, "trunk": trunk, "tasks": tasks}


def select_task_weights(weights: Dict, task: int) -> Dict:
    """Weights of the stand-alone single-task model of ``task`` (same arrays)."""
    return {"emb": weights["emb"], "trunk": weights["trunk"], "tasks": [weights["tasks"][task]]}


def widen(weights):
    """bf16 bit patterns -> float64 arrays, same nesting."""
    if isinstance(weights, dict):
        return {k: widen(v) for k, v in weights.items()}
    if isinstance(weights, list):
        return [widen(v) for v in weights]
    return bf16_bits_to_f64(weights)


# --------------------------------------------------------------------------
# weight blob (the byte format mt_load_weights / mt_load_task_weights accept)
# --------------------------------------------------------------------------

BLOB_MAGIC = 0x4D544257  # "MTBW"
BLOB_VERSION = 1
BLOB_ALIGN = 256
BLOB_HEADER_BYTES = 256
KIND_FULL = 0
KIND_TASK = 1


def _pad(n: int) -> int:
    return (n + BLOB_ALIGN - 1) // BLOB_ALIGN * BLOB_ALIGN


def _append(chunks: List[bytes], arr: np.ndarray) -> None:
    raw = np.ascontiguousarray(arr, dtype=np.uint16).tobytes()
    chunks.append(raw)
    chunks.append(b"\0" * (_pad(len(raw)) - len(raw)))


def _append_layer(chunks: List[bytes], layer: Dict[str, np.ndarray]) -> None:
    for name in LAYER_TENSORS:
        _append(chunks, layer[name])


def _append_task(chunks: List[bytes], tw: Dict) -> None:
    for layer in tw["layers"]:
        _append_layer(chunks, layer)
    for name in ("pool_w", "pool_b", "cls_w", "cls_b"):
        _append(chunks, tw[name])


def _header(cfg: TreeConfig, kind: int, task_index: int, spec: TaskSpec | None, payload: int) -> bytes:
    d, k, c = (spec.fork_depth, spec.branch_layers, spec.num_classes) if spec else (0, 0, 0)
    h = struct.pack("<IIIiiiiiiiiiiiiiQ", BLOB_MAGIC, BLOB_VERSION, kind, cfg.hidden, cfg.heads, cfg.ffn,
                    cfg.trunk_layers, cfg.vocab_size, cfg.max_position, cfg.type_vocab,
                    cfg.n_tasks, task_index, d, k, c, 0, payload)
    return h + b"\0" * (BLOB_HEADER_BYTES - len(h))


def pack_weights(cfg: TreeConfig, weights: Dict) -> np.ndarray:
    """Full-model blob: header, then embeddings, trunk layers, then every
    task's section, each tensor bf16 and padded to 256 bytes."""
    chunks: List[bytes] = []
    for name in ("word", "pos", "type", "ln_g", "ln_b"):
        _append(chunks, weights["emb"][name])
    for layer in weights["trunk"]:
        _append_layer(chunks, layer)
    for tw in weights["tasks"]:
        _append_task(chunks, tw)
    body = b"".join(chunks)
    return np.frombuffer(_header(cfg, KIND_FULL, -1, None, len(body)) + body, dtype=np.uint8).copy()


def pack_task_weights(cfg: TreeConfig, task: int, tw: Dict) -> np.ndarray:
    """Single-task blob: header naming the task, then that task's section only."""
    chunks: List[bytes] = []
    _append_task(chunks, tw)
    body = b"".join(chunks)
    return np.frombuffer(_header(cfg, KIND_TASK, task, cfg.tasks[task], len(body)) + body, dtype=np.uint8).copy()


# --------------------------------------------------------------------------
# inputs
# --------------------------------------------------------------------------


@dataclass
class Batch:
    token_ids: np.ndarray    # int32 [B, S]; 0 at padded positions
    segment_ids: np.ndarray  # int32 [B, S]; 0 at padded positions
    lengths: np.ndarray      # int32 [B]


def make_batch(cfg: TreeConfig, batch: int, seq: int, len_lo: int, len_hi: int, seed: int = 1,
               split_at: int | None = None) -> Batch:
    """Token ids uniform in [1000, vocab) at valid positions; valid lengths
    uniform on the closed range [len_lo, len_hi]; segment 0 for the first half
    of each sequence (rounded up) and 1 for the rest, or split at ``split_at``."""
    lengths = randint(seed, "lengths", batch, len_lo, len_hi).astype(np.int32)
    tok = randint(seed, "token_ids", batch * seq, 1000, cfg.vocab_size - 1).astype(np.int32).reshape(batch, seq)
    pos = np.arange(seq, dtype=np.int32)[None, :]
    valid = pos < lengths[:, None]
    first = np.full((batch, 1), split_at, dtype=np.int32) if split_at is not None else ((lengths + 1) // 2)[:, None]
    seg = ((pos >= first) & valid).astype(np.int32)
    tok = np.where(valid, tok, 0).astype(np.int32)
    return Batch(tok, seg, lengths)


def batch_tiny(cfg: TreeConfig) -> Batch:
    """2 x 32, no padding, segment 0 for the first 16 tokens and 1 after."""
    return make_batch(cfg, 2, 32, 32, 32, seed=1, split_at=16)


def batch_glue8(cfg: TreeConfig, batch: int = 32, seq: int = 128, len_lo: int = 16, len_hi: int = 128,
                seed: int = 1) -> Batch:
    return make_batch(cfg, batch, seq, len_lo, len_hi, seed=seed)
