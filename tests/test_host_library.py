"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
declared symbol, validates its arguments, sizes its blobs like the generator packs
them, and schedules exactly the layer totals the paper prints (Tables 2 and 4)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2107_05377_b200 import binding, build, synth
from test_oracle_pins import read_paper_layer_counts

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mt_bert.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mt_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/mt_bert.h but not exported"
        assert n in binding.SIGNATURES, f"{n} has no binding signature"
    assert sorted(binding.SIGNATURES) == names


def small_cfg(tasks, trunk_layers=12):
    return synth.TreeConfig(vocab_size=64, max_position=64, trunk_layers=trunk_layers,
                            tasks=tuple(synth.TaskSpec(*t) for t in tasks))


@pytest.mark.parametrize("name,total,xy", read_paper_layer_counts())
def test_scheduler_runs_the_papers_layer_totals(lib, name, total, xy):
    cfg = small_cfg([(x, y, 2) for x, y in xy])
    m = binding.MTModel(cfg, 4, 32, bind=False)
    s = m.plan_summary(m.full_mask())
    assert s["layers"] == total
    assert s["trunk_depth"] == max(x for x, _ in xy)
    assert sum(s["groups_per_wave"]) == total
    assert s["waves"] == max(x + y for x, y in xy)
    # wave w holds trunk layer w (if w <= depth) plus branch layer w - x of every task with x < w <= x + y
    for w in range(1, s["waves"] + 1):
        want = (1 if w <= s["trunk_depth"] else 0) + sum(1 for x, y in xy if x < w <= x + y)
        assert s["groups_per_wave"][w - 1] == want
    m.close()


def test_generator_paper_trees_are_the_golden_ones(lib):
    """The (x, y) lists the serving sweep runs (synth.PAPER_TREES) are those of the golden file, in its order,
    and the library schedules the printed layer totals for them."""
    golden = read_paper_layer_counts()
    assert [xy for _, _, xy in golden] == list(synth.PAPER_TREES.values())
    for (_, total, _), name in zip(golden, synth.PAPER_TREES):
        m = binding.MTModel(synth.config_paper_tree(name), 2, 32, bind=False)
        assert m.plan_summary(0xFF)["layers"] == total
        m.close()


def test_scheduler_masks_and_wavefront_of_the_8_task_tree(lib):
    cfg = synth.config_glue8()
    m = binding.MTModel(cfg, 32, 128, bind=False)
    s = m.plan_summary(0xFF)
    assert s == {"layers": 24, "waves": 10, "trunk_depth": 8, "groups_per_wave": [1, 1, 1, 1, 2, 3, 5, 6, 3, 1]}
    only6 = m.plan_summary(1 << 6)           # forks at 4, three branch layers
    assert only6["layers"] == 7 and only6["trunk_depth"] == 4 and only6["groups_per_wave"] == [1] * 7
    only7 = m.plan_summary(1 << 7)           # forks at 8, two branch layers
    assert only7["layers"] == 10 and only7["trunk_depth"] == 8
    for mask in (0b00010010, 0b10100101, 0b01000000):
        act = [t for t in range(8) if (mask >> t) & 1]
        want = max(cfg.tasks[t].fork_depth for t in act) + sum(cfg.tasks[t].branch_layers for t in act)
        assert m.plan_summary(mask)["layers"] == want
    with pytest.raises(binding.MTError):
        m.plan_summary(0)
    # fused_ln = 1: each residual GEMM carries the LayerNorm after it, so a layer on all tokens is 5 launches
    # (projection, attention, output + LN, FFN up, FFN down + LN), a first-token tail 4: its 32 rows per layer are
    # few enough for the FFN-down projection to be split over K, which keeps its LayerNorm as a launch of its own
    m.set_option("fused_ln", 1)
    assert m.plan_launches(0xFF) == 2 + 5 * 6 + 6 * 3 + 2 + 4 + 2
    m.set_option("ffn_down_split", 0)
    assert m.plan_launches(0xFF) == 2 + 5 * 6 + 6 * 3 + 2 + 3 + 2
    m.set_option("ffn_down_split", 1)
    # default (2): where at most two layers are on all tokens: waves 1-5 and wave 9
    m.set_option("fused_ln", 2)
    assert m.plan_launches(0xFF) == 2 + 5 * 4 + 5 + 7 + 8 + 8 + 6 + 2 + 5 + 2
    m.set_option("fused_ln_max_rows", 128)   # also the first-token tail (32 rows per layer)
    assert m.plan_launches(0xFF) == 2 + 5 * 4 + 5 + 7 + 8 + 8 + 6 + 2 + 4 + 2
    m.set_option("fused_ln", 3)
    assert m.plan_launches(0xFF) == 2 + 5 * 6 + 6 * 3 + 2 + 4 + 2
    m.set_option("fused_ln", 0)
    # waves 7, 8, 9 mix layers on all tokens (7 launches) with last branch layers, which only add the
    # first-token attention there; wave 10 holds a last layer alone (projection + first-token attention);
    # the rest of the eight last layers is one grouped pass of 5 launches before the pooler/head pair
    assert m.plan_launches(0xFF) == 2 + 7 * 4 + 7 + 7 + 8 + 8 + 8 + 2 + 5 + 2
    m.set_option("cls_only_last_layer", 0)
    assert m.plan_launches(0xFF) == 2 + 7 * 10 + 2   # row starts + embedding, 7 per wave, pooler + head at the end
    # early_heads: tasks finish after waves 7 (2 tasks), 8 (3), 9 (2), 10 (1): four pooler + head pairs, and
    # with first-token-only last layers four grouped tails of 5 launches instead of one
    m.set_option("early_heads", 1)
    assert m.plan_launches(0xFF) == 2 + 7 * 10 + 2 * 4
    m.set_option("cls_only_last_layer", 1)
    assert m.plan_launches(0xFF) == 2 + 7 * 4 + 7 + 7 + 8 + 8 + 8 + 2 + 5 * 4 + 2 * 4
    m.close()
    m2 = binding.MTModel(cfg, 32, 128, max_groups=2, bind=False)
    m2.set_option("cls_only_last_layer", 0)
    m2.set_option("fused_ln", 0)
    assert m2.plan_summary(0xFF)["layers"] == 24
    assert m2.plan_launches(0xFF) == 2 + 7 * (1 + 1 + 1 + 1 + 1 + 2 + 3 + 3 + 2 + 1) + 2
    m2.close()


def test_token_level_tasks_in_the_plan(lib):
    """A token-level task needs every row of its last layer (no first-token shortcut) and gets its head,
    one launch, right after the wave that completes it; sequence-level tasks are planned as before."""
    seq_only = small_cfg([(2, 2, 2), (1, 1, 3)], trunk_layers=2)
    mixed = synth.TreeConfig(trunk_layers=2, tasks=(synth.TaskSpec(2, 2, 2), synth.TaskSpec(1, 1, 3, token_level=True)))
    assert mixed.total_classes == 2 and mixed.total_token_classes == 3 and mixed.logit_offsets == [0, 0]
    a = binding.MTModel(seq_only, 2, 32, bind=False)
    b = binding.MTModel(mixed, 2, 32, bind=False)
    for m in (a, b):
        m.set_option("fused_ln", 0)
    assert a.plan_summary(0b11) == b.plan_summary(0b11)
    # wave 1: trunk (7); wave 2: trunk + the last layer of task 1: first tokens only (7 + first-token attention),
    # or all tokens for the token-level task (7, two groups); wave 3, 4: task 0 (7, then projection + first-token
    # attention); first-token tails: 5 per tail launch; heads: pooler GEMM + head = 2, token-level head = 1
    assert a.plan_launches(0b11) == 2 + 7 + 8 + 7 + 2 + 5 + 2
    assert b.plan_launches(0b11) == 2 + 7 + 7 + 1 + 7 + 2 + 5 + 2
    assert b.plan_launches(0b10) == 2 + 7 + 7 + 1
    a.close()
    b.close()


def test_create_rejects_bad_configurations(lib):
    def create(trunk_kw=None, tasks=((4, 1, 2),), max_batch=2, max_seq=32):
        kw = dict(vocab_size=64, max_position=64, type_vocab=2, hidden=768, heads=12, ffn=3072, trunk_layers=4,
                  ln_eps=1e-12, activation=0)
        kw.update(trunk_kw or {})
        trunk = binding.TrunkConfig(**kw)
        arr = (binding.TaskConfig * len(tasks))(*[binding.TaskConfig(*t) for t in tasks])
        h = C.c_void_p()
        rc = lib.mt_create(C.byref(trunk), arr, len(tasks), max_batch, max_seq, C.byref(h))
        if rc == 0:
            lib.mt_destroy(h)
        return rc

    assert create() == 0
    assert create(tasks=((5, 1, 2),)) == -1            # fork beyond the trunk
    assert create(tasks=((4, -1, 2),)) == -1
    assert create(tasks=((4, 1, 0),)) == -1
    assert create(tasks=((0, 0, 1),)) == 0              # fork at the embeddings, no branch, regression head
    assert create(tasks=((4, 1, 5, 1),)) == 0           # token-level head
    assert create(tasks=((4, 1, 5, 2),)) == -1          # unknown head kind
    assert create({"hidden": 512, "heads": 8}) == -7    # width not implemented
    assert create({"heads": 8}) == -7                   # head width != 64
    assert create({"activation": 1}) == -7
    assert create(max_seq=1024) == -7
    assert create({"max_position": 16}) == -1           # max_seq beyond the position table
    assert create(max_batch=0) == -1
    h = C.c_void_p()
    assert lib.mt_create(None, None, 1, 1, 1, C.byref(h)) == -1


def test_unbound_model_fails_loudly(lib):
    cfg = small_cfg([(1, 1, 2)], trunk_layers=1)
    m = binding.MTModel(cfg, 2, 32, bind=False)
    blob = np.zeros(m.blob_bytes(), dtype=np.uint8)
    assert lib.mt_load_weights(m.handle, blob.ctypes.data, blob.size, None) == -3
    assert lib.mt_forward(m.handle, 1, 1, 1, 1, 2, 32, 1, None) == -3
    assert lib.mt_forward(m.handle, 1, 1, 1, 1, 4, 32, 1, None) == -2      # batch beyond max_batch
    assert lib.mt_forward(m.handle, None, 1, 1, 1, 2, 32, 1, None) == -1
    assert b"mt_bind_memory" in lib.mt_last_error_string(m.handle) or True
    m.close()


def test_blob_sizes_match_the_generator(lib):
    cfg = small_cfg([(1, 1, 2), (0, 0, 1), (1, 2, 3)], trunk_layers=1)
    m = binding.MTModel(cfg, 2, 32, bind=False)
    w = synth.make_weights(cfg, seed=3)
    blob = synth.pack_weights(cfg, w)
    assert blob.size == m.blob_bytes() == m.weights_bytes() + 256
    for t in range(3):
        tb = synth.pack_task_weights(cfg, t, w["tasks"][t])
        assert tb.size == m.task_blob_bytes(t)
    assert m.task_blob_bytes(3) == 0
    assert m.workspace_bytes() > 0
    before = m.workspace_bytes()
    m.set_option("debug_capture", 1)
    assert m.workspace_bytes() > before
    with pytest.raises(binding.MTError):
        m.set_option("max_groups", 9)
    with pytest.raises(binding.MTError):
        m.set_option("nonsense", 1)
    m.close()
