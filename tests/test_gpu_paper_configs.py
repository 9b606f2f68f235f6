"""Parity at the full sizes of the secondary workloads and on the trees the paper serves.

The long-sequence workload at 16 x 512 and the BERT-large-width workload at 64 x 128 (so that the
launch shapes of those sizes - CTA-pair GEMMs at hidden 1024 / FFN 4096, many query tiles per
sequence - run inside a forward), the Appendix E shaped 21-task model with token-level heads, the
un-distilled tree of Table 2 (up to ten task layers in place in one buffer), and the paper's
correctness argument (Section 3.3: merging only shares the frozen layers) bit for bit on the
8-task tree at the benchmark's size.  The oracle is evaluated on a few sampled sequences
(sequences are independent, so each sampled row is an exact check)."""
import numpy as np
import pytest
import torch

from oracle import mt_oracle as orc
from paper_2107_05377_b200 import binding as mt
from paper_2107_05377_b200 import synth
from gpu_util import cached_weights, dev_batch, dev_bf16_to_f64, rel_l2, task_triples

pytestmark = pytest.mark.gpu

HIDDEN_REL_L2 = 1e-2
LOGIT_MAX_ABS = 2e-2


def sampled_rows(lengths, extra=()):
    order = np.argsort(lengths, kind="stable")
    return sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), *extra})


def forward(cfg, blob, batch, mask=None, debug=False, expected_tokens=None, options=()):
    B, S = batch.token_ids.shape
    model = mt.MTModel(cfg, B, S, debug_capture=debug)
    if expected_tokens is not None:
        model.set_option("expected_tokens", expected_tokens)
    for key, value in options:
        model.set_option(key, value)
    model.load_weights(blob)
    tok, seg, lens = dev_batch(batch)
    logits = torch.full((B, max(cfg.total_classes, 1)), float("nan"), device="cuda")
    tlog = None
    if cfg.total_token_classes > 0:
        tlog = torch.full((B, S, cfg.total_token_classes), float("nan"), device="cuda")
        model.forward_tokens(tok, seg, lens, logits, tlog, task_mask=mask)
    else:
        model.forward(tok, seg, lens, logits, task_mask=mask)
    torch.cuda.synchronize()
    assert model.poll_status() == 0
    return model, logits, tlog


def check(cfg, wf, batch, model, logits, tlog, rows, hidden=True):
    """Logits (both kinds) and every captured hidden state of the sampled sequences against the oracle.
    The last layer of a sequence-level branch is evaluated for the first token only: compared there."""
    B, S = batch.token_ids.shape
    hid, tl = [], []
    want = orc.forward_batch_mt(batch.token_ids, batch.segment_ids, batch.lengths, wf, task_triples(cfg), cfg.heads,
                                cfg.ln_eps, rows=rows, hidden_out=hid, token_logits_out=tl)
    got = logits.cpu().numpy().astype(np.float64)
    for b in rows:
        assert np.all(np.isfinite(got[b, :cfg.total_classes]))
        assert np.max(np.abs(got[b, :cfg.total_classes] - want[b])) <= LOGIT_MAX_ABS, f"logits of sequence {b}"
    if tlog is not None:
        got_t = tlog.cpu().numpy().astype(np.float64)
        for b in rows:
            n = int(batch.lengths[b])
            assert np.all(np.isnan(got_t[b, n:])), "positions beyond the length must stay untouched"
            assert np.max(np.abs(got_t[b, :n] - tl[0][b, :n])) <= LOGIT_MAX_ABS, f"token logits of sequence {b}"
            assert rel_l2(got_t[b, :n], tl[0][b, :n]) <= HIDDEN_REL_L2
    if not hidden:
        return
    states = {}
    for key in hid[0]:
        t, layer = (-1, key[1]) if key[0] == "trunk" else (key[1], key[2])
        states[key] = dev_bf16_to_f64(model.debug_hidden(t, layer, B, S)).reshape(B, S, cfg.hidden)
    for i, b in enumerate(rows):
        n = int(batch.lengths[b])
        for key, ref in hid[i].items():
            n_cmp = n
            if key[0] == "task":
                spec = cfg.tasks[key[1]]
                if key[2] == spec.branch_layers and not spec.token_level:
                    n_cmp = 1
            err = rel_l2(states[key][b, :n_cmp], ref[:n_cmp])
            assert err <= HIDDEN_REL_L2, f"hidden {key} of sequence {b}: rel-L2 {err}"


def test_long_sequences_at_full_batch_16x512():
    cfg = synth.config_glue8()
    w, blob, wf = cached_weights(cfg, 0)
    batch = synth.make_batch(cfg, 16, 512, 128, 512, seed=1)
    model, logits, _ = forward(cfg, blob, batch, debug=True, expected_tokens=int(batch.lengths.sum()))
    rows = sampled_rows(batch.lengths)
    check(cfg, wf, batch, model, logits, None, [rows[0], rows[-1]])
    assert torch.isfinite(logits).all()


def test_large_width_tree_at_full_batch_64x128():
    cfg = synth.config_large8()
    w, blob, wf = cached_weights(cfg, 0)
    batch = synth.make_batch(cfg, 64, 128, 32, 128, seed=1)
    model, logits, _ = forward(cfg, blob, batch, debug=True, expected_tokens=int(batch.lengths.sum()))
    rows = sampled_rows(batch.lengths)
    check(cfg, wf, batch, model, logits, None, [rows[0], rows[-1]])
    assert torch.isfinite(logits).all()
    # the same bits without the capture and whatever the row estimate (pairs or single CTAs, any tile width)
    for hint in (None, 1024):
        _, plain, _ = forward(cfg, blob, batch, expected_tokens=hint)
        assert torch.equal(plain, logits)


def test_production_shaped_21_task_model_with_token_heads_32x128():
    """Appendix E: 21 tasks, 8 shared + 32 task layers, token-level tasks beside the sequence-level ones."""
    cfg = synth.config_production21()
    w, blob, wf = cached_weights(cfg, 0)
    batch = synth.batch_glue8(cfg)
    model, logits, tlog = forward(cfg, blob, batch, debug=True)
    assert max(model.plan_summary(model.full_mask())["groups_per_wave"]) > 8
    check(cfg, wf, batch, model, logits, tlog, sampled_rows(batch.lengths)[:2])
    offs = cfg.logit_offsets
    valid = torch.from_numpy(np.arange(128)[None, :] < batch.lengths[:, None]).cuda()
    # a sequence-level task with two layers, one with one layer, a token-level task: alone == merged, bit for bit
    for t in (0, 1, 20):
        spec = cfg.tasks[t]
        _, one, one_t = forward(cfg, blob, batch, mask=1 << t)
        cols = slice(offs[t], offs[t] + spec.num_classes)
        if spec.token_level:
            assert torch.equal(one_t[..., cols][valid], tlog[..., cols][valid]), t
            assert torch.isnan(one).all()
        else:
            assert torch.equal(one[:, cols], logits[:, cols]), t
            assert torch.isnan(one_t).all()


def test_undistilled_tree_of_table_2_up_to_ten_task_layers():
    """Table 2, "ours (w/o KD)": (x, y) = (2,10)(7,5)(2,10)(4,8)(6,6)(7,5)(4,8)(4,8), 67 layers."""
    cfg = synth.config_paper_tree("ours (w/o KD)")
    w, blob, wf = cached_weights(cfg, 0)
    batch = synth.make_batch(cfg, 8, 128, 16, 128, seed=3)
    model, logits, _ = forward(cfg, blob, batch, debug=True)
    assert model.plan_summary(model.full_mask())["layers"] == 67
    rows = sampled_rows(batch.lengths)
    check(cfg, wf, batch, model, logits, None, [rows[0], rows[-1]])
    # one deep task alone (its stand-alone student shares the blob here): same bits
    _, alone, _ = forward(cfg, blob, batch, mask=1 << 2)
    off = cfg.logit_offsets[2]
    assert torch.equal(alone[:, off:off + 2], logits[:, off:off + 2])


def test_merged_equals_standalone_students_on_the_8_task_tree_32x128():
    """Section 3.3 at the benchmark's size and launch configuration: every task's columns of the merged
    model equal, bit for bit, the logits of its stand-alone student (x frozen layers + its y own layers),
    built as a model of its own from a blob of its own."""
    cfg = synth.config_glue8()
    w, blob, wf = cached_weights(cfg, 0)
    batch = synth.batch_glue8(cfg)
    tokens = int(batch.lengths.sum())
    _, merged, _ = forward(cfg, blob, batch, expected_tokens=tokens)
    offs = cfg.logit_offsets
    for t in range(cfg.n_tasks):
        st_cfg = synth.config_single_task(cfg, t)
        st_blob = synth.pack_weights(st_cfg, synth.select_task_weights(w, t))
        for hint in (tokens, None):
            _, single, _ = forward(st_cfg, st_blob, batch, expected_tokens=hint)
            cols = slice(offs[t], offs[t] + cfg.tasks[t].num_classes)
            assert torch.equal(merged[:, cols], single), f"task {t}: merged and stand-alone logits differ"
