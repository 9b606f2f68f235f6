"""Serving sweep of the merged multi-task tree (the workloads beside the headline benchmark).

    python -m paper_2107_05377_b200.sweep [--quick]

One JSON line per case:
  * the 8-task BERT-base tree at batch {1, 4, 16, 64, 256} x seq 128 (all lengths 128) with every
    task active, a seeded random half of the tasks, and single tasks (the shallowest and the deepest
    fork), eagerly launched and replayed from a CUDA graph;
  * eight independent full-depth (12-layer) single-task models over the same inputs, through the same
    library, to reproduce the paper's sharing saving (Table 2: 96 layers against the merged tree's 24);
  * the merged models whose layer totals the paper prints (Table 2, Table 4), at 32 x 128 with lengths in
    [16, 128]: measured time against the paper's cost measure, the number of layers evaluated;
  * the long-sequence variant (16 x 512, lengths in [128, 512]), the BERT-large-width tree
    (64 x 128, lengths in [32, 128]) and a 21-task tree shaped like the production model of Appendix E
    (8 shared + 32 task layers, a third of the tasks token-level; 32 x 128, lengths in [16, 128]).
Weights are seeded random (timing does not depend on their values; the eight single-task models are
loaded from one blob into eight separate arenas).  Inputs are resident on the device.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding, synth


def _dev(batch):
    return (torch.from_numpy(batch.token_ids).cuda(), torch.from_numpy(batch.segment_ids).cuda(),
            torch.from_numpy(batch.lengths).cuda())


def _time_ms(fn, iters, graph):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        g.replay()
        torch.cuda.synchronize()
        start.record()
        for _ in range(iters):
            g.replay()
        end.record()
    else:
        start.record()
        for _ in range(iters):
            fn()
        end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / iters


def flops_padded(cfg, layers, batch, seq):
    m = batch * seq
    return layers * (2.0 * m * (4 * cfg.hidden * cfg.hidden + 2 * cfg.hidden * cfg.ffn) + batch * 4.0 * cfg.hidden * seq * seq)


def run_tree(name, cfg, blob, batch, masks, iters, out, fp8=False):
    B, S = batch.token_ids.shape
    model = binding.MTModel(cfg, B, S, fp8_gemm=fp8)
    model.load_weights(blob)
    tok, seg, lens = _dev(batch)
    logits = torch.zeros(B, max(cfg.total_classes, 1), dtype=torch.float32, device="cuda")
    token_logits = torch.zeros(B, S, cfg.total_token_classes, dtype=torch.float32, device="cuda") \
        if cfg.total_token_classes > 0 else None
    for label, mask in masks:
        plan = model.plan_summary(mask)
        fn = lambda: model.forward_tokens(tok, seg, lens, logits, token_logits, task_mask=mask)  # noqa: E731
        eager = _time_ms(fn, iters, False)
        graph = _time_ms(fn, iters, True)
        assert model.poll_status() == 0
        fl = flops_padded(cfg, plan["layers"], B, S)
        out({"case": name, "batch": B, "seq": S, "tasks": label, "mask": mask, "layers": plan["layers"],
             "waves": plan["waves"], "launches": model.plan_launches(mask), "ms_eager": eager, "ms_graph": graph,
             "seq_per_s_graph": 1e3 * B / graph, "tflops_padded_graph": fl / graph / 1e9,
             "valid_fraction": float(batch.lengths.sum()) / (B * S)})
    model.close()
    del model


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="batches {1, 32} only and no wide tree")
    a = ap.parse_args()

    def out(d):
        print(json.dumps(d), flush=True)

    cfg = synth.config_glue8()
    weights = synth.make_weights(cfg, seed=0)
    blob = synth.pack_weights(cfg, weights)
    half = int(sum(1 << int(t) for t in np.random.default_rng(2).permutation(8)[:4]))
    masks = [("all 8", 0xFF), (f"random 4 (mask {half:#04x})", half), ("task 6 (fork 4, 3 layers)", 1 << 6),
             ("task 7 (fork 8, 2 layers)", 1 << 7)]
    batches = (1, 32) if a.quick else (1, 4, 16, 64, 256)

    # eight independent full-depth single-task models: one blob, eight arenas
    st_cfg = synth.config_full_depth_single(cfg, 2)
    st_w = {"emb": weights["emb"], "trunk": [], "tasks": [synth.make_task_weights(st_cfg, 0, seed=0)]}
    st_blob = synth.pack_weights(st_cfg, st_w)

    for B in batches:
        batch = synth.make_batch(cfg, B, 128, 128, 128, seed=1)
        iters = 50 if B <= 64 else 20
        run_tree("glue8 tree", cfg, blob, batch, masks, iters, out)
        models = [binding.MTModel(st_cfg, B, 128) for _ in range(8)]
        for m in models:
            m.load_weights(st_blob)
        tok, seg, lens = _dev(batch)
        lg = torch.zeros(B, 2, dtype=torch.float32, device="cuda")

        def eight():
            for m in models:
                m.forward(tok, seg, lens, lg)

        eager, graph = _time_ms(eight, iters, False), _time_ms(eight, iters, True)
        out({"case": "8 independent 12-layer single-task models (0,12)", "batch": B, "seq": 128, "layers": 96,
             "launches": 8 * models[0].plan_launches(1), "ms_eager": eager, "ms_graph": graph,
             "seq_per_s_graph": 1e3 * B / graph, "tflops_padded_graph": flops_padded(cfg, 96, B, 128) / graph / 1e9})
        for m in models:
            m.close()
        del models

    run_tree("glue8 tree, long sequences", cfg, blob, synth.make_batch(cfg, 16, 512, 128, 512, seed=1),
             [("all 8", 0xFF)], 20, out)
    run_tree("glue8 tree, headline shape", cfg, blob, synth.batch_glue8(cfg), [("all 8", 0xFF)], 50, out)
    # the 8-bit projections (option "fp8_gemm") beside bf16: where a forward is made of tensor work, not launches
    for B in (32, 256):
        hb8 = synth.batch_glue8(cfg, B, 128)
        run_tree("glue8 tree, lengths U[16,128], bf16", cfg, blob, hb8, [("all 8", 0xFF)], 20, out)
        run_tree("glue8 tree, lengths U[16,128], E4M3 projections", cfg, blob, hb8, [("all 8", 0xFF)], 20, out, fp8=True)
    # time to each task's logits with heads scheduled as early as possible (the latency limitation of Section 5.2)
    hb = synth.batch_glue8(cfg)
    for early in (0, 1):
        model = binding.MTModel(cfg, 32, 128)
        model.set_option("early_heads", early)
        model.load_weights(blob)
        tok, seg, lens = _dev(hb)
        logits = torch.zeros(32, cfg.total_classes, dtype=torch.float32, device="cuda")
        for _ in range(3):
            model.forward(tok, seg, lens, logits)
        torch.cuda.synchronize()
        acc, total, reps = [0.0] * 8, 0.0, 20
        for _ in range(reps):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(8)]
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record()
            model.forward_events(tok, seg, lens, logits, ev)
            s1.record()
            torch.cuda.synchronize()
            acc = [x + s0.elapsed_time(e) for x, e in zip(acc, ev)]
            total += s0.elapsed_time(s1)
        out({"case": "glue8 tree, headline shape, per-task completion", "batch": 32, "seq": 128, "early_heads": early,
             "launches": model.plan_launches(0xFF), "ms_total": total / reps,
             "ms_to_task_logits": [x / reps for x in acc],
             "task_finish_wave": [t.fork_depth + t.branch_layers for t in cfg.tasks]})
        model.close()
    if not a.quick:
        del weights, blob
        big = synth.config_large8()
        big_blob = synth.pack_weights(big, synth.make_weights(big, seed=0))
        run_tree("large-width tree", big, big_blob, synth.make_batch(big, 64, 128, 32, 128, seed=1),
                 [("all 8", 0xFF)], 20, out)
        del big_blob
        # the paper's own merged models (Table 2, Table 4): measured cost against its measure, the layer count
        for name in synth.PAPER_TREES:
            tree = synth.config_paper_tree(name)
            tree_blob = synth.pack_weights(tree, synth.make_weights(tree, seed=0))
            run_tree(f"paper tree: {name}", tree, tree_blob, synth.make_batch(tree, 32, 128, 16, 128, seed=1),
                     [("all 8", 0xFF)], 20, out)
            del tree_blob
        prod = synth.config_production21()
        prod_blob = synth.pack_weights(prod, synth.make_weights(prod, seed=0))
        seq_only = sum(1 << t for t, spec in enumerate(prod.tasks) if not spec.token_level)
        run_tree("production-shaped tree (21 tasks, 7 token-level)", prod, prod_blob,
                 synth.make_batch(prod, 32, 128, 16, 128, seed=1),
                 [("all 21", (1 << 21) - 1), ("the 14 sequence-level tasks", seq_only)], 20, out)


if __name__ == "__main__":
    main()
