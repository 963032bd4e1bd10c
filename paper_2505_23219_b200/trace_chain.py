"""Phase timeline of the persistent projection-chain kernel on a LLaMA-7B-shaped step.

    python -m paper_2505_23219_b200.trace_chain [--layers 4] [--nodes 64] [--kv-len 2048]

Times the step with one kernel per projection and with the chained kernel (graph replay), then
runs the chained step once with ghd_set_trace and prints, for the last chain launch of the step
(merge, O, fold, gate/up, down, fold, lm_head), when each phase was reached, when its dependency
wait ended and when it was done, as the earliest and the latest CTA, in microseconds from the start
of the first CTA.  Synthetic seeded inputs; needs a B200.
"""
from __future__ import annotations

import argparse
import sys
from pathlib import Path

import numpy as np
import torch

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))

import paper_2505_23219_b200 as ghd  # noqa: E402
import workloads as wl  # noqa: E402

PHASES = ["merge", "O", "fold", "gate/up", "down", "fold", "lm_head"]
SLOTS = ["reached", "wait end / last acc", "done", "x gate open", "first w tile", "last w tile", "last x tile", "first acc"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--nodes", type=int, default=64)
    ap.add_argument("--kv-len", type=int, default=2048)
    a = ap.parse_args()
    shape = wl.scaled(wl.LLAMA7B, n_layers=a.layers)
    n, L = a.nodes, a.kv_len
    max_kv = L + n
    parent = wl.medusa_tree(n) if n == 64 else wl.random_tree(n, 8, wl.BASE_SEED + n)
    tokens = wl.draft_tokens(parent, shape.vocab, 7)
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    head = wl.head_weights(shape, 3)
    gl = []
    gkv = []
    for l in range(shape.n_layers):
        w = wl.layer_weights(shape, 3, l)
        gl.append(ghd.LayerWeights(**{k: dev(w[k]) for k in ghd.LayerWeights.FIELDS}))
        kc, vc = wl.kv_cache(shape, 3, l, L, max_kv)
        gkv.append(ghd.KvLayer(dev(kc), dev(vc), L))
    gw = ghd.ModelWeights(dev(head["embed"]), gl, dev(head["rms_final"]), dev(head["lm_head"]))
    tok = dev(tokens)
    amax = torch.empty(n, dtype=torch.int32, device="cuda")

    def make(chain, graph):
        cfg = ghd.ModelCfg(shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab, shape.n_layers, max_kv, n,
                           shape.dtype, shape.rms_eps, shape.rope_theta)
        ctx = ghd.ghd_create(cfg)
        ghd.ghd_set_option(ctx, ghd.OPT_CHAIN, chain)
        ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, graph)
        return ctx, ghd.ghd_tree_build(ctx, parent, L)

    for chain, label in ((0, "one kernel per projection"), (1, "chained projections")):
        ctx, tree = make(chain, 2)
        for _ in range(3):
            ghd.ghd_verify_step(ctx, gw, gkv, tree, tok, logits=False, argmax=amax)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            ghd.ghd_verify_step(ctx, gw, gkv, tree, tok, logits=False, argmax=amax)
        e1.record()
        torch.cuda.synchronize()
        ghd.ghd_sync_status(ctx)
        print(f"{label}: {e0.elapsed_time(e1) / 20 * 1e3:.1f} us per {a.layers}-layer step")

    ctx, tree = make(1, 0)
    trace = ghd.ghd_set_trace(ctx, True)
    for _ in range(3):
        ghd.ghd_verify_step(ctx, gw, gkv, tree, tok, logits=False, argmax=amax)
    ghd.ghd_sync_status(ctx)
    t = trace.cpu().numpy().astype(np.int64)
    t0 = t[8, :, 0].min()
    print(f"CTAs start within {(t[8, :, 0].max() - t0) / 1e3:.1f} us")
    for ph, name in enumerate(PHASES):
        parts = [f"{name:8s}"]
        for k, slot in enumerate(SLOTS):
            seen = t[ph, :, k] > 0
            if seen.any():
                v = (t[ph, seen, k] - t0) / 1e3
                parts.append(f"{slot} {v.min():6.1f}..{v.max():6.1f}")
        print(" | ".join(parts))


if __name__ == "__main__":
    main()
