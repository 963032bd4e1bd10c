"""Verification-tree design and choice of the verification width for one B200.

Host-side part of the method (paper Sec. III-C): from calibrated per-head, per-rank accuracies
the tree of a given width is the set of candidate sequences with the highest estimated
accuracy (product of the accuracies along the sequence, added one by one), and the width to run
with is the one that maximises expected tokens per second = expected acceptance length /
measured latency of the verify step at that width.

    python -m paper_2505_23219_b200.arca [--layers 32] [--kv-len 2048] [--widths 1,4,8,...]

measures the verify step through the C-ABI at each width (synthetic LLaMA-7B-shaped weights,
synthetic accuracies 0.6 * 0.8**level * 0.5**rank capped at (10, 4, 2, 1, 1) candidates per head)
and prints latency, expected acceptance length and tokens per second per width and the choice.
"""
from __future__ import annotations

import heapq

__all__ = ["build_tree", "expected_tokens", "choose_width", "synthetic_accuracies"]


def synthetic_accuracies(caps=(10, 4, 2, 1, 1)):
    """Stand-in for a calibration run: head l's rank-r candidate is right with 0.6 * 0.8**l * 0.5**r."""
    return [[0.6 * 0.8 ** l * 0.5 ** r for r in range(c)] for l, c in enumerate(caps)]


def build_tree(acc, width: int):
    """Greedy tree of `width` nodes (root included).  acc[l][r] = accuracy of head l's rank-r candidate.

    A max-heap holds, for every node already in the tree, its best child not yet taken and, for
    every taken child, its next sibling: with accuracies that do not grow with the rank these are
    the only candidates that can be the global best.  Falls back to a full frontier when a head's
    accuracies are not sorted.  Ties: shallower node first, then the smaller rank path.
    -> (parent[] in breadth-first order, rank path of every node, acceptance probability of every node)
    """
    sorted_ranks = all(all(a[i] >= a[i + 1] for i in range(len(a) - 1)) for a in acc)
    prob = {(): 1.0}
    heap = []

    def push(path, p):
        heapq.heappush(heap, (-p, len(path), path))

    def offer_children(path, p):
        l = len(path)
        if l >= len(acc):
            return
        ranks = range(1) if sorted_ranks else range(len(acc[l]))
        for r in ranks:
            if r < len(acc[l]):
                push(path + (r,), p * acc[l][r])

    offer_children((), 1.0)
    while len(prob) < width and heap:
        negp, _, path = heapq.heappop(heap)
        if path in prob:
            continue
        prob[path] = -negp
        offer_children(path, -negp)
        if sorted_ranks:                                        # the next sibling becomes a candidate
            l, r = len(path) - 1, path[-1] + 1
            if r < len(acc[l]):
                push(path[:-1] + (r,), prob[path[:-1]] * acc[l][r])
    order = sorted(prob, key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(order)}
    return [-1 if not p else index[p[:-1]] for p in order], order, [prob[p] for p in order]


def expected_tokens(node_prob) -> float:
    """Expected tokens per verify step (the root's token is always produced)."""
    return float(sum(node_prob))


def choose_width(latency_us: dict, acc):
    """latency_us: {width: measured step latency}.  -> (chosen width, [(width, latency, tokens/step, tokens/s)])."""
    rows = []
    for w in sorted(latency_us):
        _, _, prob = build_tree(acc, w)
        tau = expected_tokens(prob)
        rows.append((w, latency_us[w], tau, tau / (latency_us[w] * 1e-6)))
    best = max(rows, key=lambda r: (r[3], -r[0]))
    return best[0], rows


def _measure(widths, layers, kv_len, draft=False):
    import sys
    from pathlib import Path

    import numpy as np
    import torch

    sys.path.insert(0, str(Path(__file__).resolve().parent.parent))
    import paper_2505_23219_b200 as ghd
    import workloads as wl

    shape = wl.scaled(wl.LLAMA7B, n_layers=layers)
    nmax = max(widths)
    max_kv = kv_len + nmax
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    head = wl.head_weights(shape, 3)
    gl, gkv = [], []
    for l in range(shape.n_layers):
        w = wl.layer_weights(shape, 3, l)
        gl.append(ghd.LayerWeights(**{k: dev(w[k]) for k in ghd.LayerWeights.FIELDS}))
        kc, vc = wl.kv_cache(shape, 3, l, kv_len, max_kv)
        gkv.append(ghd.KvLayer(dev(kc), dev(vc), kv_len))
    gw = ghd.ModelWeights(dev(head["embed"]), gl, dev(head["rms_final"]), dev(head["lm_head"]))
    cfg = ghd.ModelCfg(shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab, shape.n_layers, max_kv, nmax,
                       shape.dtype, shape.rms_eps, shape.rope_theta)
    ctx = ghd.ghd_create(cfg)
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, 2)
    acc = synthetic_accuracies()
    lat = {}
    draft_us = 0.0
    if draft:
        # the drafter of the paper's default set-up: five heads (d x d block + vocabulary projection each, random here)
        k = len(acc)
        mw = ghd.MedusaWeights(torch.randn(k, shape.d_model, shape.d_model, device="cuda", dtype=torch.float16) * 0.02,
                               torch.randn(k, shape.vocab, shape.d_model, device="cuda", dtype=torch.float16) * 0.02)
        topk = [len(a) for a in acc]
        parent, paths, _ = build_tree(acc, 64)
        level = dev(np.array([len(p) for p in paths], np.int32))
        rank = dev(np.array([p[-1] if p else 0 for p in paths], np.int32))
        tokens = dev(wl.draft_tokens(parent, shape.vocab, 5))
        tree = ghd.ghd_tree_build(ctx, parent, kv_len)
        amax = torch.empty(64, dtype=torch.int32, device="cuda")
        res = torch.zeros(2 + 2 * ghd.GHD_MAX_NODES, dtype=torch.int32, device="cuda")
        ghd.ghd_verify_step(ctx, gw, gkv, tree, tokens, logits=False, argmax=amax)
        ghd.ghd_accept(ctx, tree, tokens, amax, res)
        nxt = torch.empty(64, dtype=torch.int32, device="cuda")

        def draft_once():
            ghd.ghd_tree_fill_tokens(ctx, ghd.ghd_medusa_draft(ctx, mw, res, topk), res, level, rank, nxt)

        for _ in range(3):
            draft_once()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            draft_once()
        e1.record()
        torch.cuda.synchronize()
        ghd.ghd_sync_status(ctx)
        draft_us = e0.elapsed_time(e1) / 20 * 1e3
    for w in widths:
        parent, _, _ = build_tree(acc, w)
        tokens = dev(wl.draft_tokens(parent, shape.vocab, 11 + w))
        tree = ghd.ghd_tree_build(ctx, parent, kv_len)
        amax = torch.empty(w, dtype=torch.int32, device="cuda")
        res = torch.zeros(2 + 2 * ghd.GHD_MAX_NODES, dtype=torch.int32, device="cuda")

        def step():
            ghd.ghd_verify_step(ctx, gw, gkv, tree, tokens, logits=False, argmax=amax)
            ghd.ghd_accept(ctx, tree, tokens, amax, res)

        for _ in range(3):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            step()
        e1.record()
        torch.cuda.synchronize()
        ghd.ghd_sync_status(ctx)
        lat[w] = e0.elapsed_time(e1) / 20 * 1e3
    return lat, acc, draft_us


def main():
    import argparse
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--kv-len", type=int, default=2048)
    ap.add_argument("--widths", default="1,2,4,8,16,24,32,48,64,96,128")
    ap.add_argument("--draft", action="store_true", help="also time the five drafting heads and charge them to every width above 1")
    a = ap.parse_args()
    widths = [int(x) for x in a.widths.split(",")]
    lat, acc, draft_us = _measure(widths, a.layers, a.kv_len, a.draft)
    if a.draft:
        print(f"drafting heads + token fill: {draft_us:.1f} us per step (added to the latency of every width above 1)")
        lat = {w: l + (draft_us if w > 1 else 0.0) for w, l in lat.items()}
    best, rows = choose_width(lat, acc)
    print("| width | step latency us | expected tokens / step | tokens / s | speed-up over width 1 |")
    print("|---|---|---|---|---|")
    base = rows[0][3]
    for w, l, tau, tps in rows:
        print(f"| {w} | {l:.1f} | {tau:.3f} | {tps:.1f} | {tps / base:.2f} |")
    print(f"chosen width: {best}")


if __name__ == "__main__":
    main()
