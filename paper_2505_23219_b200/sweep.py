"""Latency of ONE decoder layer (or of its tree attention alone) against the tree size and the KV length.

    python -m paper_2505_23219_b200.sweep [--shape 7b|13b] [--what layer|attention|decode]
                                          [--nodes 1,4,...] [--kv-len 512,2048,4096] [--opt ID=VALUE ...]

--what decode times whole self-drafting decode steps instead (tree build, verify, accept, KV commit, drafting heads,
token fill; 32 layers, 64-node tree, five heads, random weights): driven by the host with one read of the accepted
length per step, against the same steps with the cache length kept on the device, recorded once into a CUDA graph.

Every (nodes, kv_len) point runs the call on COPIES distinct layers in turn (their weights and caches do not
fit the L2 together, so every call streams its bytes from HBM), recorded once into a CUDA graph and replayed:
the host's launch cost is not in the number.  Inputs are seeded random tensors of the model's shapes (values
do not matter for the time).  Prints a markdown table: microseconds per call, the HBM rate on the algorithmic
bytes (all weights once + K and V caches once + the new rows + activations in and out) as a fraction of
8 TB/s and of the measured copy peak, and the fraction of the sustained fp16 tensor rate that the
projections and the attention products reach (the roofline that binds for wide trees).
"""
from __future__ import annotations

import argparse
import json
from pathlib import Path

import numpy as np
import torch

import workloads as wl

from . import binding as ghd


def _peaks():
    p = Path(__file__).resolve().parent.parent / "MEASURED_PEAKS.json"
    try:
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 6650.0, 1400.0, "fallback"


def layer_bytes_flops(shape, n, kv_len, depths):
    s, d = shape.itemsize, shape.d_model
    nbytes = shape.params_per_layer * s + 2 * kv_len * d * s + 2 * n * d * s + 2 * n * d * s
    flops = 2.0 * n * shape.params_per_layer + 4.0 * shape.d_head * shape.n_heads * sum(kv_len + dep + 1 for dep in depths)
    return nbytes, flops


def _timed_graph(stream, body, reps):
    """Records body() into a CUDA graph on `stream` and replays it; -> microseconds per replay."""
    with torch.cuda.stream(stream):
        for _ in range(2):
            body()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            body()
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) * 1e3 / reps


def measure(shape, what, nodes, kv_lens, opts, copies, reps, tree_kind="auto"):
    d, H, dh, f = shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn
    nmax, lmax = max(nodes), max(kv_lens)
    max_kv = lmax + nmax
    stream = torch.cuda.Stream()
    rows = []
    with torch.cuda.stream(stream):
        gen = torch.Generator(device="cuda").manual_seed(wl.BASE_SEED)
        rnd = lambda *sh, std=1.0: (torch.randn(*sh, device="cuda", dtype=torch.float16, generator=gen) * std)
        cfg = ghd.ModelCfg(d, H, dh, f, shape.vocab, 1, max_kv, nmax, "f16", shape.rms_eps, shape.rope_theta)
        ctx = ghd.ghd_create(cfg)
        for spec in opts:
            o, v = spec.split("=")
            ghd.ghd_set_option(ctx, int(o), int(v))
        layers, kvs = [], []
        for _ in range(copies):
            if what == "layer":
                layers.append(ghd.LayerWeights(wqkv=rnd(3 * d, d, std=0.02), wo=rnd(d, d, std=0.02), w_gate_up=rnd(2 * f, d, std=0.02),
                                               w_down=rnd(d, f, std=0.02), rms1=torch.ones(d, device="cuda", dtype=torch.float16),
                                               rms2=torch.ones(d, device="cuda", dtype=torch.float16)))
            kvs.append((rnd(H, max_kv, dh), rnd(H, max_kv, dh)))
        for kv_len in kv_lens:
            for n in nodes:
                if tree_kind == "star":
                    parent = wl.star_tree(n)
                elif tree_kind == "chain":
                    parent = wl.chain_tree(n)
                elif n == 64 and tree_kind == "auto":
                    parent = wl.medusa_tree(n)
                else:
                    parent = wl.random_tree(n, 8, wl.BASE_SEED + 4000 + n + kv_len, max_children=6)
                depths = wl.depths_of(parent)
                tree = ghd.ghd_tree_build(ctx, parent, kv_len)
                x = rnd(n, d)
                y = torch.empty_like(x)
                kl = [ghd.KvLayer(k, v, kv_len) for k, v in kvs]

                def body():
                    for c in range(copies):
                        if what == "layer":
                            ghd.ghd_verify_layer(ctx, layers[c], kl[c], tree, x, y)
                        else:
                            ghd.ghd_tree_attention(ctx, x, kl[c], tree, y)

                us = _timed_graph(stream, body, reps) / copies
                ghd.ghd_sync_status(ctx)
                rows.append((n, kv_len, us, depths))
        ghd.ghd_destroy(ctx)
    return rows


def measure_decode(shape, kv_len, steps, opts, layers=0):
    """-> (us per step, host-driven loop), (us per step, device-driven loop in one CUDA graph), tokens per step."""
    from . import arca
    if layers:
        shape = wl.scaled(shape, n_layers=layers)
    width = 64
    acc = arca.synthetic_accuracies()
    topk = [len(a) for a in acc]
    parent, paths, _ = arca.build_tree(acc, width)
    max_kv = kv_len + (steps + 2) * (len(acc) + 1) + width + 1
    stream = torch.cuda.Stream()
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    with torch.cuda.stream(stream):
        head = wl.head_weights(shape, 3)
        gl, caches = [], []
        for l in range(shape.n_layers):
            w = wl.layer_weights(shape, 3, l)
            gl.append(ghd.LayerWeights(**{k: dev(w[k]) for k in ghd.LayerWeights.FIELDS}))
            kc, vc = wl.kv_cache(shape, 3, l, kv_len, max_kv)           # every row of the buffers holds finite data
            caches.append((dev(kc), dev(vc)))
        gw = ghd.ModelWeights(dev(head["embed"]), gl, dev(head["rms_final"]), dev(head["lm_head"]))
        k = len(acc)
        mw = ghd.MedusaWeights(torch.randn(k, shape.d_model, shape.d_model, device="cuda", dtype=torch.float16) * 0.02,
                               torch.randn(k, shape.vocab, shape.d_model, device="cuda", dtype=torch.float16) * 0.02)
        level = dev(np.array([len(p) for p in paths], np.int32))
        rank = dev(np.array([p[-1] if p else 0 for p in paths], np.int32))
        cfg = ghd.ModelCfg(shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab, shape.n_layers, max_kv, width,
                           shape.dtype, shape.rms_eps, shape.rope_theta)
        ctx = ghd.ghd_create(cfg)
        for spec in opts:
            o, v = spec.split("=")
            ghd.ghd_set_option(ctx, int(o), int(v))
        first_tokens = dev(wl.draft_tokens(parent, shape.vocab, 5))
        tok = first_tokens.clone()
        amax = torch.empty(width, dtype=torch.int32, device="cuda")
        results = torch.zeros((steps, 2 + 2 * ghd.GHD_MAX_NODES), dtype=torch.int32, device="cuda")
        tree = ghd.Tree(ctx)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def one_step(s, kv, kvs):
            ghd.ghd_tree_build(ctx, parent, kv, tree=tree)
            ghd.ghd_verify_step(ctx, gw, kvs, tree, tok, logits=False, argmax=amax)
            ghd.ghd_accept(ctx, tree, tok, amax, out=results[s])
            ghd.ghd_kv_commit(ctx, kvs, kv, results[s])
            cand = ghd.ghd_medusa_draft(ctx, mw, results[s], topk)
            ghd.ghd_tree_fill_tokens(ctx, cand, results[s], level, rank, tokens=tok)

        # (a) the host drives: it reads the number of accepted tokens after every step to know the next cache length
        def host_loop():
            L = kv_len
            for s in range(steps):
                kvs = [ghd.KvLayer(kc, vc, L) for kc, vc in caches]
                one_step(s, L, kvs)
                L += int(results[s, 0].item()) + 1
            return L
        tok.copy_(first_tokens)
        host_loop()
        tok.copy_(first_tokens)
        stream.synchronize()
        e0.record(stream)
        L_host = host_loop()
        e1.record(stream)
        stream.synchronize()
        us_host = e0.elapsed_time(e1) * 1e3 / steps
        # (b) nothing between the steps needs the host: all steps recorded once, replayed as one graph
        kvs_dev = [ghd.KvLayer(kc, vc, ghd.KV_LEN_DEVICE) for kc, vc in caches]
        ghd.ghd_kv_len_set(ctx, kv_len)
        tok.copy_(first_tokens)
        one_step(0, ghd.KV_LEN_DEVICE, kvs_dev)
        ghd.ghd_sync_status(ctx)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for s in range(steps):
                one_step(s, ghd.KV_LEN_DEVICE, kvs_dev)
        us_dev = 0.0
        for rep in range(2):
            ghd.ghd_kv_len_set(ctx, kv_len)
            tok.copy_(first_tokens)
            stream.synchronize()
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            us_dev = e0.elapsed_time(e1) * 1e3 / steps
        L_dev = ghd.ghd_kv_len_get(ctx)
        ghd.ghd_sync_status(ctx)
        assert L_dev == L_host, (L_dev, L_host)                        # both loops accepted the same tokens
        ghd.ghd_destroy(ctx)
    return us_host, us_dev, (L_dev - kv_len) / steps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shape", default="7b", choices=["7b", "13b"])
    ap.add_argument("--what", default="layer", choices=["layer", "attention", "decode"])
    ap.add_argument("--steps", type=int, default=16, help="--what decode: steps per loop")
    ap.add_argument("--layers", type=int, default=0, help="--what decode: override the layer count")
    ap.add_argument("--nodes", default="1,4,8,16,32,64,128,256")
    ap.add_argument("--kv-len", default="512,2048,4096")
    ap.add_argument("--copies", type=int, default=6, help="distinct layers (weights + caches) visited per replay")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--tree", default="auto", choices=["auto", "random", "star", "chain"],
                    help="auto: Medusa-style tree at 64 nodes, random trees of depth <= 8 otherwise")
    ap.add_argument("--opt", action="append", default=[], metavar="ID=VALUE", help="ghd_set_option knob (repeatable)")
    a = ap.parse_args()
    shape = wl.LLAMA7B if a.shape == "7b" else wl.LLAMA13B
    nodes = [int(v) for v in a.nodes.split(",")]
    kv_lens = [int(v) for v in a.kv_len.split(",")]
    hbm, tflops, kind = _peaks()
    if a.what == "decode":
        us_host, us_dev, tps = measure_decode(shape, kv_lens[0], a.steps, a.opt, a.layers)
        print(f"shape {shape.name}, self-drafting decode loop, 64-node tree, five heads, kv_len {kv_lens[0]}, {a.steps} steps, options {a.opt or 'default'}")
        print("| loop | us per step | steps / s |")
        print("|---|---|---|")
        print(f"| host reads the accepted length every step (direct launches) | {us_host:.1f} | {1e6 / us_host:.1f} |")
        print(f"| cache length on the device, all steps in one CUDA graph | {us_dev:.1f} | {1e6 / us_dev:.1f} |")
        print(f"tokens per step with these random heads: {tps:.2f}")
        return
    rows = measure(shape, a.what, nodes, kv_lens, a.opt, a.copies, a.reps, a.tree)
    print(f"shape {shape.name}, {a.what}, tree {a.tree}, options {a.opt or 'default'}; peaks ({kind}): copy {hbm:.0f} GB/s, sustained tensor {tflops:.0f} TFLOP/s")
    if a.what == "layer":
        print("| nodes | kv_len | us per layer | algorithmic MB | GB/s | of 8 TB/s | of the copy peak | GFLOP | of the sustained tensor rate |")
        print("|---|---|---|---|---|---|---|---|---|")
        for n, L, us, depths in rows:
            nb, fl = layer_bytes_flops(shape, n, L, depths)
            gbs = nb / us / 1e3
            print(f"| {n} | {L} | {us:.1f} | {nb / 1e6:.1f} | {gbs:.0f} | {100 * gbs / 8000:.1f} % | {gbs / hbm:.2f} | {fl / 1e9:.1f} | {fl / us / 1e6 / tflops:.2f} |")
    else:
        print("| nodes | kv_len | us per call | K+V MB | GB/s | of the copy peak |")
        print("|---|---|---|---|---|---|")
        for n, L, us, _ in rows:
            nb = 2 * (L + n) * shape.d_model * shape.itemsize
            print(f"| {n} | {L} | {us:.1f} | {nb / 1e6:.1f} | {nb / us / 1e3:.0f} | {nb / us / 1e3 / hbm:.2f} |")


if __name__ == "__main__":
    main()
