#!/usr/bin/env python
"""Benchmark of the tree-verification step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Workload (default): the full 32-layer LLaMA-7B-shaped verify step - half weights,
KV length 2048 per layer, 64-node Medusa-style tree, vocab-32000 lm_head, row
argmax and greedy acceptance - on synthetic seeded inputs.  One "step" is one
pass of the whole path: tree build, embedding gather, all layers, lm_head,
argmax, acceptance.  The step streams ~14.4 GB of weights and KV cache, far more
than the L2, so nothing is cache-resident between timed iterations.

With N > 1 (torchrun) every rank runs an independent replica of the same step
(the path has no cross-GPU exchange); the line reports the slowest rank.

Prints ONE JSON line.  ``--impl reference`` times the CPU oracle instead (a
deliberately plain program: context, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import workloads as wl  # noqa: E402

CONFIG_ID = 3
METRIC = "7B verify-step latency (32 layers + lm_head, 64-node tree, KV 2048)"


# ---------------------------------------------------------------- workload description
def workload(args):
    shape = wl.LLAMA7B
    if args.layers:
        shape = wl.scaled(shape, n_layers=args.layers)
    n, kv_len = args.nodes, args.kv_len
    parent = wl.medusa_tree(n) if n == 64 else wl.random_tree(n, 8, wl.BASE_SEED + n)
    fixture = ROOT / "tests" / "golden" / "c3_step_llama7b.json"
    if n == 64 and kv_len == 2048 and fixture.exists():
        tokens = np.asarray(json.loads(fixture.read_text())["tokens"], dtype=np.int32)
    else:
        tokens = wl.draft_tokens(parent, shape.vocab, wl.BASE_SEED + 1000 * CONFIG_ID + 700)
    return shape, n, kv_len, parent, tokens


def algorithmic_bytes(shape, n, kv_len):
    """Bytes one verify step must move: every weight once, K and V caches once, new K/V rows,
    embedding rows, logits; intermediates are not counted."""
    s, d = shape.itemsize, shape.d_model
    per_layer = shape.params_per_layer * s + 2 * kv_len * d * s + 2 * n * d * s
    return shape.n_layers * per_layer + shape.vocab * d * s + n * d * s + n * shape.vocab * 4


# DRAM bytes (read + written) per launch of the roofline kernel, from an ncu capture of exactly that launch;
# valid only for the kernel sources it was taken on (hash below), else the line reports null.
NCU_TRAFFIC = {"sources": ("gemm_tc.cu", "gemm_tc_dev.cuh", "tc_common.cuh"), "sha256_16": "527b8c3b9d936247",
               "bytes_per_launch": 183.18e6}


def ncu_traffic():
    import hashlib
    h = hashlib.sha256()
    try:
        for f in NCU_TRAFFIC["sources"]:
            h.update((ROOT / "paper_2505_23219_b200" / "csrc" / f).read_bytes())
    except OSError:
        return None
    return NCU_TRAFFIC["bytes_per_launch"] if h.hexdigest()[:16] == NCU_TRAFFIC["sha256_16"] else None


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ---------------------------------------------------------------- clocks sampling
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self._stop, self._t = index, [], threading.Event(), None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                self.rows.append([c.strip() for c in out.strip().split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=6)

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 6 for i in range(4) if r[2 + i].lower() == "active"})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ---------------------------------------------------------------- CPU oracle timing
def time_oracle_sample(shape, n, kv_len, parent, tokens, sample_layers: int):
    """Times the oracle on `sample_layers` layers plus the lm_head of the workload and scales the
    layer part to the full depth.  -> (estimated microseconds per full step, cores, description)."""
    import oracle
    max_kv = kv_len + n
    vis, _, pos = oracle.tree_build(parent, kv_len)
    head = wl.head_weights(shape, CONFIG_ID)
    x = head["embed"][tokens].astype(np.float64)
    t_layers = 0.0
    for l in range(sample_layers):
        w = wl.layer_weights(shape, CONFIG_ID, l)
        kc, vc = wl.kv_cache(shape, CONFIG_ID, l, kv_len, max_kv)
        t0 = time.perf_counter()
        x = oracle.layer(shape, w, kc, vc, kv_len, vis, pos, x)
        t_layers += time.perf_counter() - t0
    t0 = time.perf_counter()
    logits = oracle.linear(oracle.rmsnorm(x, head["rms_final"], shape.rms_eps), head["lm_head"])
    amax = oracle.argmax(logits)
    oracle.accept(parent, tokens, amax)
    t_head = time.perf_counter() - t0
    est = t_layers * shape.n_layers / max(sample_layers, 1) + t_head
    if sample_layers >= shape.n_layers:
        desc = (f"one whole step: all {shape.n_layers} layers ({t_layers:.2f} s) + final norm + lm_head + argmax + accept "
                f"({t_head:.2f} s), single run")
    else:
        desc = (f"layers 0..{sample_layers - 1} of {shape.n_layers} timed ({t_layers:.2f} s) and scaled by "
                f"{shape.n_layers}/{sample_layers}, plus final norm + lm_head + argmax + accept ({t_head:.2f} s)")
    return est * 1e6, oracle.n_threads(), desc


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape, n, kv_len, parent, tokens = workload(args)
    sample_layers = min(shape.n_layers, 2)
    vals = []
    for it in range(args.warmup + args.steps):
        v, cores, desc = time_oracle_sample(shape, n, kv_len, parent, tokens, sample_layers)
        if it >= args.warmup:
            vals.append(v)
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": value / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"llama7b verify step: {shape.n_layers} layers + lm_head, n={n}, kv_len={kv_len}",
                   "parallelism": "cpu"},
        "cpu_baseline": {"value": value, "unit": "us", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def slowest_rank(times, dist, device):
    """Replicas run independently; the job is as slow as its slowest rank: element-wise max over ranks."""
    if dist is None:
        return list(times)
    import torch
    t = torch.tensor(list(times), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


# ---------------------------------------------------------------- GPU arm
def run_gpu(args):
    import torch
    import paper_2505_23219_b200 as ghd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    # everything runs on one ordinary (capturable) stream: the end-to-end leg records a whole step into a CUDA graph
    side = torch.cuda.Stream()
    torch.cuda.set_stream(side)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))

    shape, n, kv_len, parent, tokens = workload(args)
    max_kv = kv_len + n
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()

    head = wl.head_weights(shape, CONFIG_ID)
    g_layers, g_kv = [], []
    for l in range(shape.n_layers):
        w = wl.layer_weights(shape, CONFIG_ID, l)
        g_layers.append(ghd.LayerWeights(**{k: dev(w[k]) for k in ghd.LayerWeights.FIELDS}))
        kc, vc = wl.kv_cache(shape, CONFIG_ID, l, kv_len, max_kv)
        g_kv.append(ghd.KvLayer(dev(kc), dev(vc), kv_len))
        del w, kc, vc
    gw = ghd.ModelWeights(dev(head["embed"]), g_layers, dev(head["rms_final"]), dev(head["lm_head"]))
    del head

    cfg = ghd.ModelCfg(shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab, shape.n_layers, max_kv, n,
                       shape.dtype, shape.rms_eps, shape.rope_theta)
    ctx = ghd.ghd_create(cfg)
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, 2)
    for spec in args.opt:
        o, v = spec.split("=")
        ghd.ghd_set_option(ctx, int(o), int(v))
    tree = ghd.Tree(ctx)
    tok_d = dev(tokens)
    amax_d = torch.empty(n, dtype=torch.int32, device="cuda")
    res_d = torch.zeros(2 + 2 * ghd.GHD_MAX_NODES, dtype=torch.int32, device="cuda")
    parent_np = np.asarray(parent, dtype=np.int32)

    def step():
        ghd.ghd_tree_build(ctx, parent_np, kv_len, tree)
        ghd.ghd_verify_step(ctx, gw, g_kv, tree, tok_d, logits=False, argmax=amax_d)
        ghd.ghd_accept(ctx, tree, tok_d, amax_d, res_d)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    ghd.ghd_sync_status(ctx)

    # ---- timed region: K steps, inputs resident
    l0 = ghd.ghd_launch_count(ctx)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        barrier()
        torch.cuda.nvtx.range_push("timed")
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        torch.cuda.nvtx.range_pop()
        launches = ghd.ghd_launch_count(ctx) - l0
        barrier()
        ms = ev0.elapsed_time(ev1)
        # keep sampling a little if the region was very short, so that the clocks line has data
        t_end = time.time() + max(0.0, 1.0 - ms / 1e3)
        while time.time() < t_end:
            step()
        torch.cuda.synchronize()
    ghd.ghd_sync_status(ctx)
    n_matched = int(res_d[0].item())
    ms_per_step = ms / args.steps

    # ---- end to end: host buffers in, host result out, every step.  The caller's side of the public API: one step =
    # copy the tokens in from pinned memory, ghd_tree_build (the parent array travels as launch arguments),
    # ghd_verify_step (plain launches: GHD_OPT_GRAPH = 0), ghd_accept, copy the result out to pinned memory; the
    # caller records that sequence ONCE into a CUDA graph of its own and then, per step, starts the graph and waits
    # for the result on the host.
    tok_h = torch.from_numpy(tokens.copy()).pin_memory()
    res_h = torch.zeros_like(res_d, device="cpu").pin_memory()
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, 0)

    def e2e_step():
        tok_d.copy_(tok_h, non_blocking=True)
        step()
        res_h.copy_(res_d, non_blocking=True)

    for _ in range(2):
        e2e_step()
    side.synchronize()
    ghd.ghd_sync_status(ctx)
    e2e_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(e2e_graph, stream=side):
        e2e_step()
    for _ in range(2):
        e2e_graph.replay()
        side.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        e2e_graph.replay()
        side.synchronize()                                  # the host reads res_h here
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.steps
    ghd.ghd_sync_status(ctx)
    assert int(res_h[0]) == n_matched, "the end-to-end leg accepted a different path"
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, 2)

    # ---- dominant kernel alone, as the step launches it: the gate/up projection with the SwiGLU epilogue
    # (half output), every layer's matrix in turn (each a distinct cold matrix), consecutive launches chained the
    # way they are inside a step (the next kernel sets up while its predecessor drains)
    d, f = shape.d_model, shape.d_ffn
    xh = dev(wl.normal((n, d), 12345, 1.0, dtype="f16"))
    u_out = torch.empty((n, f), dtype=torch.float16, device="cuda")
    reps = 3
    ghd.ghd_set_option(ctx, ghd.OPT_CHAIN_CALLS, 1)
    for lw in g_layers:
        ghd.ghd_gate_up(ctx, xh, lw.t["w_gate_up"], u_out)
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    torch.cuda.nvtx.range_push("roofline")
    k0.record()
    for _ in range(reps):
        for lw in g_layers:
            ghd.ghd_gate_up(ctx, xh, lw.t["w_gate_up"], u_out)
    k1.record()
    torch.cuda.nvtx.range_pop()
    torch.cuda.synchronize()
    ghd.ghd_set_option(ctx, ghd.OPT_CHAIN_CALLS, 0)
    ghd.ghd_sync_status(ctx)
    kern_ms = k0.elapsed_time(k1) / (reps * len(g_layers))
    kern_bytes = 2 * f * d * 2 + n * d * 2 + n * f * 2            # weights + activations in + SwiGLU output (half)
    peak, peak_kind = measured_peak()

    ms_per_step, e2e_ms, kern_ms = slowest_rank([ms_per_step, e2e_ms, kern_ms], dist, "cuda")

    if rank == 0:
        step_bytes = algorithmic_bytes(shape, n, kv_len)
        gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": ms_per_step * 1e3, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": f"llama7b verify step: {shape.n_layers} layers + lm_head (vocab {shape.vocab}), "
                                   f"n={n} ({'medusa' if n == 64 else 'random'} tree), kv_len={kv_len}, f16 weights/KV, "
                                   "f32 accumulate",
                       "parallelism": "replicas" if world > 1 else "single",
                       "cache": "inputs (14.4 GB of weights+KV per step) are larger than L2; no flush needed",
                       "launch": "value: ghd_tree_build + ghd_verify_step (library graph replay) + ghd_accept per step; "
                                 "e2e: the same calls plus the H2D / D2H copies recorded by the caller into one CUDA graph, "
                                 "started and awaited once per step"},
            "step_algorithmic_bytes": step_bytes, "step_hbm_gbs": gbs, "step_pct_of_8tbs": 100 * gbs / 8000.0,
            "step_frac_of_measured_copy_peak": gbs / peak, "steps_per_s_all_ranks": world * 1e3 / ms_per_step,
            "accepted_drafted_tokens": n_matched,
            "clocks": clocks.summary(),
            "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": int(tokens.nbytes + parent_np.nbytes),
                    "d2h_bytes_per_step": int(res_d.numel() * 4)},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": "k_gemm_tc (gate/up projection [2*11008 x 4096] half with the SwiGLU epilogue, as the step launches it)",
                         "achieved": kern_bytes / (kern_ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                         "frac": kern_bytes / (kern_ms * 1e-3) / 1e9 / peak, "peak_kind": f"of {peak_kind}",
                         "us_per_launch": kern_ms * 1e3, "bytes_per_launch": kern_bytes, "traffic": ncu_traffic()},
        }
        if world == 1 and not args.no_cpu:
            v, cores, desc = time_oracle_sample(shape, n, kv_len, parent, tokens, shape.n_layers)      # the whole step, once
            line["cpu_baseline"] = {"value": v, "unit": "us", "cores": cores, "kind": "oracle", "sample": desc}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--nodes", type=int, default=64)
    ap.add_argument("--kv-len", type=int, default=2048)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (default 32)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--opt", action="append", default=[], metavar="ID=VALUE", help="ghd_set_option knob for sweeps (repeatable)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
