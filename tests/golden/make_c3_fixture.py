"""Writes tests/golden/c3_step_llama7b.json: the CPU oracle's results for the full
32-layer LLaMA-7B-shaped verify step (KV length 2048, 64-node Medusa-style tree,
vocab 32000) with a planted accepted path of three drafted tokens.

Calls only ``oracle`` and ``workloads``; nothing here comes from the CUDA path.
Takes a few minutes and ~20 GB of host memory.  Run from the repo root:

    python tests/golden/make_c3_fixture.py
"""
import json
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parents[2]
sys.path.insert(0, str(ROOT))

import oracle  # noqa: E402
import workloads as wl  # noqa: E402

CONFIG_ID = 3
KV_LEN = 2048
N = 64
PLANT = 3
SAMPLES_PER_ROW = 512      # logit columns stored per node, the oracle's top 8 among them
HIDDEN_COLS = 64           # columns of the last layer's output stored per node


def main():
    shape = wl.LLAMA7B
    max_kv = KV_LEN + N
    t0 = time.time()
    head = wl.head_weights(shape, CONFIG_ID)
    layers = [wl.layer_weights(shape, CONFIG_ID, l) for l in range(shape.n_layers)]
    fresh = lambda: [wl.kv_cache(shape, CONFIG_ID, l, KV_LEN, max_kv) for l in range(shape.n_layers)]
    print(f"inputs generated in {time.time() - t0:.0f}s", flush=True)

    parent = wl.medusa_tree(N)
    tokens = wl.draft_tokens(parent, shape.vocab, wl.BASE_SEED + 1000 * CONFIG_ID + 700)
    # the tree's top-1 chain: first child of the root, its first child, ...
    chain = [0]
    for _ in range(PLANT):
        chain.append(parent.index(chain[-1]))

    # k sequential greedy single-token steps from the root token give the tokens to plant
    # (a width-1 tree of depth k reproduces k sequential decode steps)
    caches = fresh()
    tok, greedy = int(tokens[0]), []
    for s in range(PLANT + 1):
        vis, _, pos = oracle.tree_build([-1], KV_LEN + s)
        _, am = oracle.step(shape, head, layers, caches, KV_LEN + s, vis, pos, [tok])
        tok = int(am[0])
        greedy.append(tok)
        print(f"sequential step {s}: token {tok}  ({time.time() - t0:.0f}s)", flush=True)
    for node, g in zip(chain[1:], greedy[:PLANT]):
        tokens[node] = g
    # the path must stop after PLANT drafted tokens, and siblings must stay distinct
    for c in [c for c, p in enumerate(parent) if p == chain[-1]]:
        if tokens[c] == greedy[PLANT]:
            tokens[c] = (tokens[c] + 1) % shape.vocab
    for p in set(parent):
        sib = [int(tokens[c]) for c, q in enumerate(parent) if q == p]
        assert len(sib) == len(set(sib)), "duplicate sibling tokens after planting"

    vis, depth, pos = oracle.tree_build(parent, KV_LEN)
    logits, amax, hidden = oracle.step(shape, head, layers, fresh(), KV_LEN, vis, pos, tokens, want_hidden=True)
    print(f"full step done ({time.time() - t0:.0f}s)", flush=True)
    m, nodes, emitted = oracle.accept(parent, tokens, amax)
    assert m == PLANT and list(nodes) == chain, (m, list(nodes), chain)

    part = np.partition(logits, -2, axis=1)
    margins = part[:, -1] - part[:, -2]
    rng = wl.Rng(wl.BASE_SEED + 1000 * CONFIG_ID + 701)
    samples = []
    for i in range(N):
        cols = {int(c) for c in np.argsort(logits[i])[-8:]}
        while len(cols) < SAMPLES_PER_ROW:
            cols.add(rng.below(shape.vocab))
        cols = sorted(cols)
        samples.append({"node": i, "cols": cols, "values": [float(f"{logits[i, c]:.9e}") for c in cols]})
    hcols = sorted({rng.below(shape.d_model) for _ in range(4 * HIDDEN_COLS)})[:HIDDEN_COLS]
    out = {
        "source": "tests/golden/make_c3_fixture.py (CPU oracle only)",
        "config": {"shape": shape.name, "config_id": CONFIG_ID, "kv_len": KV_LEN, "n": N, "tree": "medusa_tree(64)"},
        "parent": list(map(int, parent)),
        "tokens": list(map(int, tokens)),
        "argmax": list(map(int, amax)),
        "n_matched": int(m),
        "accepted_nodes": list(map(int, nodes)),
        "emitted_tokens": list(map(int, emitted)),
        "logits_abs_max": float(np.abs(logits).max()),
        "min_top2_margin": float(margins.min()),
        "row_margins": [float(f"{v:.6e}") for v in margins],
        "runner_up": [int(np.argsort(logits[i])[-2]) for i in range(N)],
        "logit_samples": samples,
        "hidden_abs_max": float(np.abs(hidden).max()),
        "hidden_cols": hcols,
        "hidden_samples": [[float(f"{hidden[i, c]:.9e}") for c in hcols] for i in range(N)],
    }
    path = Path(__file__).resolve().parent / "c3_step_llama7b.json"
    path.write_text(json.dumps(out, separators=(",", ":")).replace("},{", "},\n{"))
    print(f"wrote {path} ({time.time() - t0:.0f}s); min top-2 margin {margins.min():.4f}", flush=True)


if __name__ == "__main__":
    main()
