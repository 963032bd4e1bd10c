"""GPU parity of the drafting heads (self-drafting as in Medusa, the paper's default drafter) and of a
decode loop that drafts its own trees: verify -> accept -> commit -> draft -> fill, step after step."""
import importlib.util
from pathlib import Path

import numpy as np
import pytest

import oracle
import workloads as wl
from util import gpu_cfg, gpu_layer_weights, max_rel_err, to_dev, tol_for

pytestmark = pytest.mark.gpu

SMALL32 = wl.scaled(wl.TINY, name="small32", d_model=256, n_heads=4, d_head=64, d_ffn=352, vocab=777, n_layers=2)
SMALL16 = wl.scaled(SMALL32, name="small16b", dtype="f16", d_model=512, n_heads=4, d_head=128, d_ffn=704, vocab=2048)

_spec = importlib.util.spec_from_file_location("arca", Path(__file__).resolve().parent.parent / "paper_2505_23219_b200" / "arca.py")
arca = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(arca)


@pytest.fixture(scope="module")
def ghd():
    import paper_2505_23219_b200 as g
    return g


def _heads(shape, seed, k):
    w1 = wl.normal((k, shape.d_model, shape.d_model), seed, 0.05, dtype=shape.dtype)
    w2 = wl.normal((k, shape.vocab, shape.d_model), seed + 1, 0.05, dtype=shape.dtype)
    return w1, w2


def _sorted_topk(z, t):
    return sorted(range(z.size), key=lambda i: (-z[i], i))[:t]


@pytest.mark.parametrize("shape,topk", [(SMALL32, (5, 3, 1)), (SMALL16, (10, 4, 2, 1, 1)), (SMALL16, (16,))], ids=["f32", "f16", "f16top16"])
def test_medusa_draft_against_the_oracle(ghd, shape, topk):
    n, L = 20, 50
    Lmax = L + n
    parent = wl.random_tree(n, 5, 910, max_children=4)
    tokens = wl.draft_tokens(parent, shape.vocab, 911)
    head = wl.head_weights(shape, 41)
    head["rms_final"] = wl.normal((shape.d_model,), 912, 0.1, 1.0, dtype=shape.dtype)
    layers = [wl.layer_weights(shape, 41, l, random_gains=True) for l in range(shape.n_layers)]
    caches = [wl.kv_cache(shape, 41, l, L, Lmax) for l in range(shape.n_layers)]
    vis, _, pos = oracle.tree_build(parent, L)
    _, want_amax, hidden = oracle.step(shape, head, layers, [(k.copy(), v.copy()) for k, v in caches], L, vis, pos, tokens, want_hidden=True)
    c1 = parent.index(0)
    tokens[c1] = want_amax[0]                                  # one accepted draft: the last accepted node is not the root
    _, want_amax, hidden = oracle.step(shape, head, layers, [(k.copy(), v.copy()) for k, v in caches], L, vis, pos, tokens, want_hidden=True)
    m, nodes, toks = oracle.accept(parent, tokens, want_amax)
    assert m >= 1
    w1, w2 = _heads(shape, 920, len(topk))
    h = oracle.rmsnorm(hidden[nodes[m]][None, :], head["rms_final"], shape.rms_eps)[0]
    want_cands, want_logits = oracle.medusa_draft(h, w1, w2, topk)

    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]), to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L) for k, v in caches]
    tree = ghd.ghd_tree_build(ctx, parent, L)
    tok_d = to_dev(tokens)
    for call in range(2):                                      # the second call re-uses the workspace the first one left
        _, amax = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d)
        res = ghd.ghd_accept(ctx, tree, tok_d, amax)
        cand, logits = ghd.ghd_medusa_draft(ctx, ghd.MedusaWeights(to_dev(w1), to_dev(w2)), res, topk, want_logits=True)
        ghd.ghd_sync_status(ctx)
        assert int(res.cpu()[0]) == m
        got = logits.cpu().numpy().astype(np.float64)
        assert max_rel_err(got, want_logits) <= tol_for(shape.dtype)
        cand = cand.cpu().numpy()
        err = np.abs(got - want_logits).max()
        for k, t in enumerate(topk):
            # bit-exact selection on the logits the GPU itself produced (ties to the lower id) ...
            assert list(cand[k, :t]) == _sorted_topk(got[k], t) and (cand[k, t:] == -1).all()
            # ... and the oracle's candidates wherever its ranking is clear of the logit error
            z = np.sort(want_logits[k])[::-1]
            if (z[:t] - z[1:t + 1]).min() > 8.0 * err:
                assert list(cand[k, :t]) == want_cands[k]


def test_medusa_topk_ties_and_fill_tokens_bit_exact(ghd):
    shape = SMALL32
    n, L = 6, 10
    ctx = ghd.ghd_create(gpu_cfg(shape, L + n, 9))             # the tree filled below has 9 nodes
    head = wl.head_weights(shape, 43)
    layers = [wl.layer_weights(shape, 43, l) for l in range(shape.n_layers)]
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]), to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L) for k, v in (wl.kv_cache(shape, 43, l, L, L + n) for l in range(shape.n_layers))]
    parent = wl.chain_tree(n)
    tree = ghd.ghd_tree_build(ctx, parent, L)
    tok_d = to_dev(wl.draft_tokens(parent, shape.vocab, 44))
    _, amax = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d)
    res = ghd.ghd_accept(ctx, tree, tok_d, amax)
    # W1 = 0 and groups of identical W2 rows: exact ties among the logits
    w1 = np.zeros((2, shape.d_model, shape.d_model), np.float32)
    w2 = wl.normal((2, shape.vocab, shape.d_model), 45, 0.05, dtype="f32")
    for r in range(0, shape.vocab - 3, 3):
        w2[:, r + 1] = w2[:, r]
        w2[:, r + 2] = w2[:, r]
    cand, logits = ghd.ghd_medusa_draft(ctx, ghd.MedusaWeights(to_dev(w1), to_dev(w2)), res, (16, 7), want_logits=True)
    ghd.ghd_sync_status(ctx)
    z, cand = logits.cpu().numpy(), cand.cpu().numpy()
    assert (z[:, 0] == z[:, 1]).all() and (z[:, 0] == z[:, 2]).all()
    for k, t in enumerate((16, 7)):
        assert list(cand[k, :t]) == _sorted_topk(z[k].astype(np.float64), t)
    # fill: bonus token at the root, candidates by (level, rank)
    _, paths, _ = arca.build_tree([[0.6, 0.3, 0.1], [0.5, 0.2]], 9)
    level = np.array([len(p) for p in paths], np.int32)
    rank = np.array([p[-1] if p else 0 for p in paths], np.int32)
    got = ghd.ghd_tree_fill_tokens(ctx, to_dev(cand), res, to_dev(level), to_dev(rank)).cpu().numpy()
    r = res.cpu().numpy()
    want = oracle.tree_fill_tokens([list(c) for c in cand], int(r[258 + r[0]]), level, rank)
    assert np.array_equal(got, want)


def test_self_drafting_decode_loop_is_lossless(ghd):
    """verify -> accept -> commit -> draft -> fill with random heads: whatever they draft, the emitted
    tokens are those of the oracle's plain greedy decoding."""
    shape = SMALL32
    L0, total, width = 12, 10, 14
    Lmax = L0 + total + 8 + width
    head = wl.head_weights(shape, 46)
    layers = [wl.layer_weights(shape, 46, l, random_gains=True) for l in range(shape.n_layers)]
    fresh = lambda: [wl.kv_cache(shape, 46, l, L0, Lmax) for l in range(shape.n_layers)]
    o_caches = fresh()
    g, gaps = [5], []
    for s in range(total + 8):
        vis, _, pos = oracle.tree_build([-1], L0 + s)
        logits, am = oracle.step(shape, head, layers, o_caches, L0 + s, vis, pos, [g[-1]])
        top = np.partition(logits[0], -2)
        gaps.append(float(top[-1] - top[-2]) / float(np.abs(logits[0]).max()))
        g.append(int(am[0]))
    assert min(gaps) > 25 * tol_for("f32"), "seed gives a near-tie; pick another"
    acc = [[0.6, 0.3, 0.2, 0.1], [0.5, 0.3, 0.1], [0.4, 0.2]]
    topk = tuple(len(a) for a in acc)
    parent, paths, _ = arca.build_tree(acc, width)
    level = to_dev(np.array([len(p) for p in paths], np.int32))
    rank = to_dev(np.array([p[-1] if p else 0 for p in paths], np.int32))
    w1, w2 = _heads(shape, 930, len(acc))
    mw = ghd.MedusaWeights(to_dev(w1), to_dev(w2))
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]), to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L0) for k, v in fresh()]
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, width))
    tok_d = to_dev(np.array([g[0]] + [0] * (width - 1), np.int32))     # first tree: no drafts yet, arbitrary ids
    L, out = L0, []
    while len(out) < total:
        for kv in gkv:
            kv.len = L
        tree = ghd.ghd_tree_build(ctx, parent, L)
        _, amax = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d)
        res = ghd.ghd_accept(ctx, tree, tok_d, amax)
        ghd.ghd_kv_commit(ctx, gkv, L, res)
        cand = ghd.ghd_medusa_draft(ctx, mw, res, topk)
        tok_d = ghd.ghd_tree_fill_tokens(ctx, cand, res, level, rank)
        r = res.cpu().numpy()
        m = int(r[0])
        out += [int(t) for t in r[258:259 + m]]
        assert int(tok_d.cpu()[0]) == out[-1]                  # the bonus token is the next root
        L += m + 1
    ghd.ghd_sync_status(ctx)
    assert out == g[1:len(out) + 1]


@pytest.mark.parametrize("shape,graph", [(SMALL32, 0), (SMALL16, 0), (SMALL16, 2)], ids=["f32", "f16", "f16graph"])
def test_self_drafting_loop_with_the_cache_length_on_the_device(ghd, shape, graph):
    """The same loop with no host read between steps: the cache length lives in the context's device word, which
    ghd_kv_commit advances; positions, appended rows and attention follow it.  One read-back at the end."""
    import torch
    L0, steps, width = 12, 7, 14
    acc = [[0.6, 0.3, 0.2, 0.1], [0.5, 0.3, 0.1], [0.4, 0.2]]
    most = steps * (len(acc) + 1)
    Lmax = L0 + most + width + 1
    head = wl.head_weights(shape, 46)
    layers = [wl.layer_weights(shape, 46, l, random_gains=True) for l in range(shape.n_layers)]
    fresh = lambda: [wl.kv_cache(shape, 46, l, L0, Lmax) for l in range(shape.n_layers)]
    o_caches = fresh()
    g, gaps, first_logits = [5], [], None
    for s in range(most + 1):
        vis, _, pos = oracle.tree_build([-1], L0 + s)
        logits, am = oracle.step(shape, head, layers, o_caches, L0 + s, vis, pos, [g[-1]])
        first_logits = logits[0].copy() if first_logits is None else first_logits
        top = np.partition(logits[0], -2)
        gaps.append(float(top[-1] - top[-2]))
        g.append(int(am[0]))
    topk = tuple(len(a) for a in acc)
    parent, paths, _ = arca.build_tree(acc, width)
    level = to_dev(np.array([len(p) for p in paths], np.int32))
    rank = to_dev(np.array([p[-1] if p else 0 for p in paths], np.int32))
    w1, w2 = _heads(shape, 930, len(acc))
    mw = ghd.MedusaWeights(to_dev(w1), to_dev(w2))
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]), to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), ghd.KV_LEN_DEVICE) for k, v in fresh()]     # every row finite (generated data)
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, width))
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, graph)
    ghd.ghd_kv_len_set(ctx, L0)
    tok_d = to_dev(np.array([g[0]] + [0] * (width - 1), np.int32))
    tree, results = None, []
    amax = torch.empty(width, dtype=torch.int32, device="cuda")        # fixed buffers: graph mode replays one graph
    logits_d = torch.empty((width, shape.vocab), dtype=torch.float32, device="cuda")
    first = None
    for _ in range(steps):
        tree = ghd.ghd_tree_build(ctx, parent, ghd.KV_LEN_DEVICE, tree=tree)
        ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d, logits=logits_d, argmax=amax)
        first = logits_d[0].clone() if first is None else first
        res = ghd.ghd_accept(ctx, tree, tok_d, amax)
        ghd.ghd_kv_commit(ctx, gkv, ghd.KV_LEN_DEVICE, res)
        cand = ghd.ghd_medusa_draft(ctx, mw, res, topk)
        ghd.ghd_tree_fill_tokens(ctx, cand, res, level, rank, tokens=tok_d)
        results.append(res)
    L_end = ghd.ghd_kv_len_get(ctx)                            # the only synchronising read
    ghd.ghd_sync_status(ctx)
    # token parity needs clear winners: every greedy step's top-1/top-2 gap must dwarf the logit error seen at the root
    err = np.abs(first.cpu().numpy().astype(np.float64) - first_logits).max()
    assert err <= tol_for(shape.dtype) * np.abs(first_logits).max()
    assert min(gaps) > 8.0 * err, "seed gives a near-tie; pick another"
    out = []
    for r in torch.stack(results).cpu().numpy():
        out += [int(t) for t in r[258:259 + int(r[0])]]
    assert steps <= len(out) <= most and L_end == L0 + len(out)
    assert out == g[1:len(out) + 1]
    keep = len(out)
    tol = tol_for(shape.dtype)
    for (ok, ov), kv in zip(o_caches, gkv):
        assert max_rel_err(kv.k.float().cpu().numpy()[:, L0:L0 + keep], ok[:, L0:L0 + keep]) <= tol
        assert max_rel_err(kv.v.float().cpu().numpy()[:, L0:L0 + keep], ov[:, L0:L0 + keep]) <= tol


def test_self_drafting_steps_captured_in_one_cuda_graph(ghd):
    """S consecutive draft / verify / accept / commit steps recorded ONCE into a CUDA graph by the caller and replayed:
    possible because nothing between the steps needs the host (cache length, accepted path, next root and next drafts
    all stay on the device)."""
    import torch
    shape = SMALL16
    L0, steps, width = 12, 6, 14
    acc = [[0.6, 0.3, 0.2, 0.1], [0.5, 0.3, 0.1], [0.4, 0.2]]
    most = steps * (len(acc) + 1)
    Lmax = L0 + most + width + 1
    head = wl.head_weights(shape, 46)
    layers = [wl.layer_weights(shape, 46, l, random_gains=True) for l in range(shape.n_layers)]
    fresh = lambda: [wl.kv_cache(shape, 46, l, L0, Lmax) for l in range(shape.n_layers)]
    o_caches = fresh()
    g, gaps, first_logits = [5], [], None
    for s in range(most + 1):
        vis, _, pos = oracle.tree_build([-1], L0 + s)
        logits, am = oracle.step(shape, head, layers, o_caches, L0 + s, vis, pos, [g[-1]])
        first_logits = logits[0].copy() if first_logits is None else first_logits
        top = np.partition(logits[0], -2)
        gaps.append(float(top[-1] - top[-2]))
        g.append(int(am[0]))
    topk = tuple(len(a) for a in acc)
    parent, paths, _ = arca.build_tree(acc, width)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        level = to_dev(np.array([len(p) for p in paths], np.int32))
        rank = to_dev(np.array([p[-1] if p else 0 for p in paths], np.int32))
        w1, w2 = _heads(shape, 930, len(acc))
        mw = ghd.MedusaWeights(to_dev(w1), to_dev(w2))
        gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]), to_dev(head["lm_head"]))
        gkv = [ghd.KvLayer(to_dev(k), to_dev(v), ghd.KV_LEN_DEVICE) for k, v in fresh()]
        ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, width))        # bound to `stream`
        first_tokens = to_dev(np.array([g[0]] + [0] * (width - 1), np.int32))
        tok_d = first_tokens.clone()
        amax = torch.empty(width, dtype=torch.int32, device="cuda")
        logits_d = torch.empty((width, shape.vocab), dtype=torch.float32, device="cuda")
        results = torch.zeros((steps, 2 + 2 * ghd.GHD_MAX_NODES), dtype=torch.int32, device="cuda")
        tree = ghd.Tree(ctx)

        def one_step(s):
            ghd.ghd_tree_build(ctx, parent, ghd.KV_LEN_DEVICE, tree=tree)
            ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d, logits=logits_d, argmax=amax)
            ghd.ghd_accept(ctx, tree, tok_d, amax, out=results[s])
            ghd.ghd_kv_commit(ctx, gkv, ghd.KV_LEN_DEVICE, results[s])
            cand = ghd.ghd_medusa_draft(ctx, mw, results[s], topk)
            ghd.ghd_tree_fill_tokens(ctx, cand, results[s], level, rank, tokens=tok_d)

        ghd.ghd_kv_len_set(ctx, L0)
        one_step(0)                                             # warm-up outside the capture (one-time set-up calls)
        first = logits_d[0].clone()
        ghd.ghd_sync_status(ctx)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for s in range(steps):
                one_step(s)
        for rep in range(2):                                    # the same graph, started twice from the same state
            ghd.ghd_kv_len_set(ctx, L0)
            tok_d.copy_(first_tokens)
            graph.replay()
            L_end = ghd.ghd_kv_len_get(ctx)
            ghd.ghd_sync_status(ctx)
            out = []
            for r in results.cpu().numpy():
                out += [int(t) for t in r[258:259 + int(r[0])]]
            assert steps <= len(out) <= most and L_end == L0 + len(out)
            assert out == g[1:len(out) + 1]
    err = np.abs(first.cpu().numpy().astype(np.float64) - first_logits).max()
    assert err <= tol_for(shape.dtype) * np.abs(first_logits).max()
    assert min(gaps) > 8.0 * err, "seed gives a near-tie; pick another"
