"""GPU parity of the step after verification: KV commit, and several speculative steps in a row
(verify -> accept -> commit -> next root) against plain greedy decoding by the oracle."""
import numpy as np
import pytest

import oracle
import workloads as wl
from util import gpu_cfg, gpu_layer_weights, max_rel_err, to_dev, tol_for

pytestmark = pytest.mark.gpu

SMALL32 = wl.scaled(wl.TINY, name="small32", d_model=256, n_heads=4, d_head=64, d_ffn=352, vocab=777, n_layers=2)
SMALL16 = wl.scaled(SMALL32, name="small16b", dtype="f16", d_model=512, n_heads=4, d_head=128, d_ffn=704)


@pytest.fixture(scope="module")
def ghd():
    import paper_2505_23219_b200 as g
    return g


def _greedy(sh, head, layers, caches, L, first_tok, count):
    """Oracle: sequential single-token decoding.
    -> (tokens [first, g1, ...], top-1/top-2 logit gap of every step, logits of the first step)."""
    seq, gaps, first = [int(first_tok)], [], None
    for s in range(count):
        vis, _, pos = oracle.tree_build([-1], L + s)
        logits, am = oracle.step(sh, head, layers, caches, L + s, vis, pos, [seq[-1]])
        first = logits[0].copy() if first is None else first
        top = np.partition(logits[0], -2)
        gaps.append(float(top[-1] - top[-2]))
        seq.append(int(am[0]))
    return seq, gaps, first


def _plant(parent, tokens, chain_tokens, vocab):
    tokens = np.array(tokens, dtype=np.int32)
    node = 0
    for t in chain_tokens:
        kids = [c for c, p in enumerate(parent) if p == node]
        if not kids:
            break
        tokens[kids[0]] = t
        for c in kids[1:]:
            while tokens[c] == t or any(tokens[c] == tokens[o] for o in kids if o != c):
                tokens[c] = (tokens[c] + 1) % vocab
        node = kids[0]
    return tokens


def test_kv_commit_moves_exactly_the_accepted_rows(ghd):
    shape, L, n = SMALL16, 37, 40
    Lmax = L + n
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    caches = [wl.kv_cache(shape, 31, l, Lmax, Lmax) for l in range(3)]        # every row holds data
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L) for k, v in caches]
    for nodes in ([0], [0, 1, 2, 3], [0, 3, 17, 18, 39], [0, 2, 4, 6, 8, 10, 12, 14, 16, 18, 20]):
        res = np.zeros(2 + 2 * ghd.GHD_MAX_NODES, dtype=np.int32)
        res[0], res[1] = len(nodes) - 1, len(nodes)
        res[2:2 + len(nodes)] = nodes
        ghd.ghd_kv_commit(ctx, gkv, L, to_dev(res))
        ghd.ghd_sync_status(ctx)
        oracle.kv_commit(caches, L, nodes)
        for (k, v), g in zip(caches, gkv):
            assert np.array_equal(g.k.cpu().numpy(), k) and np.array_equal(g.v.cpu().numpy(), v)   # a copy: bit-exact


@pytest.mark.parametrize("shape,graph", [(SMALL32, 0), (SMALL16, 0), (SMALL16, 2)], ids=["f32", "f16", "f16graph"])
def test_speculative_steps_emit_the_oracle_greedy_sequence(ghd, shape, graph):
    L0, total, n = 20, 14, 12
    Lmax = L0 + total + 8 + n
    head = wl.head_weights(shape, 42)
    layers = [wl.layer_weights(shape, 42, l, random_gains=True) for l in range(shape.n_layers)]
    fresh = lambda: [wl.kv_cache(shape, 42, l, L0, Lmax) for l in range(shape.n_layers)]
    o_caches = fresh()
    g, gaps, first_logits = _greedy(shape, head, layers, o_caches, L0, 5, total + 8)
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]),
                          to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L0) for k, v in fresh()]
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, graph)
    L, root, out, step_no = L0, g[0], [], 0
    while len(out) < total:
        parent = wl.random_tree(n, 4, 500 + step_no, max_children=3)
        at = len(out)
        tokens = _plant(parent, wl.draft_tokens(parent, shape.vocab, 600 + step_no), g[at + 1:at + 1 + step_no % 4], shape.vocab)
        tokens[0] = root
        for kv in gkv:
            kv.len = L
        tree = ghd.ghd_tree_build(ctx, parent, L)
        tok_d = to_dev(tokens)
        logits, amax = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d)
        if step_no == 0:
            # token parity needs clear winners: every greedy step's top-1/top-2 gap must dwarf the logit error seen here
            err = np.abs(logits[0].cpu().numpy().astype(np.float64) - first_logits).max()
            assert err <= tol_for(shape.dtype) * np.abs(first_logits).max()
            assert min(gaps) > 8.0 * err, "seed gives a near-tie; pick another"
        res_d = ghd.ghd_accept(ctx, tree, tok_d, amax)
        ghd.ghd_kv_commit(ctx, gkv, L, res_d)
        res = res_d.cpu().numpy()
        m = int(res[0])
        out += [int(t) for t in res[258:259 + m]]
        L += m + 1
        root = out[-1]
        step_no += 1
    ghd.ghd_sync_status(ctx)
    assert out == g[1:len(out) + 1]
    assert step_no < total                                    # drafts were accepted along the way
    # the committed cache is the cache of sequential decoding of the same tokens
    keep = min(L - L0, total + 8)
    tol = tol_for(shape.dtype)
    for (ok, ov), kv in zip(o_caches, gkv):
        assert max_rel_err(kv.k.float().cpu().numpy()[:, L0:L0 + keep], ok[:, L0:L0 + keep]) <= tol
        assert max_rel_err(kv.v.float().cpu().numpy()[:, L0:L0 + keep], ov[:, L0:L0 + keep]) <= tol


def _accepted(parent, tokens, greedy_next):
    """Accepted path when the target's argmax along it is the greedy sequence: -> number of matched drafts."""
    node, m = 0, 0
    while True:
        kids = [c for c, p in enumerate(parent) if p == node and tokens[c] == greedy_next[m]]
        if not kids:
            return m
        node, m = kids[0], m + 1


@pytest.mark.parametrize("shape,graph", [(SMALL32, 0), (SMALL16, 0), (SMALL16, 2)], ids=["f32", "f16", "f16graph"])
def test_speculative_steps_without_a_host_read_between_steps(ghd, shape, graph):
    """The cache length lives in the context's device word (GHD_KV_LEN_DEVICE): tree positions, appended rows,
    attention and commit follow it, ghd_kv_commit advances it, the next root token is picked on the device.
    The drafts of every step are planted from the oracle's greedy sequence, whose acceptance the host can
    foresee, so all steps are enqueued before anything is read back."""
    import torch
    L0, steps, n = 20, 6, 12
    plant = [s % 4 for s in range(steps)]
    most = sum(plant) + steps + 4
    Lmax = L0 + most + n + 1
    head = wl.head_weights(shape, 42)
    layers = [wl.layer_weights(shape, 42, l, random_gains=True) for l in range(shape.n_layers)]
    fresh = lambda: [wl.kv_cache(shape, 42, l, L0, Lmax) for l in range(shape.n_layers)]
    o_caches = fresh()
    g, gaps, first_logits = _greedy(shape, head, layers, o_caches, L0, 5, most + 4)
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]),
                          to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), ghd.KV_LEN_DEVICE) for k, v in fresh()]
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, graph)
    ghd.ghd_kv_len_set(ctx, L0)
    tok_d = torch.zeros(n, dtype=torch.int32, device="cuda")
    amax = torch.empty(n, dtype=torch.int32, device="cuda")
    logits = torch.empty((n, shape.vocab), dtype=torch.float32, device="cuda")
    tree, results, want_m, at = None, [], [], 0
    first = None
    for s in range(steps):
        parent = wl.random_tree(n, 4, 500 + s, max_children=3)
        tokens = _plant(parent, wl.draft_tokens(parent, shape.vocab, 600 + s), g[at + 1:at + 1 + plant[s]], shape.vocab)
        tokens[0] = g[at]                                       # the host's forecast; the device overwrites it below
        m = _accepted(parent, tokens, g[at + 1:])
        want_m.append(m)
        at += m + 1
        new_tok = to_dev(tokens)
        if results:                                            # root = last token the previous step emitted, taken on the device
            prev = results[-1]
            new_tok[0:1] = prev[(258 + prev[0:1]).long()]
        tok_d.copy_(new_tok)
        tree = ghd.ghd_tree_build(ctx, parent, ghd.KV_LEN_DEVICE, tree=tree)
        ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d, logits=logits, argmax=amax)
        if s == 0:
            first = logits[0].clone()
        res = ghd.ghd_accept(ctx, tree, tok_d, amax)
        ghd.ghd_kv_commit(ctx, gkv, ghd.KV_LEN_DEVICE, res)
        results.append(res)
    L_end = ghd.ghd_kv_len_get(ctx)                            # the only synchronising read of the loop
    ghd.ghd_sync_status(ctx)
    err = np.abs(first.cpu().numpy().astype(np.float64) - first_logits).max()
    assert err <= tol_for(shape.dtype) * np.abs(first_logits).max()
    assert min(gaps) > 8.0 * err, "seed gives a near-tie; pick another"
    out, got_m = [], []
    for r in torch.stack(results).cpu().numpy():
        got_m.append(int(r[0]))
        out += [int(t) for t in r[258:259 + int(r[0])]]
    assert got_m == want_m and sum(want_m) > 0                  # drafts were accepted along the way
    assert out == g[1:len(out) + 1] and L_end == L0 + len(out)
    tol = tol_for(shape.dtype)
    for (ok, ov), kv in zip(o_caches, gkv):
        assert max_rel_err(kv.k.float().cpu().numpy()[:, L0:L_end], ok[:, L0:L_end]) <= tol
        assert max_rel_err(kv.v.float().cpu().numpy()[:, L0:L_end], ov[:, L0:L_end]) <= tol


def test_a_cache_length_on_the_device_that_leaves_the_cache_is_reported(ghd):
    """The word is clamped by every kernel (nothing is written out of bounds) and the tree kernel records the overflow."""
    shape, n = SMALL16, 12
    Lmax = 40
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    ghd.ghd_kv_len_set(ctx, Lmax - 3)                           # 37 + 12 nodes > 40 rows
    ghd.ghd_tree_build(ctx, wl.random_tree(n, 4, 1), ghd.KV_LEN_DEVICE)
    with pytest.raises(ghd.GhdError) as err:
        ghd.ghd_sync_status(ctx)
    assert "GHD_ENOSPACE" in str(err.value)
    ghd.ghd_sync_status(ctx)                                    # cleared
    assert ghd.ghd_kv_len_get(ctx) == Lmax - 3
    ghd.ghd_kv_len_set(ctx, 5)
    ghd.ghd_tree_build(ctx, wl.random_tree(n, 4, 1), ghd.KV_LEN_DEVICE)
    ghd.ghd_sync_status(ctx)
