"""GPU parity at the full sizes of the five benchmark configurations (config 1 and 2
live in test_gpu_parity.py): the tree-size sweep on the 7B-shaped layer, the 13B-shaped
stress layer with a 256-node tree and a lookahead-style explicit mask, and the full
32-layer verify step against stored oracle results."""
import json
from pathlib import Path

import numpy as np
import pytest

import oracle
import workloads as wl
from util import gpu_cfg, gpu_layer_weights, max_rel_err, to_dev, tol_for

pytestmark = pytest.mark.gpu
GOLDEN = Path(__file__).resolve().parent / "golden"


@pytest.fixture(scope="module")
def ghd():
    import paper_2505_23219_b200 as g
    return g


def _layer_parity(ghd, shape, w, gw, config_id, n, L, parent=None, vis=None, depth=None, sparse=0):
    Lmax = L + n
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    ghd.ghd_set_option(ctx, ghd.OPT_ATTN_SPARSE, sparse)
    kc, vc = wl.kv_cache(shape, config_id, 0, L, Lmax)
    x = wl.layer_input(shape, config_id, n)
    if vis is None:
        ovis, _, opos = oracle.tree_build(parent, L)
        tree = ghd.ghd_tree_build(ctx, parent, L)
    else:
        ovis, opos = vis.astype(np.uint8), (L + depth).astype(np.int32)
        tree = ghd.ghd_tree_from_mask(ctx, ghd.pack_mask(vis), L, depth=depth)
    okc, ovc = kc.copy(), vc.copy()
    want = oracle.layer(shape, w, okc, ovc, L, ovis, opos, x)
    kv = ghd.KvLayer(to_dev(kc), to_dev(vc), L)
    y = ghd.ghd_verify_layer(ctx, gw, kv, tree, to_dev(x))
    ghd.ghd_sync_status(ctx)
    tol = tol_for(shape.dtype)
    err = max_rel_err(y.float().cpu().numpy(), want)
    kerr = max_rel_err(kv.k.float().cpu().numpy()[:, L:], okc[:, L:])
    verr = max_rel_err(kv.v.float().cpu().numpy()[:, L:], ovc[:, L:])
    assert err <= tol and kerr <= tol and verr <= tol, (n, L, err, kerr, verr)
    ghd.ghd_destroy(ctx)
    return err


def test_config4_tree_size_sweep_on_the_7b_layer(ghd):
    """N in {1..256} x KV length in {512, 2048, 4096}, random trees of depth <= 8."""
    shape = wl.LLAMA7B
    w = wl.layer_weights(shape, 4, 0)
    gw = gpu_layer_weights(w)
    worst = 0.0
    for L in (512, 2048, 4096):
        for n in (1, 4, 8, 16, 32, 64, 128, 256):
            parent = wl.random_tree(n, 8, wl.BASE_SEED + 4000 + n + L)
            worst = max(worst, _layer_parity(ghd, shape, w, gw, 4, n, L, parent=parent))
    assert worst <= 2e-2


def test_config5_llama13b_layer_wide_tree_and_lookahead_mask(ghd):
    """13B-shaped layer, KV 4096: 256-node tree (depth 8, <= 6 children) and the 49-node
    lookahead pattern (window 7, 5 guess n-grams) given as an explicit mask."""
    shape = wl.LLAMA13B
    w = wl.layer_weights(shape, 5, 0)
    gw = gpu_layer_weights(w)
    parent = wl.random_tree(256, 8, wl.BASE_SEED + 5000, max_children=6)
    assert max(wl.depths_of(parent)) == 8
    _layer_parity(ghd, shape, w, gw, 5, 256, 4096, parent=parent)
    _layer_parity(ghd, shape, w, gw, 5, 256, 4096, parent=parent, sparse=1)        # sparse part from the coordinate index
    vis, depth, _ = wl.lookahead_pattern(7, 5, 5)
    _layer_parity(ghd, shape, w, gw, 5, vis.shape[0], 4096, vis=vis, depth=depth)
    _layer_parity(ghd, shape, w, gw, 5, vis.shape[0], 4096, vis=vis, depth=depth, sparse=1)


def test_config3_full_32_layer_step_against_stored_oracle_results(ghd):
    """Same launch configuration as the benchmark (graph replay).  Expected values come from
    tests/golden/c3_step_llama7b.json, written by make_c3_fixture.py from the CPU oracle alone."""
    fx = json.loads((GOLDEN / "c3_step_llama7b.json").read_text())
    shape, cid, L, n = wl.LLAMA7B, fx["config"]["config_id"], fx["config"]["kv_len"], fx["config"]["n"]
    Lmax = L + n
    parent = fx["parent"]
    assert parent == wl.medusa_tree(n)
    tokens = np.asarray(fx["tokens"], dtype=np.int32)
    head = wl.head_weights(shape, cid)
    layers, kvs = [], []
    for l in range(shape.n_layers):
        layers.append(gpu_layer_weights(wl.layer_weights(shape, cid, l)))
        kc, vc = wl.kv_cache(shape, cid, l, L, Lmax)
        kvs.append(ghd.KvLayer(to_dev(kc), to_dev(vc), L))
    gw = ghd.ModelWeights(to_dev(head["embed"]), layers, to_dev(head["rms_final"]), to_dev(head["lm_head"]))
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, n))
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, 2)
    tree = ghd.ghd_tree_build(ctx, parent, L)
    tok = to_dev(tokens)
    for _ in range(2):                                         # capture, then replay
        logits, amax = ghd.ghd_verify_step(ctx, gw, kvs, tree, tok)
    hidden = ghd.ghd_copy_hidden(ctx, n)
    res = ghd.ghd_accept(ctx, tree, tok, amax).cpu().numpy()
    ghd.ghd_sync_status(ctx)
    got = logits.cpu().numpy()
    # the last layer's output (before the final norm) on the stored sample of columns, every node
    hid = hidden.cpu().numpy()[:, fx["hidden_cols"]].astype(np.float64)
    assert np.abs(hid - np.asarray(fx["hidden_samples"])).max() / fx["hidden_abs_max"] <= 2e-2
    # sampled logits (512 columns per node, the oracle's top 8 among them), normalised by the oracle's largest |logit|
    abs_err = 0.0
    assert len(fx["logit_samples"]) == n and all(len(r["cols"]) >= 512 for r in fx["logit_samples"])
    for srow in fx["logit_samples"]:
        g = got[srow["node"], srow["cols"]].astype(np.float64)
        abs_err = max(abs_err, float(np.abs(g - np.asarray(srow["values"])).max()))
    assert abs_err / fx["logits_abs_max"] <= 2e-2
    # argmax tokens: exact where the oracle's top-2 gap clears 8x the observed error, else top-1 or runner-up
    amax = amax.cpu().numpy()
    decided = 0
    for i in range(n):
        if fx["row_margins"][i] > 8.0 * abs_err:
            assert amax[i] == fx["argmax"][i], (i, fx["row_margins"][i], abs_err)
            decided += 1
        else:
            assert amax[i] in (fx["argmax"][i], fx["runner_up"][i])
    assert decided >= n // 2
    # acceptance: the planted path of three drafted tokens
    m = fx["n_matched"]
    assert res[0] == m == 3 and res[1] == m + 1
    assert list(res[2:3 + m]) == fx["accepted_nodes"]
    for j, node in enumerate(fx["accepted_nodes"]):
        if fx["row_margins"][node] > 8.0 * abs_err:
            assert res[258 + j] == fx["emitted_tokens"][j]
