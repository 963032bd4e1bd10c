"""Pins of the CPU oracle against things other than itself: hand-derived
fixtures, closed forms, brute force written a different way, textbook/library
special cases and the invariants of tree verification.  CPU only."""
import itertools
from pathlib import Path

import numpy as np
import pytest

import oracle
import workloads as wl

GOLDEN = Path(__file__).resolve().parent / "golden"


def _rows(name):
    return [l.split() for l in (GOLDEN / name).read_text().splitlines() if l.strip() and not l.startswith("#")]


# ---------------------------------------------------------------- tree build
def test_tree_worked_example_fixture():
    rows = _rows("tree_worked_example.txt")
    parent = [int(r[1]) for r in rows]
    vis, depth, pos = oracle.tree_build(parent, kv_len=10)
    for r in rows:
        i = int(r[0])
        assert depth[i] == int(r[2])
        assert pos[i] == int(r[3])
        assert set(np.nonzero(vis[i])[0]) == {int(t) for t in r[4].split(",")}


def _ancestors_by_sets(parent):
    anc = []
    for i, p in enumerate(parent):
        anc.append({i} | (anc[p] if p >= 0 else set()))
    return anc


@pytest.mark.parametrize("n,seed", [(1, 0), (2, 1), (8, 2), (63, 3), (64, 4), (65, 5), (200, 6), (256, 7)])
def test_tree_build_matches_set_recursion(n, seed):
    parent = wl.random_tree(n, 8, seed)
    vis, depth, pos = oracle.tree_build(parent, kv_len=77)
    anc = _ancestors_by_sets(parent)
    for i in range(n):
        assert set(np.nonzero(vis[i])[0]) == anc[i]
        assert depth[i] == len(anc[i]) - 1 == vis[i].sum() - 1
        assert pos[i] == 77 + depth[i]
        for j in anc[i]:                                  # closure: ancestors' sets are subsets
            assert anc[j] <= anc[i]


def test_tree_build_chain_and_star():
    vis, depth, _ = oracle.tree_build(wl.chain_tree(9), 0)
    assert np.array_equal(vis, np.tril(np.ones((9, 9), dtype=np.uint8)))
    assert list(depth) == list(range(9))
    vis, depth, _ = oracle.tree_build(wl.star_tree(9), 0)
    want = np.eye(9, dtype=np.uint8)
    want[:, 0] = 1
    assert np.array_equal(vis, want)
    assert list(depth) == [0] + [1] * 8


@pytest.mark.parametrize("n,seed", [(1, 0), (9, 1), (64, 2), (130, 3), (256, 4)])
def test_coo_index_lists_every_root_path(n, seed):
    """For a tree the index of node i is its root path in ascending order: depth + 1 entries, ending in i,
    each entry the parent of the next; the total is the sum of depth + 1."""
    parent = wl.random_tree(n, 8, 900 + seed, max_children=6)
    vis, depth, _ = oracle.tree_build(parent, 5)
    ptr, cols = oracle.coo_index(vis)
    assert ptr[0] == 0 and ptr[-1] == len(cols) == int((depth + 1).sum())
    for i in range(n):
        path = list(cols[ptr[i]:ptr[i + 1]])
        assert len(path) == depth[i] + 1 and path[-1] == i and path[0] == 0
        assert all(parent[b] == a for a, b in zip(path, path[1:]))


def test_coo_index_of_an_arbitrary_mask_round_trips():
    rng = np.random.default_rng(4)
    vis = np.tril(rng.random((37, 37)) < 0.3)
    np.fill_diagonal(vis, True)
    ptr, cols = oracle.coo_index(vis)
    back = np.zeros_like(vis)
    for i in range(37):
        assert list(cols[ptr[i]:ptr[i + 1]]) == sorted(cols[ptr[i]:ptr[i + 1]])
        back[i, cols[ptr[i]:ptr[i + 1]]] = True
    assert np.array_equal(back, vis) and ptr[-1] == vis.sum()


@pytest.mark.parametrize("bad", [[], [0], [-1, 1], [-1, -1], [-1, 0, 3], [-1, 0, 2]])
def test_tree_build_rejects_bad_parent(bad):
    with pytest.raises(ValueError):
        oracle.tree_build(bad, 0)


def test_lookahead_pattern_is_the_tree_of_its_parent_array():
    vis, depth, parent = wl.lookahead_pattern(7, 5, 5)
    assert vis.shape == (49, 49)
    v2, d2, _ = oracle.tree_build(parent, 0)
    assert np.array_equal(v2.astype(bool), vis)
    assert np.array_equal(d2, depth)


def test_medusa_tree_shape():
    parent = wl.medusa_tree(64, (10, 4, 2, 1, 1))
    assert len(parent) == 64 and max(wl.depths_of(parent)) == 5
    depth = wl.depths_of(parent)
    for node in range(64):                                 # per-level branching caps hold
        kids = [c for c, p in enumerate(parent) if p == node]
        assert len(kids) <= (10, 4, 2, 1, 1, 0)[depth[node]]


# ---------------------------------------------------------------- rmsnorm
def test_rmsnorm_constant_row_closed_form():
    d, c, eps = 16, 3.0, 1e-6
    g = np.linspace(0.5, 2.0, d).astype(np.float32)
    out = oracle.rmsnorm(np.full((2, d), c), g, eps)
    assert np.allclose(out, g.astype(np.float64) * c / np.sqrt(c * c + eps), rtol=1e-14)


def test_rmsnorm_scale_invariance_and_unit_rms():
    x = wl.normal((5, 64), 11).astype(np.float64)
    g = np.ones(64, dtype=np.float32)
    a, b = oracle.rmsnorm(x, g, 0.0), oracle.rmsnorm(7.5 * x, g, 0.0)
    assert np.allclose(a, b, rtol=1e-13)
    assert np.allclose((a * a).mean(axis=1), 1.0, rtol=1e-13)


# ---------------------------------------------------------------- linear
@pytest.mark.parametrize("dt", ["f32", "f16"])
def test_linear_is_x_times_w_transposed(dt):
    x = wl.normal((7, 40), 21).astype(np.float64)
    w = wl.normal((13, 40), 22, 0.02, dtype=dt)
    assert np.allclose(oracle.linear(x, w), x @ w.astype(np.float64).T, rtol=1e-12, atol=1e-15)


def test_linear_identity_and_single_entry():
    x = wl.normal((3, 8), 23).astype(np.float64)
    assert np.array_equal(oracle.linear(x, np.eye(8, dtype=np.float32)), x)
    w = np.zeros((5, 8), dtype=np.float32)
    w[4, 2] = 2.0                                          # output feature 4 reads input feature 2
    y = oracle.linear(x, w)
    assert np.array_equal(y[:, 4], 2.0 * x[:, 2]) and not y[:, :4].any()


# ---------------------------------------------------------------- rope
def test_rope_is_a_plane_rotation_by_pos():
    # d_head = 2: one pair, frequency theta^0 = 1 -> rotation by `pos` radians.
    u = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])
    r = oracle.rope(u, [3, 5], 10000.0)
    assert np.allclose(r[0, 0], [np.cos(3.0), np.sin(3.0)], atol=1e-15)
    assert np.allclose(r[1, 0], [-np.sin(5.0), np.cos(5.0)], atol=1e-15)


def test_rope_pairing_and_frequencies():
    # d_head = 4: pairs (0,2) and (1,3); second pair turns by pos * theta^(-1/2).
    u = np.array([[[1.0, 1.0, 0.0, 0.0]]])
    r = oracle.rope(u, [2], 100.0)[0, 0]
    assert np.allclose(r, [np.cos(2.0), np.cos(0.2), np.sin(2.0), np.sin(0.2)], atol=1e-15)


def test_rope_identity_norm_and_relative_property():
    q = wl.normal((1, 2, 16), 31).astype(np.float64)
    k = wl.normal((1, 2, 16), 32).astype(np.float64)
    assert np.array_equal(oracle.rope(q, [0], 10000.0), q)
    rq = oracle.rope(q, [17], 10000.0)
    assert np.allclose((rq ** 2).sum(-1), (q ** 2).sum(-1), rtol=1e-13)
    dots = [(oracle.rope(q, [m], 1e4) * oracle.rope(k, [m - 4], 1e4)).sum(-1) for m in (4, 9, 40)]
    assert np.allclose(dots[0], dots[1], rtol=1e-11) and np.allclose(dots[0], dots[2], rtol=1e-11)


# ---------------------------------------------------------------- attention
def _rand_attn_inputs(n, h, dh, L, Lmax, seed, dt="f32"):
    q = wl.normal((n, h, dh), seed).astype(np.float64)
    kn = wl.normal((n, h, dh), seed + 1).astype(np.float64)
    vn = wl.normal((n, h, dh), seed + 2).astype(np.float64)
    kc = np.zeros((h, Lmax, dh), dtype=np.float32 if dt == "f32" else np.float16)
    vc = np.zeros_like(kc)
    kc[:, :L] = wl.normal((h, L, dh), seed + 3, dtype=dt)
    vc[:, :L] = wl.normal((h, L, dh), seed + 4, dtype=dt)
    return q, kn, vn, kc, vc


def test_attention_zero_keys_gives_mean_of_visible_values():
    n, h, dh, L, Lmax = 12, 2, 8, 5, 32
    parent = wl.random_tree(n, 4, 41)
    vis, depth, _ = oracle.tree_build(parent, L)
    q, kn, vn, kc, vc = _rand_attn_inputs(n, h, dh, L, Lmax, 42)
    kn[:] = 0
    kc[:] = 0
    out = oracle.tree_attention(q, kn, vn, kc, vc, L, vis)
    anc = _ancestors_by_sets(parent)
    for i in range(n):
        for hh in range(h):
            rows = [vc[hh, j].astype(np.float64) for j in range(L)] + [vn[j, hh] for j in sorted(anc[i])]
            assert len(rows) == L + depth[i] + 1
            assert np.allclose(out[i, hh], np.mean(rows, axis=0), rtol=1e-13, atol=1e-15)


def test_attention_scale_is_inverse_sqrt_dhead():
    # one head, d_head 4, no cache, chain of 2: node 1 sees keys k0 = 0 and k1 = c*ones,
    # q1 = a*ones -> scores 0 and 4ac/sqrt(4) = 2ac.
    a, c = 0.7, 0.9
    q = np.zeros((2, 1, 4)); q[1] = a
    kn = np.zeros((2, 1, 4)); kn[1] = c
    vn = np.zeros((2, 1, 4)); vn[0, 0, 0] = 1.0; vn[1, 0, 1] = 1.0
    empty = np.zeros((1, 4, 4), dtype=np.float32)
    vis, _, _ = oracle.tree_build([-1, 0], 0)
    out = oracle.tree_attention(q, kn, vn, empty, empty, 0, vis)
    p1 = 1.0 / (1.0 + np.exp(-2 * a * c))
    assert np.allclose(out[1, 0], [1 - p1, p1, 0, 0], rtol=1e-14)
    assert np.allclose(out[0, 0], [1, 0, 0, 0])            # L = 0, node 0 alone -> its own value


def _causal_attention_numpy(q_all, k_all, v_all):
    """Textbook causal softmax attention over one sequence, [T][h][dh] each."""
    T, h, dh = q_all.shape
    out = np.zeros_like(q_all)
    for hh in range(h):
        s = q_all[:, hh] @ k_all[:, hh].T / np.sqrt(dh)
        s = np.where(np.tril(np.ones((T, T), dtype=bool)), s, -np.inf)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        out[:, hh] = p @ v_all[:, hh]
    return out


@pytest.mark.parametrize("dt", ["f32", "f16"])
def test_chain_tree_equals_causal_attention(dt):
    n, h, dh, L, Lmax = 6, 3, 16, 9, 20
    q, kn, vn, kc, vc = _rand_attn_inputs(n, h, dh, L, Lmax, 51, dt)
    vis, _, _ = oracle.tree_build(wl.chain_tree(n), L)
    out = oracle.tree_attention(q, kn, vn, kc, vc, L, vis)
    k_all = np.concatenate([kc[:, :L].astype(np.float64).transpose(1, 0, 2), kn])
    v_all = np.concatenate([vc[:, :L].astype(np.float64).transpose(1, 0, 2), vn])
    q_all = np.concatenate([np.zeros((L, h, dh)), q])
    ref = _causal_attention_numpy(q_all, k_all, v_all)[L:]
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-14)


def test_attention_sibling_permutation_permutes_outputs():
    """Renumbering the nodes (here: the two subtrees below the root swap places, and they differ in
    shape: one is a chain of three, the other a single leaf with a two-leaf fan below the root's other
    child) permutes the rows of the result and changes nothing else."""
    n, h, dh, L, Lmax = 7, 2, 8, 4, 16
    q, kn, vn, kc, vc = _rand_attn_inputs(n, h, dh, L, Lmax, 61)
    parent = [-1, 0, 0, 1, 3, 2, 2]                       # subtree A: 1 -> 3 -> 4 (a chain); subtree B: 2 -> {5, 6}
    # new numbering: B first.  new index -> old index
    old_of_new = [0, 2, 1, 5, 6, 3, 4]
    new_of_old = {o: i for i, o in enumerate(old_of_new)}
    parent_p = [-1 if parent[o] < 0 else new_of_old[parent[o]] for o in old_of_new]
    assert parent_p == [-1, 0, 0, 1, 1, 2, 5] and parent_p != parent
    vis, _, _ = oracle.tree_build(parent, L)
    a = oracle.tree_attention(q, kn, vn, kc, vc, L, vis)
    visp, _, _ = oracle.tree_build(parent_p, L)
    assert not np.array_equal(visp, vis)
    b = oracle.tree_attention(q[old_of_new], kn[old_of_new], vn[old_of_new], kc, vc, L, visp)
    assert np.allclose(b, a[old_of_new], rtol=1e-13)
    # and the rows really differ between nodes (the check above is not vacuous)
    assert np.abs(a[3] - a[5]).max() > 1e-3


# ---------------------------------------------------------------- layer
SMALL = wl.scaled(wl.TINY, name="small", d_model=32, n_heads=4, d_head=8, d_ffn=24, vocab=50, n_layers=2)


def _small_layer(config_id=7, layer=0, gains=True, shape=SMALL):
    return wl.layer_weights(shape, config_id, layer, random_gains=gains)


def test_layer_zero_weights_is_identity():
    w = _small_layer()
    for k in ("wqkv", "wo", "w_gate_up", "w_down"):
        w[k] = np.zeros_like(w[k])
    kc, vc = wl.kv_cache(SMALL, 7, 0, 5, 16)
    x = wl.layer_input(SMALL, 7, 4).astype(np.float64)
    vis, _, pos = oracle.tree_build(wl.chain_tree(4), 5)
    assert np.array_equal(oracle.layer(SMALL, w, kc, vc, 5, vis, pos, x), x)


def test_layer_swiglu_and_residual_closed_form():
    # d=4, one head of 4, f=2.  wo = 0 removes attention, so y = x and
    # z = x + W_down (SiLU(g) * u) with g, u the gate/up pre-activations.
    sh = wl.scaled(wl.TINY, name="cf", d_model=4, n_heads=1, d_head=4, d_ffn=2, rms_eps=0.0)
    c = 2.0
    x = np.full((1, 4), c)
    gate = np.array([[0.25] * 4, [-0.5] * 4], dtype=np.float32)      # pre-act  1.0, -2.0
    up = np.array([[0.5] * 4, [0.125] * 4], dtype=np.float32)        # pre-act  2.0,  0.5
    w = {"wqkv": np.zeros((12, 4), np.float32), "wo": np.zeros((4, 4), np.float32),
         "w_gate_up": np.concatenate([gate, up]), "rms1": np.ones(4, np.float32), "rms2": np.ones(4, np.float32),
         "w_down": np.array([[1, 0], [0, 1], [1, 1], [0, 0]], dtype=np.float32)}
    kc = np.zeros((1, 4, 4), np.float32)
    vis, _, pos = oracle.tree_build([-1], 0)
    z = oracle.layer(sh, w, kc, kc.copy(), 0, vis, pos, x)
    silu = lambda a: a / (1 + np.exp(-a))
    u0, u1 = silu(1.0) * 2.0, silu(-2.0) * 0.5
    assert np.allclose(z[0], [c + u0, c + u1, c + u0 + u1, c], rtol=1e-14)


def test_layer_appends_rotated_keys_and_values():
    w = _small_layer()
    L, n, Lmax = 3, 4, 12
    kc, vc = wl.kv_cache(SMALL, 7, 0, L, Lmax)
    k0, v0 = kc.copy(), vc.copy()
    x = wl.layer_input(SMALL, 7, n).astype(np.float64)
    parent = [-1, 0, 0, 2]
    vis, _, pos = oracle.tree_build(parent, L)
    oracle.layer(SMALL, w, kc, vc, L, vis, pos, x)
    assert np.array_equal(kc[:, :L], k0[:, :L]) and np.array_equal(vc[:, :L], v0[:, :L])
    assert not kc[:, L + n:].any() and not vc[:, L + n:].any()
    h = oracle.rmsnorm(x, w["rms1"], SMALL.rms_eps)
    qkv = oracle.linear(h, w["wqkv"])
    d = SMALL.d_model
    k_new = oracle.rope(qkv[:, d:2 * d].reshape(n, 4, 8), pos, SMALL.rope_theta)
    v_new = qkv[:, 2 * d:].reshape(n, 4, 8)
    assert np.allclose(kc[:, L:L + n].transpose(1, 0, 2), k_new, rtol=1e-6)
    assert np.allclose(vc[:, L:L + n].transpose(1, 0, 2), v_new, rtol=1e-6)


def _layer_from_pieces_numpy(sh, w, kc, vc, L, vis, pos, x):
    """One decoder layer written out with numpy only (paper Sec. II-B: attention block, then MLP block, each
    with a residual connection; Eq. (1) per head): its own RMSNorm formula, `@` for the projections, an explicit
    cos/sin rotation of q AND k at position pos, a masked softmax over cache + visible new rows, SwiGLU.
    -> (layer output [n][d], concatenated attention output [n][d])."""
    d, H, dh, f = sh.d_model, sh.n_heads, sh.d_head, sh.d_ffn
    n = x.shape[0]
    W = {k: np.asarray(v, dtype=np.float64) for k, v in w.items()}

    def rms(a, g):
        return a * g[None, :] / np.sqrt((a * a).mean(axis=1, keepdims=True) + sh.rms_eps)

    def rotate(u):                                         # u [n][H][dh], pairs (t, t + dh/2)
        half = dh // 2
        ang = np.asarray(pos, dtype=np.float64)[:, None] * sh.rope_theta ** (-2.0 * np.arange(half) / dh)[None, :]
        c, s_ = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        a, b = u[..., :half], u[..., half:]
        return np.concatenate([a * c - b * s_, b * c + a * s_], axis=-1)

    h1 = rms(x, W["rms1"])
    q = (h1 @ W["wqkv"][:d].T).reshape(n, H, dh)
    k = (h1 @ W["wqkv"][d:2 * d].T).reshape(n, H, dh)
    v = (h1 @ W["wqkv"][2 * d:].T).reshape(n, H, dh)
    q, k = rotate(q), rotate(k)
    allowed = np.concatenate([np.ones((n, L), dtype=bool), np.asarray(vis, dtype=bool)], axis=1)
    att = np.zeros((n, H, dh))
    for hh in range(H):
        k_all = np.concatenate([np.asarray(kc[hh, :L], dtype=np.float64), k[:, hh]])
        v_all = np.concatenate([np.asarray(vc[hh, :L], dtype=np.float64), v[:, hh]])
        s = np.where(allowed, q[:, hh] @ k_all.T / np.sqrt(dh), -np.inf)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        att[:, hh] = (p / p.sum(axis=1, keepdims=True)) @ v_all
    att = att.reshape(n, d)
    y1 = x + att @ W["wo"].T
    h2 = rms(y1, W["rms2"])
    g, up = h2 @ W["w_gate_up"][:f].T, h2 @ W["w_gate_up"][f:].T
    return y1 + (g / (1.0 + np.exp(-g)) * up) @ W["w_down"].T, att


@pytest.mark.parametrize("dt,seed", [("f32", 0), ("f16", 1), ("f32", 2)])
def test_layer_equals_its_pieces_written_in_numpy(dt, seed):
    """Pins the composition of the layer: rms1 for the attention block and rms2 (different gains) for the MLP
    block, rotated queries as well as keys, a non-zero output projection, both residuals added once."""
    sh = wl.scaled(SMALL, name="pieces", dtype=dt)
    L, n, Lmax = 7, 11, 24
    w = _small_layer(30 + seed, 0, gains=True, shape=sh)
    # gains far from one and different for the two norms; weights large enough that every term matters
    w["rms1"] = wl.normal((sh.d_model,), 900 + seed, 0.4, 1.5, dtype=dt)
    w["rms2"] = wl.normal((sh.d_model,), 910 + seed, 0.4, 0.6, dtype=dt)
    for key in ("wqkv", "wo", "w_gate_up", "w_down"):
        w[key] = wl.normal(w[key].shape, 920 + seed + len(key), 0.35, dtype=dt)
    assert np.abs(w["rms1"].astype(np.float64) - w["rms2"].astype(np.float64)).min() > 1e-3
    kc, vc = wl.kv_cache(sh, 30 + seed, 0, L, Lmax)
    k0, v0 = kc.copy(), vc.copy()
    x = wl.layer_input(sh, 30 + seed, n).astype(np.float64)
    parent = wl.random_tree(n, 4, 500 + seed, max_children=3)
    vis, _, pos = oracle.tree_build(parent, L)
    want, want_att = _layer_from_pieces_numpy(sh, w, k0, v0, L, vis, pos, x)
    got, got_att = oracle.layer(sh, w, kc, vc, L, vis, pos, x, want_attn=True)
    assert np.allclose(got_att, want_att, rtol=1e-10, atol=1e-12)
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)
    # every block contributes visibly (so that a dropped or doubled term cannot hide below the tolerance)
    assert np.abs(want_att).max() > 1e-2 and np.abs(want - x).max() > 1e-2


def test_layer_pieces_with_a_mask_that_is_not_a_tree():
    """The oracle takes any visibility matrix: a row may see node j without j's ancestors."""
    sh, L, n, Lmax = SMALL, 5, 9, 20
    w = _small_layer(33, 0)
    rng = np.random.default_rng(12)
    vis = np.tril(rng.random((n, n)) < 0.4)
    np.fill_diagonal(vis, True)
    pos = (L + vis.sum(axis=1) - 1).astype(np.int32)
    kc, vc = wl.kv_cache(sh, 33, 0, L, Lmax)
    x = wl.layer_input(sh, 33, n).astype(np.float64)
    want, want_att = _layer_from_pieces_numpy(sh, w, kc.copy(), vc.copy(), L, vis, pos, x)
    got, got_att = oracle.layer(sh, w, kc, vc, L, vis.astype(np.uint8), pos, x, want_attn=True)
    assert np.allclose(got_att, want_att, rtol=1e-10, atol=1e-12) and np.allclose(got, want, rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("seed", [0, 1])
def test_every_node_equals_causal_forward_over_its_root_path(seed):
    """Row i of the tree forward = last row of a chain forward over root..i (two layers deep)."""
    L, n, Lmax = 6, 9, 24
    parent = wl.random_tree(n, 4, 100 + seed)
    vis, _, pos = oracle.tree_build(parent, L)
    ws = [_small_layer(8, l) for l in range(2)]
    x = wl.layer_input(SMALL, 8 + seed, n).astype(np.float64)

    def run(x_in, vis_in, pos_in):
        cur = x_in
        for l in range(2):
            kc, vc = wl.kv_cache(SMALL, 8, l, L, Lmax)
            cur = oracle.layer(SMALL, ws[l], kc, vc, L, vis_in, pos_in, cur)
        return cur

    full = run(x, vis, pos)
    for i in range(n):
        path = sorted(_ancestors_by_sets(parent)[i])
        cvis, _, cpos = oracle.tree_build(wl.chain_tree(len(path)), L)
        sub = run(x[path], cvis, cpos)
        assert np.allclose(sub[-1], full[i], rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- step, argmax, accept
def test_argmax_first_index_on_ties():
    lg = np.array([[0.0, 3.0, 3.0, 1.0], [5.0, 5.0, 5.0, 5.0], [-1.0, -2.0, -0.5, -0.5]])
    assert list(oracle.argmax(lg)) == [1, 0, 2]


def _greedy_walk(parent, tokens, amax):
    """Independent top-down formulation: explore every matching child, keep the deepest path."""
    kids = {}
    for c, p in enumerate(parent):
        kids.setdefault(p, []).append(c)
    best = [0]

    def go(path):
        nonlocal best
        if len(path) > len(best) or (len(path) == len(best) and path[-1] < best[-1]):
            best = list(path)
        for c in kids.get(path[-1], []):
            if tokens[c] == amax[path[-1]]:
                go(path + [c])

    go([0])
    return best


def _all_trees(n):
    for rest in itertools.product(*[range(i) for i in range(1, n)]):
        yield [-1] + list(rest)


def test_accept_exhaustive_small_trees_binary_alphabet():
    for n in range(1, 6):
        for parent in _all_trees(n):
            for bits in itertools.product((0, 1), repeat=2 * n):
                tokens, amax = list(bits[:n]), list(bits[n:])
                m, nodes, toks = oracle.accept(parent, tokens, amax)
                best = _greedy_walk(parent, tokens, amax)
                assert m == len(best) - 1
                assert list(nodes) == best
                assert list(toks) == [amax[c] for c in best]


def test_accept_planted_path_and_width1_boundary():
    parent = wl.medusa_tree(64)
    tokens = wl.draft_tokens(parent, 32000, 5)
    rng = wl.Rng(9)
    amax = np.array([rng.below(32000) for _ in parent], dtype=np.int32)
    path = [0]
    for _ in range(3):                                     # follow first children three levels down
        path.append(parent.index(path[-1]))
    for a, b in zip(path[:-1], path[1:]):
        amax[a] = tokens[b]
    kids_last = [c for c, p in enumerate(parent) if p == path[-1]]
    amax[path[-1]] = max(tokens[c] for c in kids_last) + 1 if kids_last else 3
    m, nodes, toks = oracle.accept(parent, tokens, amax)
    assert m == 3 and list(nodes) == path and list(toks) == [amax[c] for c in path]
    (width, length), = _rows("table1_width1.txt")
    m, nodes, toks = oracle.accept([-1], [7], [9])
    assert int(width) == 1 and m + 1 == int(length) and list(toks) == [9]


def test_width1_tree_of_depth_k_reproduces_sequential_greedy_decoding():
    sh = SMALL
    k, L, Lmax = 4, 5, 16
    head = wl.head_weights(sh, 9)
    layers = [_small_layer(9, l) for l in range(sh.n_layers)]
    fresh = lambda: [wl.kv_cache(sh, 9, l, L, Lmax) for l in range(sh.n_layers)]
    # sequential: k + 1 single-token steps, each appending its K/V and feeding its argmax on
    caches = fresh()
    tok, seq = 17, []
    for s in range(k + 1):
        vis, _, pos = oracle.tree_build([-1], L + s)
        _, am = oracle.step(sh, head, layers, caches, L + s, vis, pos, [tok])
        seq.append(int(am[0]))
        tok = seq[-1]
    # one chain-shaped verify step over the root and the k tokens sequential decoding produced
    parent = wl.chain_tree(k + 1)
    vis, _, pos = oracle.tree_build(parent, L)
    tokens = [17] + seq[:k]
    logits, am = oracle.step(sh, head, layers, fresh(), L, vis, pos, tokens)
    assert list(am) == seq
    m, nodes, toks = oracle.accept(parent, tokens, am)
    assert m == k and list(toks) == seq
    # a wrong draft at depth 2 cuts acceptance there and the bonus token is the true one
    bad = list(tokens)
    bad[2] = (bad[2] + 1) % sh.vocab
    _, am2 = oracle.step(sh, head, layers, fresh(), L, vis, pos, bad)
    m2, _, toks2 = oracle.accept(parent, bad, am2)
    assert m2 == 1 and list(toks2) == seq[:2]


def test_step_is_embedding_layers_final_norm_lm_head():
    sh = SMALL
    L, Lmax = 3, 12
    head = wl.head_weights(sh, 10)
    head["rms_final"] = wl.normal((sh.d_model,), 77, 0.1, 1.0)
    layers = [_small_layer(10, l) for l in range(sh.n_layers)]
    parent = [-1, 0, 0, 1]
    tokens = [3, 9, 4, 0]
    vis, _, pos = oracle.tree_build(parent, L)
    # no layers: hidden is the embedding rows of the tokens
    caches = [wl.kv_cache(sh, 10, l, L, Lmax) for l in range(sh.n_layers)]
    _, _, hid0 = oracle.step(sh, head, [], caches[:1], L, vis, pos, tokens, want_hidden=True)
    assert np.array_equal(hid0, head["embed"][tokens].astype(np.float64))
    # with layers: hidden = layer(layer(embed)), logits = lm_head(final norm(hidden))
    logits, am, hid = oracle.step(sh, head, layers, caches, L, vis, pos, tokens, want_hidden=True)
    cur = hid0
    for l in range(sh.n_layers):
        kc, vc = wl.kv_cache(sh, 10, l, L, Lmax)
        cur = oracle.layer(sh, layers[l], kc, vc, L, vis, pos, cur)
    assert np.array_equal(cur, hid)
    ref = (oracle.rmsnorm(hid, head["rms_final"], sh.rms_eps)) @ head["lm_head"].astype(np.float64).T
    assert np.allclose(logits, ref, rtol=1e-12, atol=1e-14)
    assert list(am) == list(np.argmax(logits, axis=1))


# ---------------------------------------------------------------- KV commit and multi-step decoding
def _greedy(sh, head, layers, caches, L, first_tok, count):
    """Plain sequential decoding: `count` single-token steps, each feeding the previous argmax.
    -> tokens [first_tok, g1, ..., g_count]; caches are appended to in place."""
    seq = [int(first_tok)]
    for s in range(count):
        vis, _, pos = oracle.tree_build([-1], L + s)
        _, am = oracle.step(sh, head, layers, caches, L + s, vis, pos, [seq[-1]])
        seq.append(int(am[0]))
    return seq


def _plant(parent, tokens, chain_tokens, vocab):
    """Writes chain_tokens along the first-child chain below the root; other nodes keep their
    random ids, moved off the planted id where a sibling would collide."""
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


def test_kv_commit_leaves_the_cache_of_sequential_decoding():
    sh = SMALL
    L, Lmax = 6, 40
    head = wl.head_weights(sh, 21)
    layers = [_small_layer(21, l) for l in range(sh.n_layers)]
    fresh = lambda: [wl.kv_cache(sh, 21, l, L, Lmax) for l in range(sh.n_layers)]
    seq_caches = fresh()
    g = _greedy(sh, head, layers, seq_caches, L, 11, 4)          # rows L .. L+3 now hold tokens g[0..3]
    parent = [-1, 0, 0, 0, 1, 1, 2, 4, 4, 7, 7, 5, 9, 3]         # first-child chain 0 -> 1 -> 4 -> 7 -> 9 -> 12
    tokens = _plant(parent, wl.draft_tokens(parent, sh.vocab, 78), g[1:4], sh.vocab)
    tokens[0] = g[0]
    caches = fresh()
    vis, _, pos = oracle.tree_build(parent, L)
    _, am = oracle.step(sh, head, layers, caches, L, vis, pos, tokens)
    m, nodes, toks = oracle.accept(parent, tokens, am)
    assert m >= 3 and list(toks[:4]) == g[1:5]
    assert all(nodes[j] >= j for j in range(m + 1)) and any(nodes[j] != j for j in range(m + 1))   # rows really move
    oracle.kv_commit(caches, L, nodes)
    keep = min(m + 1, 4)
    for (k, v), (sk, sv) in zip(caches, seq_caches):
        assert np.array_equal(k[:, :L], sk[:, :L])
        assert np.allclose(k[:, L:L + keep].astype(np.float64), sk[:, L:L + keep].astype(np.float64), rtol=1e-6, atol=1e-7)
        assert np.allclose(v[:, L:L + keep].astype(np.float64), sv[:, L:L + keep].astype(np.float64), rtol=1e-6, atol=1e-7)


def test_kv_commit_is_a_gather_of_rows():
    rng = np.random.default_rng(5)
    k = rng.standard_normal((3, 20, 4)).astype(np.float32)
    v = rng.standard_normal((3, 20, 4)).astype(np.float32)
    k0, v0 = k.copy(), v.copy()
    oracle.kv_commit([(k, v)], 5, [0, 2, 3, 9])
    for j, node in enumerate([0, 2, 3, 9]):
        assert np.array_equal(k[:, 5 + j], k0[:, 5 + node]) and np.array_equal(v[:, 5 + j], v0[:, 5 + node])
    assert np.array_equal(k[:, :5], k0[:, :5]) and np.array_equal(k[:, 9:], k0[:, 9:])


def test_speculative_steps_emit_exactly_the_greedy_sequence():
    """Tree verification is lossless: whatever is drafted, verify + accept + commit, step after step,
    produces the tokens of plain greedy decoding (paper Sec. II-C: the verified prefix plus the
    model's own next token)."""
    sh = SMALL
    L0, Lmax, total = 4, 64, 18
    head = wl.head_weights(sh, 22)
    layers = [_small_layer(22, l) for l in range(sh.n_layers)]
    fresh = lambda: [wl.kv_cache(sh, 22, l, L0, Lmax) for l in range(sh.n_layers)]
    g = _greedy(sh, head, layers, fresh(), L0, 7, total + 8)
    caches = fresh()
    L, root, out, step_no = L0, g[0], [], 0
    while len(out) < total:
        parent = wl.random_tree(10, 4, 300 + step_no, max_children=3)
        tokens = wl.draft_tokens(parent, sh.vocab, 400 + step_no)
        at = len(out)                                         # root token is g[at]
        tokens = _plant(parent, tokens, g[at + 1:at + 1 + step_no % 4], sh.vocab)   # 0..3 correct drafts
        tokens[0] = root
        vis, _, pos = oracle.tree_build(parent, L)
        _, am = oracle.step(sh, head, layers, caches, L, vis, pos, tokens)
        m, nodes, toks = oracle.accept(parent, tokens, am)
        chain, node = 0, 0                                    # length of the first-child chain the drafts were planted on
        while node in parent:
            node = parent.index(node)
            chain += 1
        assert m >= min(step_no % 4, chain)                   # every planted draft is accepted
        oracle.kv_commit(caches, L, nodes)
        out += [int(t) for t in toks]
        L += m + 1
        root = int(toks[-1])
        step_no += 1
    assert out == g[1:len(out) + 1]
    assert step_no < total                                    # some drafts were accepted: fewer steps than tokens


# ---------------------------------------------------------------- drafting heads
def test_medusa_head_closed_forms():
    h = np.array([1.0, -2.0, 0.5])
    eye = np.eye(3)
    # W1 = I: y = h + h * sigmoid(h), written out; W2 = I: the logits are y itself
    sig = 1.0 / (1.0 + np.exp(-h))
    cands, logits = oracle.medusa_draft(h, [eye], [eye], [3])
    assert np.allclose(logits[0], h + h * sig, rtol=1e-15)
    assert np.allclose(logits[0], [1.7310585786300048, -2.2384058440442351, 0.8112296656009273], rtol=1e-14)   # 1 + s(1), -2 - 2 s(-2), .5 + .5 s(.5)
    assert cands[0] == [0, 2, 1]
    # W1 = 0: SiLU(0) = 0, the head is a plain projection of h (library matmul + stable sort as the check)
    rng = np.random.default_rng(3)
    h = rng.standard_normal(16)
    w2 = rng.standard_normal((2, 40, 16)).astype(np.float32)
    cands, logits = oracle.medusa_draft(h, np.zeros((2, 16, 16), np.float32), w2, [5, 2])
    for k, t in enumerate([5, 2]):
        z = w2[k].astype(np.float64) @ h
        assert np.allclose(logits[k], z, rtol=1e-13)
        assert cands[k] == list(np.argsort(-z, kind="stable")[:t])


def test_medusa_topk_ties_go_to_the_lower_id():
    h = np.array([1.0, 0.0])
    w2 = np.array([[[0.5, 0], [2.0, 0], [2.0, 0], [0.5, 0], [3.0, 0]]])
    cands, _ = oracle.medusa_draft(h, np.zeros((1, 2, 2)), w2, [5])
    assert cands[0] == [4, 1, 2, 0, 3]


def test_tree_fill_tokens_example():
    cands = [[11, 12, 13], [21, 22], [31]]
    #        root  L1 r0 L1 r1 L1 r2 L2 r0 (child of node 1) L2 r1  L3 r0
    level = [0, 1, 1, 1, 2, 2, 3]
    rank = [0, 0, 1, 2, 0, 1, 0]
    assert list(oracle.tree_fill_tokens(cands, 99, level, rank)) == [99, 11, 12, 13, 21, 22, 31]
