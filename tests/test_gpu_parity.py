"""GPU parity: every call goes through the C-ABI and is compared with the CPU
oracle on the same seeded inputs.  Integer results bit-exact; floating point
within max|got-want|/max|want| <= 1e-4 (float mode) or 2e-2 (half mode)."""
import itertools

import numpy as np
import pytest

import oracle
import workloads as wl
from util import (argmax_margin_ok, gpu_cfg, gpu_layer_weights, max_rel_err, to_dev, tol_for, unpack_mask)

pytestmark = pytest.mark.gpu

SMALL32 = wl.scaled(wl.TINY, name="small32", d_model=256, n_heads=4, d_head=64, d_ffn=352, vocab=777, n_layers=2)
SMALL16 = wl.scaled(SMALL32, name="small16", dtype="f16")
SMALL16_DH128 = wl.scaled(SMALL16, name="small16b", d_model=512, n_heads=4, d_head=128, d_ffn=704)


@pytest.fixture(scope="module")
def ghd():
    import paper_2505_23219_b200 as g
    return g


def make_ctx(ghd, shape, max_kv_len, max_nodes, n_layers=None):
    return ghd.ghd_create(gpu_cfg(shape, max_kv_len, max_nodes, n_layers))


# ---------------------------------------------------------------- tree build (bit-exact)
TREES = [("chain1", wl.chain_tree(1)), ("chain9", wl.chain_tree(9)), ("star33", wl.star_tree(33)),
         ("medusa64", wl.medusa_tree(64)), ("rand8", wl.random_tree(8, 4, 1)), ("rand63", wl.random_tree(63, 8, 2)),
         ("rand65", wl.random_tree(65, 8, 3)), ("rand129", wl.random_tree(129, 8, 4)),
         ("rand256", wl.random_tree(256, 8, 5, max_children=6)), ("chain256", wl.chain_tree(256))]


@pytest.mark.parametrize("name,parent", TREES, ids=[t[0] for t in TREES])
def test_tree_build_bit_exact(ghd, name, parent):
    ctx = make_ctx(ghd, SMALL32, 1024, 256)
    kv_len = 300
    tree = ghd.ghd_tree_build(ctx, parent, kv_len)
    ghd.ghd_sync_status(ctx)
    n = len(parent)
    vis, depth, pos = oracle.tree_build(parent, kv_len)
    assert tree.c.n == n and tree.c.n_words == (n + 63) // 64
    assert np.array_equal(unpack_mask(tree.mask_words(), n), vis)
    assert np.array_equal(tree.depth[:n].cpu().numpy(), depth)
    assert np.array_equal(tree.pos[:n].cpu().numpy(), pos)
    assert np.array_equal(tree.parent[:n].cpu().numpy(), np.asarray(parent, dtype=np.int32))
    # the same visibility as a coordinate index (sparse part by list, Sec. III-B-3)
    want_ptr, want_cols = oracle.coo_index(vis)
    got_ptr, got_cols = tree.coo()
    assert tree.c.nnz == want_ptr[-1] and np.array_equal(got_ptr, want_ptr) and np.array_equal(got_cols, want_cols)
    # rotary table: cos/sin of pos * theta^(-2t/dh), checked through the oracle's rotation of unit vectors
    dh = SMALL32.d_head
    unit = np.zeros((n, 1, dh))
    unit[:, 0, : dh // 2] = 1.0
    rot = oracle.rope(unit, pos, SMALL32.rope_theta)[:, 0]
    table = tree.rope[: n * dh].cpu().numpy().reshape(n, dh // 2, 2)
    assert np.abs(table[:, :, 0] - rot[:, : dh // 2]).max() < 1e-6
    assert np.abs(table[:, :, 1] - rot[:, dh // 2:]).max() < 1e-6


def test_tree_from_explicit_lookahead_mask_equals_tree_build(ghd):
    ctx = make_ctx(ghd, SMALL32, 1024, 64)
    vis, depth, parent = wl.lookahead_pattern(7, 5, 5)
    a = ghd.ghd_tree_from_mask(ctx, ghd.pack_mask(vis), 100, parent=parent)
    b = ghd.ghd_tree_build(ctx, parent, 100)
    c = ghd.ghd_tree_from_mask(ctx, ghd.pack_mask(vis), 100, depth=depth)
    ghd.ghd_sync_status(ctx)
    n = len(parent)
    assert np.array_equal(a.mask_words(), b.mask_words())
    for t in (a, c):
        assert all(np.array_equal(x, y) for x, y in zip(t.coo(), b.coo())) and t.c.nnz == b.c.nnz
        assert all(np.array_equal(x, y) for x, y in zip(t.coo(), oracle.coo_index(vis)))
        assert np.array_equal(t.depth[:n].cpu().numpy(), b.depth[:n].cpu().numpy())
        assert np.array_equal(t.pos[:n].cpu().numpy(), b.pos[:n].cpu().numpy())
        assert np.array_equal(t.rope.cpu().numpy(), b.rope.cpu().numpy())
    assert np.array_equal(unpack_mask(a.mask_words(), n), vis.astype(np.uint8))


def test_argument_errors_launch_nothing(ghd):
    ctx = make_ctx(ghd, SMALL32, 128, 16)
    before = ghd.ghd_launch_count(ctx)
    cases = [([0, 0], 0, "GHD_ETREE"), ([-1, 1], 0, "GHD_ETREE"), ([-1, -1], 0, "GHD_ETREE"),
             ([-1] + [0] * 16, 0, "GHD_ETREE"), ([], 0, "GHD_ETREE"), ([-1, 0], 127, "GHD_ENOSPACE"),
             ([-1, 0], -2, "GHD_EINVAL")]      # -1 would be GHD_KV_LEN_DEVICE
    for parent, kv_len, want in cases:
        with pytest.raises(ghd.GhdError) as e:
            ghd.ghd_tree_build(ctx, parent, kv_len)
        assert e.value.name == want
    bad = ghd.pack_mask(np.array([[1, 0], [1, 0]], dtype=bool))          # row 1 lacks its own bit
    with pytest.raises(ghd.GhdError) as e:
        ghd.ghd_tree_from_mask(ctx, bad, 0)
    assert e.value.name == "GHD_ETREE"
    up = ghd.pack_mask(np.array([[1, 1], [1, 1]], dtype=bool))           # bit above the diagonal
    with pytest.raises(ghd.GhdError):
        ghd.ghd_tree_from_mask(ctx, up, 0)
    assert ghd.ghd_launch_count(ctx) == before
    with pytest.raises(ghd.GhdError) as e:                               # unsupported shapes
        ghd.ghd_create(gpu_cfg(wl.scaled(SMALL32, d_head=32, n_heads=8), 128, 16))
    assert e.value.name == "GHD_ESHAPE"
    with pytest.raises(ghd.GhdError) as e:
        ghd.ghd_create(gpu_cfg(SMALL32, 128, 257))
    assert e.value.name == "GHD_EINVAL"
    # a tree that was never built is refused by the compute calls
    tree = ghd.Tree(ctx)
    with pytest.raises(ghd.GhdError):
        ghd.ghd_accept(ctx, tree, to_dev(np.zeros(4, np.int32)), to_dev(np.zeros(4, np.int32)))
    ghd.ghd_sync_status(ctx)


# ---------------------------------------------------------------- building blocks
@pytest.mark.parametrize("shape", [SMALL32, SMALL16], ids=["f32", "f16"])
@pytest.mark.parametrize("n", [1, 5, 8, 37])
def test_rmsnorm(ghd, shape, n):
    ctx = make_ctx(ghd, shape, 128, 64)
    x = wl.normal((n, shape.d_model), 301, 3.0)
    g = wl.normal((shape.d_model,), 302, 0.1, 1.0, dtype=shape.dtype)
    out = ghd.ghd_rmsnorm(ctx, to_dev(x), to_dev(g))
    ghd.ghd_sync_status(ctx)
    want = oracle.rmsnorm(x, g, shape.rms_eps)
    assert max_rel_err(out.cpu().numpy(), want) <= (1e-6 if shape.dtype == "f32" else 1e-3)


@pytest.mark.parametrize("shape", [SMALL32, SMALL16], ids=["f32", "f16"])
@pytest.mark.parametrize("n,k,m", [(1, 256, 40), (7, 352, 256), (8, 256, 1001), (19, 1376, 130), (64, 512, 96)])
def test_linear_cuda_core_path(ghd, shape, n, k, m):
    ctx = make_ctx(ghd, shape, 128, 64)
    ghd.ghd_set_option(ctx, ghd.OPT_GEMM_PATH, 1)
    x = wl.normal((n, k), 311, 1.0, dtype=shape.dtype)
    w = wl.normal((m, k), 312, 0.02, dtype=shape.dtype)
    y = ghd.ghd_linear(ctx, to_dev(x), to_dev(w))
    ghd.ghd_sync_status(ctx)
    assert max_rel_err(y.cpu().numpy(), oracle.linear(x, w)) <= 2e-6


@pytest.mark.parametrize("shape", [SMALL32, SMALL16, SMALL16_DH128], ids=["f32", "f16", "f16dh128"])
@pytest.mark.parametrize("n", [1, 19, 64, 130])
def test_gate_up_with_fused_swiglu(ghd, shape, n):
    """First half of the MLP block as the layer runs it: u = SiLU(h Wg^T) * (h Wu^T)."""
    ctx = make_ctx(ghd, shape, 128, 256)
    d, f, dt = shape.d_model, shape.d_ffn, shape.dtype
    h = wl.normal((n, d), 351, 1.0, dtype=dt)
    w = wl.normal((2 * f, d), 352, 0.05, dtype=dt)
    u = ghd.ghd_gate_up(ctx, to_dev(h), to_dev(w))
    ghd.ghd_sync_status(ctx)
    gu = oracle.linear(h, w)
    g, up = gu[:, :f], gu[:, f:]
    want = g / (1.0 + np.exp(-g)) * up
    assert max_rel_err(u.float().cpu().numpy(), want) <= (2e-6 if dt == "f32" else 2e-3)


TC_SHAPES = [(1, 64, 128), (5, 256, 40), (16, 512, 256), (17, 320, 130), (64, 4096, 1024), (64, 11008, 512),
             (100, 1024, 1001), (128, 512, 384), (200, 2048, 256), (256, 1024, 640)]


@pytest.mark.parametrize("n,k,m", TC_SHAPES)
def test_linear_tcgen05_path(ghd, n, k, m):
    ctx = make_ctx(ghd, SMALL16, 128, 256)
    ghd.ghd_set_option(ctx, ghd.OPT_GEMM_PATH, 2)
    x = wl.normal((n, k), 321, 1.0, dtype="f16")
    w = wl.normal((m, k), 322, 0.02, dtype="f16")
    xd, wd = to_dev(x), to_dev(w)
    y = ghd.ghd_linear(ctx, xd, wd)
    ghd.ghd_sync_status(ctx)
    want = oracle.linear(x, w)
    assert max_rel_err(y.cpu().numpy(), want) <= 2e-5        # exact products, float accumulation
    y2 = ghd.ghd_linear(ctx, xd, wd)
    ghd.ghd_sync_status(ctx)
    assert np.array_equal(y.cpu().numpy(), y2.cpu().numpy())  # fixed reduction order -> reproducible
    for ctas in (1, 7, 64):                                   # result must not depend on the work split
        ghd.ghd_set_option(ctx, ghd.OPT_GEMM_CTAS, ctas)
        y3 = ghd.ghd_linear(ctx, xd, wd)
        ghd.ghd_sync_status(ctx)
        assert max_rel_err(y3.cpu().numpy(), want) <= 2e-5


PAIR_SHAPES = [(17, 320, 130), (33, 512, 256), (64, 4096, 1024), (100, 1024, 1001), (128, 512, 768), (200, 2048, 256),
               (256, 1024, 512), (256, 4096, 2048)]


@pytest.mark.parametrize("n,k,m", PAIR_SHAPES)
def test_linear_tcgen05_on_cta_pairs(ghd, n, k, m):
    """Clusters of two CTAs (cta_group::2): each CTA loads its weight tile and half of the activation rows."""
    ctx = make_ctx(ghd, SMALL16, 128, 256)
    ghd.ghd_set_option(ctx, ghd.OPT_GEMM_PATH, 2)
    ghd.ghd_set_option(ctx, ghd.OPT_GEMM_PAIR, 2)
    x = wl.normal((n, k), 331, 1.0, dtype="f16")
    w = wl.normal((m, k), 332, 0.02, dtype="f16")
    xd, wd = to_dev(x), to_dev(w)
    y = ghd.ghd_linear(ctx, xd, wd)
    ghd.ghd_sync_status(ctx)
    assert ghd.ghd_path_count(ctx, ghd.PATH_GEMM_PAIR) == 1, "the paired kernel did not run"
    want = oracle.linear(x, w)
    assert max_rel_err(y.cpu().numpy(), want) <= 2e-5
    y2 = ghd.ghd_linear(ctx, xd, wd)
    ghd.ghd_sync_status(ctx)
    assert np.array_equal(y.cpu().numpy(), y2.cpu().numpy())  # fixed reduction order -> reproducible
    for ctas in (2, 6, 64):                                   # result must not depend on the work split
        ghd.ghd_set_option(ctx, ghd.OPT_GEMM_CTAS, ctas)
        y3 = ghd.ghd_linear(ctx, xd, wd)
        ghd.ghd_sync_status(ctx)
        assert max_rel_err(y3.cpu().numpy(), want) <= 2e-5


@pytest.mark.parametrize("n,L", [(13, 100), (64, 77), (100, 300), (128, 9), (200, 5), (256, 31)])
def test_small_layers_with_projections_on_cta_pairs(ghd, n, L):
    import paper_2505_23219_b200 as g
    ctx = _layer_case(ghd, SMALL16_DH128, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6), opts=[(g.OPT_GEMM_PAIR, 2)])
    assert ghd.ghd_path_count(ctx, ghd.PATH_GEMM_PAIR) >= (3 if n > 16 else 0)     # QKV, O, down (gate/up has 11 tiles)


def _attention_case(ghd, shape, n, L, parent, splits, seed=400, path=0, sparse=0, on_device=False, opts=()):
    Lmax = L + n + (150 if on_device else 3)               # on_device: the kernels see cache rows far past kv_len + n
    ctx = make_ctx(ghd, shape, Lmax, max(n, 8))
    if path:
        ghd.ghd_set_option(ctx, ghd.OPT_ATTN_PATH, path)
    ghd.ghd_set_option(ctx, ghd.OPT_ATTN_SPARSE, sparse)
    for o, v in opts:
        ghd.ghd_set_option(ctx, o, v)
    if splits:
        ghd.ghd_set_option(ctx, ghd.OPT_ATTN_SPLITS, splits)
    H, dh, dt = shape.n_heads, shape.d_head, shape.dtype
    q = wl.normal((n, H, dh), seed, dtype=dt)
    kc = wl.normal((H, Lmax, dh), seed + 1, dtype=dt)      # rows [L, L+n) play the appended new rows
    vc = wl.normal((H, Lmax, dh), seed + 2, dtype=dt)
    vis, _, _ = oracle.tree_build(parent, L)
    k_new = kc[:, L:L + n].transpose(1, 0, 2)
    v_new = vc[:, L:L + n].transpose(1, 0, 2)
    want = oracle.tree_attention(q, k_new, v_new, kc, vc, L, vis)
    if on_device:                                           # the length comes from the context's device word
        ghd.ghd_kv_len_set(ctx, L)
        L = ghd.KV_LEN_DEVICE
    tree = ghd.ghd_tree_build(ctx, parent, L)
    out = ghd.ghd_tree_attention(ctx, to_dev(q.reshape(n, H * dh)), ghd.KvLayer(to_dev(kc), to_dev(vc), L), tree)
    ghd.ghd_sync_status(ctx)
    if sparse:
        assert ghd.ghd_path_count(ctx, ghd.PATH_ATTN_COO) == 1, "the coordinate-index kernel did not run"
    return max_rel_err(out.cpu().numpy().reshape(n, H, dh), want)


ATTN_CASES = [(1, 0, 0), (1, 1, 1), (8, 256, 0), (9, 63, 1), (33, 65, 3), (64, 300, 0), (64, 300, 16), (130, 17, 2),
              (256, 129, 0)]


@pytest.mark.parametrize("shape", [SMALL32, SMALL16, SMALL16_DH128], ids=["f32", "f16", "f16dh128"])
@pytest.mark.parametrize("n,L,splits", ATTN_CASES)
def test_tree_attention(ghd, shape, n, L, splits):
    parent = wl.random_tree(n, 8, 1000 + n, max_children=6)
    err = _attention_case(ghd, shape, n, L, parent, splits)
    assert err <= (2e-5 if shape.dtype == "f32" else 2e-3)


@pytest.mark.parametrize("shape", [SMALL32, SMALL16, SMALL16_DH128], ids=["f32", "f16", "f16dh128"])
@pytest.mark.parametrize("n,L,splits", ATTN_CASES)
def test_tree_attention_sparse_part_from_the_coordinate_index(ghd, shape, n, L, splits):
    """Same problems, the new keys gathered per query from the coordinate index instead of bitmask-skipped groups."""
    parent = wl.random_tree(n, 8, 1000 + n, max_children=6)
    err = _attention_case(ghd, shape, n, L, parent, splits, sparse=1)
    assert err <= (2e-5 if shape.dtype == "f32" else 2e-3)
    if shape.dtype == "f16":
        assert _attention_case(ghd, shape, n, L, parent, splits, path=1, sparse=1) <= 2e-3      # cache part on CUDA cores


@pytest.mark.parametrize("shape", [SMALL32, SMALL16, SMALL16_DH128], ids=["f32", "f16", "f16dh128"])
@pytest.mark.parametrize("n,L,splits", ATTN_CASES + [(64, 2048, 0), (200, 1000, 7)])
def test_tree_attention_with_the_cache_length_on_the_device(ghd, shape, n, L, splits):
    """GHD_KV_LEN_DEVICE: the kernels read the length from the device word; the cache buffers are longer than
    kv_len + n and every row of them holds (finite) data that must not leak into the result."""
    parent = wl.random_tree(n, 8, 1000 + n, max_children=6)
    tol = 2e-5 if shape.dtype == "f32" else 2e-3
    assert _attention_case(ghd, shape, n, L, parent, splits, on_device=True) <= tol
    assert _attention_case(ghd, shape, n, L, parent, splits, sparse=1, on_device=True) <= tol
    if shape.dtype == "f16":
        assert _attention_case(ghd, shape, n, L, parent, splits, path=1, on_device=True) <= tol


@pytest.mark.parametrize("shape", [SMALL16, SMALL16_DH128], ids=["f16", "f16dh128"])
@pytest.mark.parametrize("n,L,splits", [(1, 0, 0), (1, 1, 1), (8, 256, 0), (9, 63, 1), (33, 65, 3), (64, 300, 0), (64, 300, 16), (64, 2048, 0),
                                        (49, 640, 5), (17, 129, 2), (64, 127, 0), (40, 4096, 0)])
def test_tree_attention_small_tree_kernel_with_128_key_units(ghd, shape, n, L, splits):
    """GHD_OPT_ATTN_SMALL: 128-key units, output accumulator resident in tensor memory (rescaled in place when the
    reference maximum rises); plain, with the coordinate index for the new rows, and with the cache length on the device."""
    parent = wl.random_tree(n, 8, 1000 + n, max_children=6)
    small = [(ghd.OPT_ATTN_SMALL, 1)]
    assert _attention_case(ghd, shape, n, L, parent, splits, opts=small) <= 2e-3
    assert _attention_case(ghd, shape, n, L, parent, splits, sparse=1, opts=small) <= 2e-3
    assert _attention_case(ghd, shape, n, L, parent, splits, on_device=True, opts=small) <= 2e-3
    assert _attention_case(ghd, wl.scaled(shape, name="chain"), n, L, wl.chain_tree(n), splits, opts=small) <= 2e-3


@pytest.mark.parametrize("shape", [SMALL16, SMALL16_DH128], ids=["f16", "f16dh128"])
@pytest.mark.parametrize("n,L,splits", [(65, 0, 0), (100, 300, 0), (128, 1000, 3), (130, 17, 2), (200, 1000, 0), (256, 129, 0), (256, 2048, 0),
                                        (256, 4096, 2), (129, 127, 1)])
def test_tree_attention_128_key_unit_kernel_on_wide_trees(ghd, shape, n, L, splits):
    """The same kernel on 128 distinct query rows per CTA with four groups of softmax warps (GHD_OPT_ATTN_SMALL = 1)."""
    parent = wl.random_tree(n, 8, 1000 + n, max_children=6)
    wide = [(ghd.OPT_ATTN_SMALL, 1)]
    assert _attention_case(ghd, shape, n, L, parent, splits, opts=wide) <= 2e-3
    assert _attention_case(ghd, shape, n, L, parent, splits, sparse=1, opts=wide) <= 2e-3
    assert _attention_case(ghd, shape, n, L, parent, splits, on_device=True, opts=wide) <= 2e-3
    assert _attention_case(ghd, shape, n, L, wl.star_tree(n), splits, opts=wide) <= 2e-3


@pytest.mark.parametrize("n,L", [(1, 40), (13, 100), (64, 77)])
def test_small_layers_with_the_small_tree_attention_kernel(ghd, n, L):
    import paper_2505_23219_b200 as g
    _layer_case(ghd, SMALL16_DH128, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6), opts=[(g.OPT_ATTN_SMALL, 1)])


@pytest.mark.parametrize("n,L,splits", [(64, 2048, 0), (64, 2048, 5), (200, 1000, 0), (256, 4096, 0), (49, 640, 3)])
def test_tree_attention_long_cache_both_paths(ghd, n, L, splits):
    parent = wl.random_tree(n, 8, 2000 + n, max_children=6)
    assert _attention_case(ghd, SMALL16_DH128, n, L, parent, splits) <= 2e-3               # tcgen05 kernel (automatic choice)
    assert _attention_case(ghd, SMALL16_DH128, n, L, parent, splits, opts=[(ghd.OPT_ATTN_SMALL, 2)]) <= 2e-3   # 64-key units
    assert _attention_case(ghd, SMALL16_DH128, n, L, parent, splits, path=1) <= 2e-3       # CUDA-core kernel


def _random_mask(n, seed, density=0.3):
    """Lower-triangular visibility with the diagonal set and NO closure under ancestry: row i may see
    node j without seeing what j sees, which no parent array can express."""
    rng = np.random.default_rng(seed)
    vis = np.tril(rng.random((n, n)) < density)
    np.fill_diagonal(vis, True)
    return vis


@pytest.mark.parametrize("shape", [SMALL16, SMALL16_DH128, SMALL32], ids=["f16", "f16dh128", "f32"])
@pytest.mark.parametrize("n,L", [(49, 200), (130, 77), (256, 300)])
def test_tree_attention_with_a_mask_that_is_not_a_tree(ghd, shape, n, L):
    vis = _random_mask(n, 7000 + n)
    assert any(vis[i, j] and not (vis[j] <= vis[i]).all() for i in range(n) for j in range(i))   # really not prefix-closed
    Lmax = L + n
    ctx = make_ctx(ghd, shape, Lmax, n)
    H, dh, dt = shape.n_heads, shape.d_head, shape.dtype
    q = wl.normal((n, H, dh), 7100, dtype=dt)
    kc = wl.normal((H, Lmax, dh), 7101, dtype=dt)
    vc = wl.normal((H, Lmax, dh), 7102, dtype=dt)
    want = oracle.tree_attention(q, kc[:, L:L + n].transpose(1, 0, 2), vc[:, L:L + n].transpose(1, 0, 2), kc, vc, L, vis.astype(np.uint8))
    tree = ghd.ghd_tree_from_mask(ctx, ghd.pack_mask(vis), L)
    assert np.array_equal(unpack_mask(tree.mask_words(), n), vis.astype(np.uint8))
    out = ghd.ghd_tree_attention(ctx, to_dev(q.reshape(n, H * dh)), ghd.KvLayer(to_dev(kc), to_dev(vc), L), tree)
    ghd.ghd_sync_status(ctx)
    assert max_rel_err(out.cpu().numpy().reshape(n, H, dh), want) <= (2e-5 if dt == "f32" else 2e-3)


def test_chain_tree_is_causal_attention_and_star_sees_only_root(ghd):
    for parent in (wl.chain_tree(40), wl.star_tree(40)):
        assert _attention_case(ghd, SMALL32, 40, 50, parent, 0) <= 2e-5
        assert _attention_case(ghd, SMALL16, 40, 50, parent, 0) <= 2e-3


def test_argmax_bit_exact_including_ties(ghd):
    ctx = make_ctx(ghd, SMALL32, 128, 64)
    v = 32000
    lg = wl.normal((9, v), 500).astype(np.float32)
    lg[1, 100] = lg[1, 31999] = 50.0            # tie -> first index
    lg[2, :] = 0.0                              # all equal -> 0
    lg[3, 31999] = 60.0                         # maximum in the last column
    lg[4, 0] = 60.0
    lg[5, 777] = lg[5, 778] = 55.0
    out = ghd.ghd_argmax(ctx, to_dev(lg))
    ghd.ghd_sync_status(ctx)
    assert np.array_equal(out.cpu().numpy(), oracle.argmax(lg))
    small = wl.normal((3, 5), 501).astype(np.float32)
    assert np.array_equal(ghd.ghd_argmax(ctx, to_dev(small)).cpu().numpy(), oracle.argmax(small))


def _accept_gpu(ghd, ctx, parent, tokens, amax):
    tree = ghd.ghd_tree_build(ctx, parent, 0)
    res = ghd.ghd_accept(ctx, tree, to_dev(np.asarray(tokens, np.int32)), to_dev(np.asarray(amax, np.int32)))
    r = res.cpu().numpy()
    m = int(r[0])
    return m, int(r[1]), r[2:2 + m + 1], r[2 + 256:2 + 256 + m + 1]


def test_accept_bit_exact(ghd):
    ctx = make_ctx(ghd, SMALL32, 1024, 256)
    cases = []
    for n in (1, 2, 3, 4):                                   # all small trees, binary alphabet (duplicates included)
        for rest in itertools.product(*[range(i) for i in range(1, n)]):
            for bits in itertools.product((0, 1), repeat=2 * n):
                cases.append(([-1] + list(rest), bits[:n], bits[n:]))
    rng = wl.Rng(77)
    for trial in range(40):                                  # bigger trees with planted partial matches
        n = [5, 17, 64, 65, 200, 256][trial % 6]
        parent = wl.random_tree(n, 8, 600 + trial, max_children=6)
        tokens = wl.draft_tokens(parent, 50, 700 + trial)
        amax = np.array([rng.below(50) for _ in range(n)], dtype=np.int32)
        for c in range(1, n):
            if rng.below(3):
                amax[parent[c]] = tokens[c]
        cases.append((parent, tokens, amax))
    for parent, tokens, amax in cases:
        m, emitted, nodes, toks = _accept_gpu(ghd, ctx, parent, tokens, amax)
        wm, wnodes, wtoks = oracle.accept(parent, tokens, amax)
        assert (m, emitted) == (wm, wm + 1)
        assert np.array_equal(nodes, wnodes) and np.array_equal(toks, wtoks)
    ghd.ghd_sync_status(ctx)


def test_device_wait_status_is_reported_once_and_the_context_stays_usable(ghd):
    """A kernel whose bounded wait runs out leaves a code in the status word at the start of the workspace and
    returns; here the word is set by hand (no kernel is made to wait): ghd_sync_status must report
    GHD_ETIMEOUT once, clear the word, and the context must work afterwards."""
    import torch
    ctx = make_ctx(ghd, SMALL16, 64, 8)
    x = wl.normal((4, 256), 1, 1.0, dtype="f16")
    w = wl.normal((128, 256), 2, 0.02, dtype="f16")
    y0 = ghd.ghd_linear(ctx, to_dev(x), to_dev(w))
    ghd.ghd_sync_status(ctx)
    ctx.workspace[:4].copy_(torch.tensor([2, 0, 0, 0], dtype=torch.uint8))      # int32 code 2 in the status word
    with pytest.raises(ghd.GhdError) as err:
        ghd.ghd_sync_status(ctx)
    assert "GHD_ETIMEOUT" in str(err.value)
    ghd.ghd_sync_status(ctx)                                                    # cleared
    y1 = ghd.ghd_linear(ctx, to_dev(x), to_dev(w))
    ghd.ghd_sync_status(ctx)
    assert np.array_equal(y0.cpu().numpy(), y1.cpu().numpy())


# ---------------------------------------------------------------- layer
def _layer_case(ghd, shape, config_id, n, L, parent, vis=None, depth=None, gains=True, opts=()):
    Lmax = L + n
    ctx = make_ctx(ghd, shape, Lmax, max(n, 1))
    for o, v in opts:
        ghd.ghd_set_option(ctx, o, v)
    w = wl.layer_weights(shape, config_id, 0, random_gains=gains)
    kc, vc = wl.kv_cache(shape, config_id, 0, L, Lmax)
    x = wl.layer_input(shape, config_id, n)
    if vis is None:
        ovis, _, opos = oracle.tree_build(parent, L)
        tree = ghd.ghd_tree_build(ctx, parent, L)
    else:
        odepth = depth if depth is not None else vis.sum(axis=1) - 1      # the library's default: visible nodes - 1
        ovis, opos = vis.astype(np.uint8), (L + odepth).astype(np.int32)
        tree = ghd.ghd_tree_from_mask(ctx, ghd.pack_mask(vis), L, depth=depth)
    okc, ovc = kc.copy(), vc.copy()
    want = oracle.layer(shape, w, okc, ovc, L, ovis, opos, x)
    kv = ghd.KvLayer(to_dev(kc), to_dev(vc), L)
    y = ghd.ghd_verify_layer(ctx, gpu_layer_weights(w), kv, tree, to_dev(x))
    ghd.ghd_sync_status(ctx)
    tol = tol_for(shape.dtype)
    assert max_rel_err(y.float().cpu().numpy(), want) <= tol
    gk, gv = kv.k.float().cpu().numpy(), kv.v.float().cpu().numpy()
    assert np.array_equal(gk[:, :L], kc[:, :L].astype(np.float32))       # old rows untouched
    assert max_rel_err(gk[:, L:], okc[:, L:]) <= tol and max_rel_err(gv[:, L:], ovc[:, L:]) <= tol
    return ctx


def test_config1_tiny_layer_f32(ghd):
    """d_model 512, 8 heads x 64, FFN 1376, KV 256, 8-node random tree of depth <= 4."""
    _layer_case(ghd, wl.TINY, 1, 8, 256, wl.random_tree(8, 4, wl.BASE_SEED + 1000))


@pytest.mark.parametrize("shape", [SMALL32, SMALL16, SMALL16_DH128], ids=["f32", "f16", "f16dh128"])
@pytest.mark.parametrize("n,L", [(1, 0), (1, 40), (13, 100), (64, 77), (100, 300), (256, 31)])
def test_small_layers(ghd, shape, n, L):
    _layer_case(ghd, shape, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6))


@pytest.mark.parametrize("n,L", [(1, 40), (13, 100), (64, 77)])
def test_small_layers_half_on_cuda_cores(ghd, n, L):
    import paper_2505_23219_b200 as g
    _layer_case(ghd, SMALL16_DH128, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6),
                opts=[(g.OPT_GEMM_PATH, 1), (g.OPT_ATTN_PATH, 1)])


@pytest.mark.parametrize("n,L", [(1, 40), (13, 100), (64, 77), (200, 5)])
def test_small_layers_forced_tcgen05_gemm(ghd, n, L):
    import paper_2505_23219_b200 as g
    _layer_case(ghd, SMALL16_DH128, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6),
                opts=[(g.OPT_GEMM_PATH, 2)])


@pytest.mark.parametrize("n,L", [(1, 40), (13, 100), (64, 77), (256, 31)])
def test_small_layers_with_the_norms_in_the_projection_epilogues(ghd, n, L):
    """RMSNorm as (gain-weighted rows + per-tile sums of squares) out of one projection and a 1 / rms column scale in the next."""
    import paper_2505_23219_b200 as g
    ctx = _layer_case(ghd, SMALL16_DH128, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6), opts=[(g.OPT_FUSED_NORM, 1)])
    assert ghd.ghd_path_count(ctx, ghd.PATH_GEMM_TILE) >= 4


def test_config2_llama7b_layer_f16_with_the_norms_in_the_projection_epilogues(ghd):
    import paper_2505_23219_b200 as g
    _layer_case(ghd, wl.LLAMA7B, 2, 64, 1024, wl.medusa_tree(64), gains=False, opts=[(g.OPT_FUSED_NORM, 1)])


def test_config2_llama7b_layer_f16(ghd):
    """LLaMA-7B-shaped layer, half weights, KV 1024, 64-node Medusa-style tree."""
    _layer_case(ghd, wl.LLAMA7B, 2, 64, 1024, wl.medusa_tree(64), gains=False)


@pytest.mark.parametrize("n,L", [(49, 200), (130, 77), (256, 300)])
def test_layer_with_a_mask_that_is_not_a_tree(ghd, n, L):
    """Whole layer under an arbitrary lower-triangular mask (position = kv_len + number of visible nodes - 1)."""
    vis = _random_mask(n, 7200 + n)
    depth = (vis.sum(axis=1) - 1).astype(np.int32)
    _layer_case(ghd, SMALL16_DH128, 15, n, L, None, vis=vis, depth=depth)
    _layer_case(ghd, SMALL16_DH128, 15, n, L, None, vis=vis, depth=None)      # depth taken from the popcount on the device


def test_forced_tcgen05_gemm_refuses_a_reduction_length_off_the_64_grid(ghd):
    """The tcgen05 projection walks the reduction in 64-wide slabs: k % 64 != 0 is outside it.  Forcing that path
    must fail cleanly (nothing launched); the automatic choice takes the CUDA-core kernel and matches the oracle."""
    ctx = make_ctx(ghd, SMALL16, 128, 64)
    n, k, m = 17, 352, 130
    x = wl.normal((n, k), 341, 1.0, dtype="f16")
    w = wl.normal((m, k), 342, 0.02, dtype="f16")
    ghd.ghd_set_option(ctx, ghd.OPT_GEMM_PATH, 2)
    before = ghd.ghd_launch_count(ctx)
    with pytest.raises(ghd.GhdError) as e:
        ghd.ghd_linear(ctx, to_dev(x), to_dev(w))
    assert e.value.name == "GHD_EUNSUPPORTED" and ghd.ghd_launch_count(ctx) == before
    ghd.ghd_set_option(ctx, ghd.OPT_GEMM_PATH, 0)
    y = ghd.ghd_linear(ctx, to_dev(x), to_dev(w))
    ghd.ghd_sync_status(ctx)
    assert ghd.ghd_path_count(ctx, ghd.PATH_GEMM_SIMT) == 1
    assert max_rel_err(y.cpu().numpy(), oracle.linear(x, w)) <= 2e-5


def test_graph_replay_notices_a_changed_option(ghd):
    """The cached graph of a step is keyed on every option that changes what is enqueued: switching the
    attention path between two graph-mode steps must re-capture, not replay the old kernels."""
    shape, n, L = SMALL16_DH128, 12, 40
    Lmax = L + n
    parent = wl.random_tree(n, 4, 811)
    head, layers, caches, gw, gkv = _model(ghd, shape, 16, L, Lmax)
    ctx = make_ctx(ghd, shape, Lmax, n)
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, 2)
    tree = ghd.ghd_tree_build(ctx, parent, L)
    tok = to_dev(wl.draft_tokens(parent, shape.vocab, 812))
    l0, a0 = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok)
    assert ghd.ghd_path_count(ctx, ghd.PATH_ATTN_TC) == shape.n_layers and ghd.ghd_path_count(ctx, ghd.PATH_ATTN_SIMT) == 0
    ghd.ghd_set_option(ctx, ghd.OPT_ATTN_PATH, 1)
    l1, a1 = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok)
    ghd.ghd_sync_status(ctx)
    assert ghd.ghd_path_count(ctx, ghd.PATH_ATTN_SIMT) == shape.n_layers, "the old graph was replayed"
    assert max_rel_err(l1.cpu().numpy(), l0.cpu().numpy()) <= 2e-2 and np.array_equal(a0.cpu().numpy(), a1.cpu().numpy())


def test_layer_with_explicit_lookahead_mask(ghd):
    vis, depth, parent = wl.lookahead_pattern(7, 5, 5)
    _layer_case(ghd, SMALL16_DH128, 12, len(parent), 200, parent, vis=vis, depth=depth)
    _layer_case(ghd, SMALL16_DH128, 12, len(parent), 200, parent, vis=vis, depth=depth, opts=[(9, 1)])     # OPT_ATTN_SPARSE: index lists


@pytest.mark.parametrize("n,L", [(13, 100), (64, 77), (256, 31)])
def test_small_layers_sparse_part_from_the_coordinate_index(ghd, n, L):
    import paper_2505_23219_b200 as g
    for shape in (SMALL32, SMALL16_DH128):
        ctx = _layer_case(ghd, shape, 11, n, L, wl.random_tree(n, 8, 40 + n, max_children=6), opts=[(g.OPT_ATTN_SPARSE, 1)])
        assert g.ghd_path_count(ctx, g.PATH_ATTN_COO) == 1


# ---------------------------------------------------------------- step
def _model(ghd, shape, config_id, L, Lmax):
    head = wl.head_weights(shape, config_id)
    layers = [wl.layer_weights(shape, config_id, l, random_gains=True) for l in range(shape.n_layers)]
    caches = [wl.kv_cache(shape, config_id, l, L, Lmax) for l in range(shape.n_layers)]
    gw = ghd.ModelWeights(to_dev(head["embed"]), [gpu_layer_weights(w) for w in layers], to_dev(head["rms_final"]),
                          to_dev(head["lm_head"]))
    gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L) for k, v in caches]
    return head, layers, caches, gw, gkv


@pytest.mark.parametrize("shape,graph", [(SMALL32, 0), (SMALL16, 0), (SMALL16, 2), (SMALL16_DH128, 0), (SMALL16_DH128, 2), (SMALL16_DH128, -1)],
                         ids=["f32", "f16", "f16graph", "f16dh128", "f16dh128graph", "f16dh128-norms-in-epilogues"])
def test_small_step_logits_argmax_accept(ghd, shape, graph):
    n, L = 24, 90
    Lmax = L + n
    parent = wl.random_tree(n, 6, 801, max_children=4)
    tokens = wl.draft_tokens(parent, shape.vocab, 802)
    head, layers, caches, gw, gkv = _model(ghd, shape, 13, L, Lmax)
    vis, _, pos = oracle.tree_build(parent, L)
    want_logits, want_amax = oracle.step(shape, head, layers, caches, L, vis, pos, tokens)
    # plant a two-token accepted path so that acceptance is not trivially zero
    c1 = parent.index(0)
    tokens[c1] = want_amax[0]
    want_logits, want_amax = oracle.step(shape, head, layers, [wl.kv_cache(shape, 13, l, L, Lmax) for l in range(shape.n_layers)],
                                         L, vis, pos, tokens)
    ctx = make_ctx(ghd, shape, Lmax, n)
    if graph < 0:
        graph = 0
        ghd.ghd_set_option(ctx, ghd.OPT_FUSED_NORM, 1)
    ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, graph)
    tree = ghd.ghd_tree_build(ctx, parent, L)
    tok_d = to_dev(tokens)
    for _ in range(2 if graph else 1):                        # second call replays the captured graph
        logits, amax = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d)
    res = ghd.ghd_accept(ctx, tree, tok_d, amax).cpu().numpy()
    ghd.ghd_sync_status(ctx)
    got = logits.cpu().numpy()
    assert max_rel_err(got, want_logits) <= tol_for(shape.dtype)
    assert argmax_margin_ok(want_logits, np.abs(got - want_logits).max()), "seed gives a near-tie; pick another"
    assert np.array_equal(amax.cpu().numpy(), want_amax)
    m, nodes, toks = oracle.accept(parent, tokens, want_amax)
    assert m >= 1 and res[0] == m and res[1] == m + 1
    assert np.array_equal(res[2:3 + m], nodes) and np.array_equal(res[258:259 + m], toks)


@pytest.mark.parametrize("n", [24, 64, 130, 200])
def test_step_is_bit_reproducible_across_reruns_and_launch_modes(ghd, n):
    """Fixed reduction orders everywhere (split tiles in worker order, KV splits in split order): the same step gives
    the same bits when it is run again, replayed from the library's graph, or run with the norms in the epilogues twice."""
    shape, L = SMALL16_DH128, 90
    Lmax = L + n
    parent = wl.random_tree(n, 6, 811 + n, max_children=4)
    tokens = wl.draft_tokens(parent, shape.vocab, 812 + n)
    head, layers, caches, gw, _ = _model(ghd, shape, 13, L, Lmax)
    tok_d = to_dev(tokens)

    def run(opts, graph, reps):
        ctx = make_ctx(ghd, shape, Lmax, n)
        for o, v in opts:
            ghd.ghd_set_option(ctx, o, v)
        ghd.ghd_set_option(ctx, ghd.OPT_GRAPH, graph)
        tree = ghd.ghd_tree_build(ctx, parent, L)
        outs = []
        for _ in range(reps):
            gkv = [ghd.KvLayer(to_dev(k), to_dev(v), L) for k, v in caches]
            logits, amax = ghd.ghd_verify_step(ctx, gw, gkv, tree, tok_d)
            ghd.ghd_sync_status(ctx)
            outs.append((logits.cpu().numpy().copy(), gkv[-1].k.cpu().numpy().copy()))
        return outs

    direct = run([], 0, 2)
    replay = run([], 2, 2)
    for lg, kc in direct[1:] + replay:
        assert np.array_equal(lg, direct[0][0]) and np.array_equal(kc, direct[0][1])
    fused = run([(ghd.OPT_FUSED_NORM, 1)], 0, 2)
    assert np.array_equal(fused[0][0], fused[1][0]) and np.array_equal(fused[0][1], fused[1][1])


def test_width1_chain_reproduces_sequential_greedy_steps_on_gpu(ghd):
    shape, k, L = SMALL32, 5, 30
    Lmax = L + k + 1
    head, layers, _, gw, _ = _model(ghd, shape, 14, L, Lmax)
    ctx = make_ctx(ghd, shape, Lmax, k + 1)
    fresh = lambda: [ghd.KvLayer(to_dev(kc), to_dev(vc), L) for kc, vc in
                     (wl.kv_cache(shape, 14, l, L, Lmax) for l in range(shape.n_layers))]
    gkv = fresh()
    tok, seq = 5, []
    for s in range(k + 1):                                    # sequential decoding, one node per step
        for kv in gkv:
            kv.len = L + s
        tree = ghd.ghd_tree_build(ctx, [-1], L + s)
        _, am = ghd.ghd_verify_step(ctx, gw, gkv, tree, to_dev(np.array([tok], np.int32)))
        tok = int(am.cpu()[0])
        seq.append(tok)
    parent = wl.chain_tree(k + 1)
    tree = ghd.ghd_tree_build(ctx, parent, L)
    tokens = to_dev(np.array([5] + seq[:k], np.int32))
    _, am = ghd.ghd_verify_step(ctx, gw, fresh(), tree, tokens)
    res = ghd.ghd_accept(ctx, tree, tokens, am).cpu().numpy()
    ghd.ghd_sync_status(ctx)
    assert list(am.cpu().numpy()) == seq
    assert res[0] == k and list(res[258:259 + k]) == seq
