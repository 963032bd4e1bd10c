"""The allocation-free attention entry point against the CPU oracle and the ordinary entry point.

``ghd_tree_attention_static`` serves callers that are not allowed to allocate GPU
memory (code living inside someone else's fixed memory pool, plugins with a frozen
memory budget, loops where cudaMalloc may not be called): it keeps its split
partials in an array compiled into the library instead of a caller workspace.  Here
it is called twice in a row, on two different problems, and each result must match
``oracle.tree_attention`` (and ``ghd_tree_attention``) within the tolerance the other
attention tests use.  The
second call sees whatever the first one left in the shared array, which is the
point of running two.  This file is named so that pytest collects it last.
"""
import numpy as np
import pytest

import oracle
import workloads as wl
from util import gpu_cfg, max_rel_err, to_dev

pytestmark = pytest.mark.gpu

SHAPE16 = wl.scaled(wl.TINY, name="na16", d_model=512, n_heads=4, d_head=128, d_ffn=704, vocab=100, n_layers=1,
                    dtype="f16")
SHAPE32 = wl.scaled(wl.TINY, name="na32", d_model=256, n_heads=4, d_head=64, d_ffn=352, vocab=100, n_layers=1)


def _both(ghd, shape, n, L, seed):
    import torch
    Lmax = L + n + 5
    ctx = ghd.ghd_create(gpu_cfg(shape, Lmax, 64))
    H, dh, dt = shape.n_heads, shape.d_head, shape.dtype
    q_h = wl.normal((n, H, dh), seed, dtype=dt)
    kc_h = wl.normal((H, Lmax, dh), seed + 1, dtype=dt)          # rows [L, L+n) play the appended new rows
    vc_h = wl.normal((H, Lmax, dh), seed + 2, dtype=dt)
    parent = wl.random_tree(n, 6, seed + 3, max_children=5)
    vis, _, _ = oracle.tree_build(parent, L)
    want = oracle.tree_attention(q_h, kc_h[:, L:L + n].transpose(1, 0, 2), vc_h[:, L:L + n].transpose(1, 0, 2), kc_h, vc_h, L, vis)
    q, kc, vc = to_dev(q_h.reshape(n, H * dh)), to_dev(kc_h), to_dev(vc_h)
    tree = ghd.ghd_tree_build(ctx, parent, L)
    other = ghd.ghd_tree_attention(ctx, q, ghd.KvLayer(kc, vc, L), tree)
    ghd.ghd_sync_status(ctx)
    got = ghd.ghd_tree_attention_static(q, kc, vc, tree.mask, H, dh, L)
    torch.cuda.synchronize()
    return got.float().cpu().numpy(), want.reshape(n, H * dh), other.float().cpu().numpy()


def test_static_scratch_attention_matches_the_oracle_twice_in_a_row():
    import paper_2505_23219_b200 as ghd
    # first call: 8 splits over a long cache; second: a short problem that uses fewer slots
    for shape, n, L, seed in [(SHAPE16, 64, 1900, 9100), (SHAPE32, 9, 70, 9200)]:
        got, want, other = _both(ghd, shape, n, L, seed)
        tol = 2e-5 if shape.dtype == "f32" else 2e-3
        assert np.isfinite(got).all()
        assert max_rel_err(got, want) <= tol                      # the CPU oracle
        assert max_rel_err(got, other) <= tol                     # the entry point that takes a workspace


def test_static_scratch_attention_rejects_sizes_beyond_its_array():
    import torch
    import paper_2505_23219_b200 as ghd
    q = torch.zeros((65, 256), dtype=torch.float16, device="cuda")
    kc = torch.zeros((4, 128, 64), dtype=torch.float16, device="cuda")
    mask = torch.zeros(65 * 2, dtype=torch.int64, device="cuda")
    with pytest.raises(ghd.GhdError) as e:                      # 65 nodes > 64
        ghd.ghd_tree_attention_static(q, kc, kc, mask, 4, 64, 10)
    assert e.value.name == "GHD_ENOSPACE" and "64 tree nodes" in str(e.value)
    wide = torch.zeros((4, 8192), dtype=torch.float16, device="cuda")
    kw = torch.zeros((64, 16, 128), dtype=torch.float16, device="cuda")
    with pytest.raises(ghd.GhdError) as e:                      # 64 heads x 128 > 4096
        ghd.ghd_tree_attention_static(wide, kw, kw, mask, 64, 128, 4)
    assert e.value.name == "GHD_ENOSPACE"
