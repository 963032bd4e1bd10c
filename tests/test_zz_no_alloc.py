"""The allocation-free attention entry point against the ordinary one.

``ghd_tree_attention_static`` serves callers that are not allowed to allocate GPU
memory (code living inside someone else's fixed memory pool, plugins with a frozen
memory budget, loops where cudaMalloc may not be called): it keeps its split
partials in an array compiled into the library instead of a caller workspace.  Here
it is called twice in a row, on two different problems, and each result must match
``ghd_tree_attention`` within the tolerance the other attention tests use.  The
second call sees whatever the first one left in the shared array, which is the
point of running two.  This file is named so that pytest collects it last.
"""
import numpy as np
import pytest

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
    q = to_dev(wl.normal((n, H * dh), seed, dtype=dt))
    kc = to_dev(wl.normal((H, Lmax, dh), seed + 1, dtype=dt))
    vc = to_dev(wl.normal((H, Lmax, dh), seed + 2, dtype=dt))
    tree = ghd.ghd_tree_build(ctx, wl.random_tree(n, 6, seed + 3, max_children=5), L)
    want = ghd.ghd_tree_attention(ctx, q, ghd.KvLayer(kc, vc, L), tree)
    ghd.ghd_sync_status(ctx)
    got = ghd.ghd_tree_attention_static(q, kc, vc, tree.mask, H, dh, L)
    torch.cuda.synchronize()
    return got.float().cpu().numpy(), want.float().cpu().numpy()


def test_static_scratch_attention_matches_workspace_attention_twice_in_a_row():
    import paper_2505_23219_b200 as ghd
    # first call: 8 splits over a long cache; second: a short problem that uses fewer slots
    for shape, n, L, seed in [(SHAPE16, 64, 1900, 9100), (SHAPE32, 9, 70, 9200)]:
        got, want = _both(ghd, shape, n, L, seed)
        assert np.isfinite(got).all()
        assert max_rel_err(got, want) <= (2e-5 if shape.dtype == "f32" else 2e-3)


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
