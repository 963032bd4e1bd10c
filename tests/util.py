"""Helpers shared by the GPU parity tests: upload seeded inputs, compare with the oracle."""
from __future__ import annotations

import numpy as np

import workloads as wl


def max_rel_err(got, want) -> float:
    """max_i |got_i - want_i| / max_j |want_j| over the whole tensor."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    scale = np.abs(want).max()
    return float(np.abs(got - want).max() / (scale if scale > 0 else 1.0))


def unpack_mask(words: np.ndarray, n: int) -> np.ndarray:
    """uint64 [n][W] -> uint8 [n][n]."""
    out = np.zeros((n, n), dtype=np.uint8)
    for i in range(n):
        for j in range(n):
            out[i, j] = (int(words[i, j // 64]) >> (j % 64)) & 1
    return out


def tol_for(dtype: str) -> float:
    # stated bar: 2e-2 with half inputs / float accumulation, 1e-4 in float mode
    return 1e-4 if dtype == "f32" else 2e-2


def to_dev(a: np.ndarray):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_cfg(shape: wl.ModelShape, max_kv_len: int, max_nodes: int, n_layers: int | None = None):
    import paper_2505_23219_b200 as ghd
    return ghd.ModelCfg(shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab,
                        shape.n_layers if n_layers is None else n_layers, max_kv_len, max_nodes, shape.dtype,
                        shape.rms_eps, shape.rope_theta)


def gpu_layer_weights(w: dict):
    import paper_2505_23219_b200 as ghd
    return ghd.LayerWeights(**{k: to_dev(w[k]) for k in ghd.LayerWeights.FIELDS})


def argmax_margin_ok(logits64: np.ndarray, abs_err: float) -> bool:
    """True when every row's top-1/top-2 gap exceeds 8x the observed absolute logit error."""
    part = np.partition(logits64, -2, axis=1)
    return bool(((part[:, -1] - part[:, -2]) > 8.0 * abs_err).all())
