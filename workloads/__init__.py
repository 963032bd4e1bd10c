"""Seeded synthetic inputs for the tree-verification step.

Everything here only *describes* inputs: model shapes, pseudo-random tensors,
draft-tree topologies and draft tokens.  None of the verify step's arithmetic
(norms, projections, attention, acceptance) lives in this package; it serves
both the CPU oracle's tests and the GPU path's tests and benchmark so that the
two sides always see byte-identical inputs.

Tensors come from a counter-based generator (SplitMix64 + Box-Muller, see
``gen.c``) compiled on first use into ``libwl.so`` next to this file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_LIB = None

BASE_SEED = 20250523


def build(force: bool = False) -> Path:
    """Compile ``gen.c`` into ``libwl.so`` (no-op when it is up to date)."""
    src, out = _HERE / "gen.c", _HERE / "libwl.so"
    if force or not out.exists() or out.stat().st_mtime < src.stat().st_mtime:
        tmp = out.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(src), "-lm"])
        os.replace(tmp, out)
    return out


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(str(build()))
        u64, dbl, vp = ctypes.c_uint64, ctypes.c_double, ctypes.c_void_p
        lib.wl_fill_normal_f32.argtypes = [vp, u64, u64, u64, dbl, dbl]
        lib.wl_fill_normal_f16.argtypes = [vp, u64, u64, u64, dbl, dbl]
        lib.wl_fill_u64.argtypes = [vp, u64, u64, u64]
        for f in (lib.wl_fill_normal_f32, lib.wl_fill_normal_f16, lib.wl_fill_u64):
            f.restype = None
        _LIB = lib
    return _LIB


# --------------------------------------------------------------------------
# tensors
# --------------------------------------------------------------------------
def normal(shape, seed: int, std: float = 1.0, mean: float = 0.0, dtype="f32",
           first: int = 0) -> np.ndarray:
    """N(mean, std) tensor of ``shape``; dtype 'f32' -> float32, 'f16' -> float16."""
    count = int(np.prod(shape, dtype=np.int64))
    if dtype == "f32":
        out = np.empty(count, dtype=np.float32)
        _lib().wl_fill_normal_f32(out.ctypes.data, first, count, seed & (2**64 - 1), mean, std)
    elif dtype == "f16":
        out = np.empty(count, dtype=np.float16)
        _lib().wl_fill_normal_f16(out.ctypes.data, first, count, seed & (2**64 - 1), mean, std)
    else:
        raise ValueError(dtype)
    return out.reshape(shape)


def u64_stream(count: int, seed: int, first: int = 0) -> np.ndarray:
    out = np.empty(count, dtype=np.uint64)
    _lib().wl_fill_u64(out.ctypes.data, first, count, seed & (2**64 - 1))
    return out


class Rng:
    """Small sequential integer source on top of the counter-based stream."""

    def __init__(self, seed: int):
        self.seed, self.ctr = seed, 0

    def u64(self) -> int:
        v = int(u64_stream(1, self.seed, self.ctr)[0])
        self.ctr += 1
        return v

    def below(self, n: int) -> int:
        return self.u64() % n


# --------------------------------------------------------------------------
# model shapes
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class ModelShape:
    name: str
    d_model: int
    n_heads: int
    d_head: int
    d_ffn: int
    vocab: int
    n_layers: int
    dtype: str            # 'f32' or 'f16' (storage type of weights, KV and activations)
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0

    @property
    def params_per_layer(self) -> int:
        d, f = self.d_model, self.d_ffn
        return 4 * d * d + 3 * d * f

    @property
    def itemsize(self) -> int:
        return 4 if self.dtype == "f32" else 2


TINY = ModelShape("tiny", 512, 8, 64, 1376, 1000, 1, "f32")
LLAMA7B = ModelShape("llama7b", 4096, 32, 128, 11008, 32000, 32, "f16")
LLAMA13B = ModelShape("llama13b", 5120, 40, 128, 13824, 32000, 40, "f16")


def scaled(shape: ModelShape, **kw) -> ModelShape:
    return replace(shape, **kw)


def _tensor_seed(config_id: int, tensor_id: int) -> int:
    return BASE_SEED + 1000 * config_id + tensor_id


def layer_weights(shape: ModelShape, config_id: int, layer: int = 0,
                  random_gains: bool = False) -> dict:
    """Weights of one decoder layer, stored [out_features][in_features], N(0, 0.02)."""
    d, f, dt = shape.d_model, shape.d_ffn, shape.dtype
    s = lambda t: _tensor_seed(config_id, 16 * layer + t)
    w = {
        "wqkv": normal((3 * d, d), s(0), 0.02, dtype=dt),
        "wo": normal((d, d), s(1), 0.02, dtype=dt),
        "w_gate_up": normal((2 * f, d), s(2), 0.02, dtype=dt),
        "w_down": normal((d, f), s(3), 0.02, dtype=dt),
    }
    if random_gains:
        w["rms1"] = normal((d,), s(4), 0.02, 1.0, dtype=dt)
        w["rms2"] = normal((d,), s(5), 0.02, 1.0, dtype=dt)
    else:
        w["rms1"] = np.ones(d, dtype=np.float32 if dt == "f32" else np.float16)
        w["rms2"] = np.ones(d, dtype=np.float32 if dt == "f32" else np.float16)
    return w


def head_weights(shape: ModelShape, config_id: int, embed_std: float = 1.0) -> dict:
    """Embedding table, final norm gain and lm_head ([vocab][d_model])."""
    d, v, dt = shape.d_model, shape.vocab, shape.dtype
    s = lambda t: _tensor_seed(config_id, 900 + t)
    return {
        "embed": normal((v, d), s(0), embed_std, dtype=dt),
        "rms_final": np.ones(d, dtype=np.float32 if dt == "f32" else np.float16),
        "lm_head": normal((v, d), s(1), 0.02, dtype=dt),
    }


def kv_cache(shape: ModelShape, config_id: int, layer: int, kv_len: int, max_kv_len: int):
    """K and V caches [n_heads][max_kv_len][d_head]; rows < kv_len are N(0,1), the rest 0."""
    h, dh, dt = shape.n_heads, shape.d_head, shape.dtype
    npdt = np.float32 if dt == "f32" else np.float16
    out = []
    for which in (0, 1):
        c = np.zeros((h, max_kv_len, dh), dtype=npdt)
        if kv_len:
            c[:, :kv_len, :] = normal((h, kv_len, dh), _tensor_seed(config_id, 500 + 16 * layer + which),
                                      1.0, dtype=dt)
        out.append(c)
    return out[0], out[1]


def layer_input(shape: ModelShape, config_id: int, n: int) -> np.ndarray:
    return normal((n, shape.d_model), _tensor_seed(config_id, 990), 1.0, dtype=shape.dtype)


# --------------------------------------------------------------------------
# draft trees (parent arrays; node 0 is the root, parent[i] < i)
# --------------------------------------------------------------------------
def depths_of(parent) -> list:
    depth = [0] * len(parent)
    for i in range(1, len(parent)):
        depth[i] = depth[parent[i]] + 1
    return depth


def chain_tree(n: int) -> list:
    return [-1] + list(range(n - 1))


def star_tree(n: int) -> list:
    return [-1] + [0] * (n - 1)


def random_tree(n: int, max_depth: int, seed: int, max_children: int | None = None) -> list:
    """parent[i] uniform among earlier nodes of depth < max_depth (and with room for a child)."""
    rng = Rng(seed)
    parent, depth, kids = [-1], [0], [0]
    for i in range(1, n):
        cand = [j for j in range(i) if depth[j] < max_depth
                and (max_children is None or kids[j] < max_children)]
        p = cand[rng.below(len(cand))]
        parent.append(p)
        depth.append(depth[p] + 1)
        kids[p] += 1
        kids.append(0)
    return parent


def medusa_tree(n: int = 64, caps=(10, 4, 2, 1, 1)) -> list:
    """Static Medusa-style tree grown greedily by estimated path accuracy.

    Candidate (level l, rank r) gets a synthetic accuracy 0.6 * 0.8**l * 0.5**r;
    a node's score is the product along its path.  Starting from the root, the
    best-scoring candidate whose parent is already in the tree is added until
    the tree has ``n`` nodes (root included); ties go to the shallower node,
    then the lexicographically smaller rank path.  Nodes are renumbered in
    breadth-first order.
    """
    acc = lambda l, r: 0.6 * 0.8 ** l * 0.5 ** r
    chosen = {(): 1.0}
    while len(chosen) < n:
        best = None
        for path, score in chosen.items():
            l = len(path)
            if l >= len(caps):
                continue
            for r in range(caps[l]):
                child = path + (r,)
                if child in chosen:
                    continue
                key = (-score * acc(l, r), l + 1, child)
                if best is None or key < best[0]:
                    best = (key, child, score * acc(l, r))
                break  # ranks are added in order: only the lowest missing rank is a candidate
        if best is None:
            raise ValueError("caps too small for requested width")
        chosen[best[1]] = best[2]
    order = sorted(chosen, key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(order)}
    return [-1 if not p else index[p[:-1]] for p in order]


def lookahead_pattern(window: int = 7, ngram: int = 5, guesses: int = 5):
    """Lookahead-decoding style 2-D window plus guess n-grams, as an explicit visibility matrix.

    Nodes: the root; (ngram-1) window levels of ``window`` columns; ``guesses``
    chains of (ngram-1) tokens.  Window token (level r, column c) sees the root,
    level-0 columns 0..c and levels 1..r of column c; a guess token sees the
    root and the earlier tokens of its own n-gram.  Returns (visible[n][n] bool,
    depth[n], parent[n]) where ``parent`` is the tree this pattern is equivalent
    to (every visible set is a prefix-closed chain).
    """
    lv = ngram - 1
    idx_w = lambda r, c: 1 + r * window + c
    idx_g = lambda g, t: 1 + lv * window + g * lv + t
    n = 1 + lv * window + guesses * lv
    vis = np.zeros((n, n), dtype=bool)
    parent = [-1] * n
    vis[0, 0] = True
    for r in range(lv):
        for c in range(window):
            i = idx_w(r, c)
            vis[i, 0] = True
            for cc in range(c + 1):
                vis[i, idx_w(0, cc)] = True
            for rr in range(1, r + 1):
                vis[i, idx_w(rr, c)] = True
            parent[i] = (0 if c == 0 else idx_w(0, c - 1)) if r == 0 else idx_w(r - 1, c)
    for g in range(guesses):
        for t in range(lv):
            i = idx_g(g, t)
            vis[i, 0] = True
            for tt in range(t + 1):
                vis[i, idx_g(g, tt)] = True
            parent[i] = 0 if t == 0 else idx_g(g, t - 1)
    depth = (vis.sum(axis=1) - 1).astype(np.int32)
    return vis, depth, parent


def draft_tokens(parent, vocab: int, seed: int) -> np.ndarray:
    """Token id per node, uniform in [0, vocab), siblings pairwise distinct."""
    rng = Rng(seed)
    n = len(parent)
    tok = np.zeros(n, dtype=np.int32)
    used = {}
    for i in range(n):
        taken = used.setdefault(parent[i], set())
        while True:
            t = rng.below(vocab)
            if t not in taken:
                break
        taken.add(t)
        tok[i] = t
    return tok
