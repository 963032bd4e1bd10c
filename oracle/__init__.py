"""ctypes front end of the CPU oracle (``ghd_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline use it; the GPU package never imports it and it never imports the GPU
package.  All floating-point arrays crossing this interface are float64 except
weights, embeddings and KV caches, which keep their storage type (float16 or
float32) and are read exactly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "ghd_oracle.cpp"
_SO = _HERE / "libghd_oracle.so"
_INFO = _HERE / "libghd_oracle.buildinfo"
_LIB = None

_DT = {np.dtype(np.float32): 0, np.dtype(np.float16): 1, np.dtype(np.float64): 2}


def _cpu_flags() -> set:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("flags"):
                return set(line.split(":", 1)[1].split())
    except OSError:
        pass
    return set()


def build(force: bool = False) -> Path:
    """Compile the oracle; rebuilt when the source is newer or this CPU lacks a
    vector extension the existing binary was compiled for."""
    have = _cpu_flags()
    want = [f for f in ("avx2", "fma", "f16c") if f in have]
    stale = force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime
    if not stale:
        built = _INFO.read_text().split() if _INFO.exists() else ["?"]
        stale = any(f not in have for f in built)
    if stale:
        tmp = _SO.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp"] + [f"-m{f}" for f in want]
        subprocess.check_call(cmd + ["-o", str(tmp), str(_SRC)])
        os.replace(tmp, _SO)
        _INFO.write_text(" ".join(want))
    return _SO


class _Cfg(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in
                ("d_model", "n_heads", "d_head", "d_ffn", "vocab", "n_layers", "max_kv_len", "dtype")] + \
               [("rms_eps", ctypes.c_double), ("rope_theta", ctypes.c_double)]


class _LayerW(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in ("wqkv", "wo", "w_gate_up", "w_down", "rms1", "rms2")]


class _KV(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p)]


def _lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(str(build()))
        _LIB.orc_tree_build.restype = ctypes.c_int
        _LIB.orc_accept.restype = ctypes.c_int
    return _LIB


def n_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else len(os.sched_getaffinity(0))


def _p(a):
    return ctypes.c_void_p(a.ctypes.data)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _stored(a):
    a = np.ascontiguousarray(a)
    if a.dtype not in _DT:
        raise TypeError(a.dtype)
    return a


def _cfg(shape, max_kv_len: int, n_layers: int | None = None) -> _Cfg:
    return _Cfg(shape.d_model, shape.n_heads, shape.d_head, shape.d_ffn, shape.vocab,
                shape.n_layers if n_layers is None else n_layers, max_kv_len,
                0 if shape.dtype == "f32" else 1, shape.rms_eps, shape.rope_theta)


def tree_build(parent, kv_len: int):
    """-> (vis uint8 [n][n], depth int32 [n], pos int32 [n]); ValueError on a bad parent array."""
    parent = _i32(parent)
    n = parent.size
    vis = np.zeros((max(n, 1), max(n, 1)), dtype=np.uint8)
    depth = np.zeros(max(n, 1), dtype=np.int32)
    pos = np.zeros(max(n, 1), dtype=np.int32)
    if n == 0 or _lib().orc_tree_build(_p(parent), n, kv_len, _p(vis), _p(depth), _p(pos)) != 0:
        raise ValueError("invalid parent array")
    return vis, depth, pos


def coo_index(vis):
    """The visibility among the drafted nodes as a sparse index in coordinate order (paper Sec. III-B-3: the
    index of the token pairs to verify is written down before the inference): every (query i, node j) with
    vis[i][j] set, sorted by i then j, plus the row starts.  -> (ptr int32 [n + 1], cols int32 [nnz]).
    Plain restatement: a scan of the matrix, one pair at a time."""
    vis = np.asarray(vis)
    n = vis.shape[0]
    ptr, cols = [0], []
    for i in range(n):
        for j in range(n):
            if vis[i][j]:
                cols.append(j)
        ptr.append(len(cols))
    return np.asarray(ptr, dtype=np.int32), np.asarray(cols, dtype=np.int32)


def rmsnorm(x, g, eps: float):
    x, g = _f64(x), _stored(g)
    out = np.empty_like(x)
    _lib().orc_rmsnorm(_p(x), _p(g), _DT[g.dtype], x.shape[0], x.shape[1], ctypes.c_double(eps), _p(out))
    return out


def linear(x, w):
    """x [n][k] (any float type, used as double) times w [m][k] transposed -> [n][m] float64."""
    x, w = _f64(x), _stored(w)
    n, k = x.shape
    m = w.shape[0]
    assert w.shape[1] == k
    y = np.empty((n, m), dtype=np.float64)
    _lib().orc_linear(_p(x), _p(w), _DT[w.dtype], n, k, m, _p(y))
    return y


def rope(u, pos, theta: float):
    """u [n][heads][dh] -> rotated copy."""
    u = _f64(u).copy()
    pos = _i32(pos)
    n, h, dh = u.shape
    _lib().orc_rope(_p(u), _p(pos), n, h, dh, ctypes.c_double(theta))
    return u


def tree_attention(q, k_new, v_new, k_cache, v_cache, kv_len: int, vis):
    """q, k_new, v_new [n][heads][dh]; caches [heads][Lmax][dh] -> out [n][heads][dh]."""
    q, k_new, v_new = _f64(q), _f64(k_new), _f64(v_new)
    k_cache, v_cache = _stored(k_cache), _stored(v_cache)
    vis = np.ascontiguousarray(vis, dtype=np.uint8)
    n, h, dh = q.shape
    out = np.empty_like(q)
    _lib().orc_tree_attention(_p(q), _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), _DT[k_cache.dtype],
                              n, h, dh, kv_len, k_cache.shape[1], _p(vis), _p(out))
    return out


def _layer_struct(w: dict) -> _LayerW:
    return _LayerW(*[w[k].ctypes.data for k in ("wqkv", "wo", "w_gate_up", "w_down", "rms1", "rms2")])


def layer(shape, w: dict, k_cache, v_cache, kv_len: int, vis, pos, x, want_attn: bool = False):
    """One decoder layer; writes the new K/V rows into the caches in place.
    -> y float64 [n][d]  (and the concatenated attention output if asked)."""
    x = _f64(x)
    n = x.shape[0]
    vis = np.ascontiguousarray(vis, dtype=np.uint8)
    pos = _i32(pos)
    assert k_cache.flags.c_contiguous and v_cache.flags.c_contiguous
    assert kv_len + n <= k_cache.shape[1]
    cfg = _cfg(shape, k_cache.shape[1])
    lw = _layer_struct(w)
    kv = _KV(k_cache.ctypes.data, v_cache.ctypes.data)
    y = np.empty_like(x)
    attn = np.empty_like(x) if want_attn else None
    _lib().orc_layer(ctypes.byref(cfg), ctypes.byref(lw), ctypes.byref(kv), kv_len, n, _p(vis), _p(pos),
                     _p(x), _p(y), _p(attn) if want_attn else None)
    return (y, attn) if want_attn else y


def argmax(logits):
    logits = _f64(logits)
    out = np.empty(logits.shape[0], dtype=np.int32)
    _lib().orc_argmax(_p(logits), logits.shape[0], logits.shape[1], _p(out))
    return out


def step(shape, head: dict, layers: list, caches: list, kv_len: int, vis, pos, tokens,
         want_hidden: bool = False):
    """Whole verify step.  caches: list of (k, v) per layer, appended to in place.
    -> (logits float64 [n][vocab], argmax int32 [n])  (+ hidden [n][d] if asked)."""
    tokens = _i32(tokens)
    n = tokens.size
    vis = np.ascontiguousarray(vis, dtype=np.uint8)
    pos = _i32(pos)
    nl = len(layers)
    cfg = _cfg(shape, caches[0][0].shape[1], nl)
    lws = (_LayerW * nl)(*[_layer_struct(w) for w in layers])
    kvs = (_KV * nl)(*[_KV(k.ctypes.data, v.ctypes.data) for k, v in caches[:nl]])
    logits = np.empty((n, shape.vocab), dtype=np.float64)
    amax = np.empty(n, dtype=np.int32)
    hidden = np.empty((n, shape.d_model), dtype=np.float64) if want_hidden else None
    _lib().orc_step(ctypes.byref(cfg), _p(head["embed"]), lws, _p(head["rms_final"]), _p(head["lm_head"]),
                    kvs, kv_len, n, _p(vis), _p(pos), _p(tokens), _p(logits), _p(amax),
                    _p(hidden) if want_hidden else None)
    return (logits, amax, hidden) if want_hidden else (logits, amax)


def accept(parent, tokens, amax):
    """-> (n_matched, nodes int32 [n_matched+1], emitted tokens int32 [n_matched+1])."""
    parent, tokens, amax = _i32(parent), _i32(tokens), _i32(amax)
    n = parent.size
    nodes = np.zeros(n, dtype=np.int32)
    toks = np.zeros(n, dtype=np.int32)
    m = _lib().orc_accept(_p(parent), _p(tokens), _p(amax), n, _p(nodes), _p(toks))
    return m, nodes[:m + 1].copy(), toks[:m + 1].copy()


def kv_commit(caches: list, kv_len: int, nodes) -> None:
    """What a step keeps of the rows it appended (paper Sec. II-A, II-C): in every layer's (k, v) the
    row of accepted node nodes[j], written at slot kv_len + nodes[j], becomes row kv_len + j.
    Plain definition: all sources are read from a snapshot before anything is written."""
    nodes = [int(x) for x in nodes]
    for k, v in caches:
        for a in (k, v):
            snap = a[:, kv_len:kv_len + max(nodes) + 1].copy()
            for j, node in enumerate(nodes):
                a[:, kv_len + j] = snap[:, node]


# ---------------------------------------------------------------- verification-tree design and width choice
# Paper Sec. III-C-1: the accuracy of a candidate sequence is estimated as the product of the calibrated
# accuracies of its tokens; the expected acceptance length is the sum over the candidate sequences; the tree
# for a given width is grown by adding the node of highest estimated accuracy one by one.  Sec. III-C-2 /
# IV-C: the width is the one that maximises decoding speed, acceptance length over measured step latency.
def arca_tree(acc, width: int):
    """acc[l][r]: accuracy of the rank-r candidate of drafting head l (level l + 1 of the tree).
    -> (parent list in breadth-first order, probability that each node is accepted).
    Plain restatement: every round scans every node of the tree and every child it could still get."""
    chosen = {(): 1.0}
    while len(chosen) < width:
        best = None
        for path, prob in chosen.items():
            if len(path) >= len(acc):
                continue
            for r in range(len(acc[len(path)])):
                child = path + (r,)
                if child in chosen:
                    continue
                cand = (prob * acc[len(path)][r], -len(child), tuple(-x for x in child))
                if best is None or cand > best[0]:
                    best = (cand, child)
        if best is None:
            break
        chosen[best[1]] = best[0][0]
    order = sorted(chosen, key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(order)}
    return [-1 if not p else index[p[:-1]] for p in order], [chosen[p] for p in order]


def expected_acceptance(node_prob) -> float:
    """Expected tokens per step: every accepted node yields one token and the root's is certain
    (acceptance length 1 at width 1, paper Table I)."""
    return float(sum(node_prob))


def best_width(latency_us: dict, acc, widths=None):
    """-> (width with the highest expected tokens per second, {width: (tokens per step, tokens per second)})."""
    table = {}
    for w in (widths or sorted(latency_us)):
        _, prob = arca_tree(acc, w)
        tau = expected_acceptance(prob)
        table[w] = (tau, tau / (latency_us[w] * 1e-6))
    return max(table, key=lambda w: (table[w][1], -w)), table


# ---------------------------------------------------------------- drafting heads
def medusa_draft(h, w1, w2, topk):
    """Self-drafting heads on one hidden state h [d] (paper Sec. II-C: extra heads at the tail of the model predict
    the tokens of the following slots; head internals as in Medusa: y_k = h + SiLU(W1_k h), logits_k = W2_k y_k).
    w1 [K][d][d], w2 [K][V][d] in storage type, read exactly; arithmetic in float64.
    -> (candidates: list of K int lists, best first, ties to the lower id; logits float64 [K][V])."""
    h = np.asarray(h, dtype=np.float64)
    cands, logits = [], []
    for k in range(len(topk)):
        a = np.asarray(w1[k], dtype=np.float64) @ h
        y = h + a / (1.0 + np.exp(-a))
        z = np.asarray(w2[k], dtype=np.float64) @ y
        order = sorted(range(z.size), key=lambda i: (-z[i], i))
        cands.append(order[:topk[k]])
        logits.append(z)
    return cands, np.stack(logits)


def tree_fill_tokens(cands, bonus: int, level, rank):
    """Token slots of the next tree: the root carries the bonus token, node i the rank[i]-th candidate of head level[i] - 1."""
    return np.array([bonus] + [cands[level[i] - 1][rank[i]] for i in range(1, len(level))], dtype=np.int32)
