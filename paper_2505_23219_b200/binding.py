"""ctypes binding of ``libghd.so``: same names as the C-ABI, torch tensors in.

Only argument marshalling happens here.  Device buffers are torch tensors (the
library borrows them), the stream is torch's current stream at context creation.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import numpy as np
import torch

from . import build as _build

__all__ = [
    "GhdError", "ModelCfg", "LayerWeights", "ModelWeights", "KvLayer", "Tree", "Ctx", "load_library",
    "ghd_create", "ghd_destroy", "ghd_set_option", "ghd_tree_build", "ghd_tree_from_mask", "ghd_verify_layer",
    "ghd_verify_step", "ghd_accept", "ghd_linear", "ghd_rmsnorm", "ghd_tree_attention", "ghd_argmax",
    "ghd_sync_status", "ghd_launch_count", "pack_mask", "ghd_copy_hidden", "ghd_gate_up", "ghd_tree_attention_static", "ghd_path_count", "ghd_kv_commit", "ghd_medusa_draft", "ghd_tree_fill_tokens",
    "ghd_kv_len_set", "ghd_kv_len_get", "KV_LEN_DEVICE", "MedusaWeights", "GHD_MAX_TOPK",
    "PATH_GEMM_TILE", "PATH_GEMM_SIMT", "PATH_ATTN_TC", "PATH_ATTN_SIMT", "PATH_ATTN_COO", "PATH_GEMM_PAIR", "OPT_GEMM_PAIR", "OPT_ATTN_ROWS", "OPT_GEMM_SKEW", "OPT_ATTN_SMALL",
    "GHD_F32", "GHD_F16", "GHD_MAX_NODES", "OPT_GEMM_PATH", "OPT_ATTN_SPLITS", "OPT_ATTN_PATH", "OPT_GRAPH",
    "OPT_GEMM_CTAS", "OPT_GEMM_BURST", "OPT_NO_PDL", "OPT_GEMM_STAGES", "OPT_GEMM_EPI", "OPT_ATTN_SPARSE", "OPT_CHAIN_CALLS", "OPT_FUSED_NORM", "EXPORTS",
]

GHD_F32, GHD_F16 = 0, 1
GHD_MAX_NODES = 256
GHD_MAX_TOPK = 16
KV_LEN_DEVICE = -1      # "take the cache length from the context's device word"
OPT_GEMM_PATH, OPT_ATTN_SPLITS, OPT_ATTN_PATH, OPT_GRAPH, OPT_GEMM_CTAS, OPT_GEMM_BURST, OPT_NO_PDL = 0, 1, 2, 3, 4, 5, 6
OPT_GEMM_STAGES, OPT_GEMM_EPI, OPT_ATTN_SPARSE, OPT_CHAIN_CALLS, OPT_FUSED_NORM = 7, 8, 9, 10, 11
PATH_GEMM_TILE, PATH_GEMM_SIMT, PATH_ATTN_TC, PATH_ATTN_SIMT, PATH_ATTN_COO, PATH_GEMM_PAIR = 0, 1, 2, 3, 4, 5
OPT_GEMM_PAIR, OPT_ATTN_ROWS, OPT_GEMM_SKEW, OPT_ATTN_SMALL = 12, 13, 14, 15
_STATUS = ["GHD_OK", "GHD_EINVAL", "GHD_ESHAPE", "GHD_ETREE", "GHD_ENOSPACE", "GHD_ECUDA", "GHD_ETIMEOUT",
           "GHD_EUNSUPPORTED"]

# every symbol include/ghd.h declares
EXPORTS = [
    "ghd_create", "ghd_destroy", "ghd_workspace_bytes", "ghd_set_workspace", "ghd_set_option", "ghd_tree_build",
    "ghd_tree_from_mask", "ghd_verify_layer", "ghd_verify_step", "ghd_accept", "ghd_linear", "ghd_rmsnorm",
    "ghd_tree_attention", "ghd_argmax", "ghd_sync_status", "ghd_status_str", "ghd_last_error", "ghd_launch_count",
    "ghd_tree_attention_static", "ghd_path_count", "ghd_kv_commit", "ghd_kv_len_set", "ghd_kv_len_get",
    "ghd_medusa_draft", "ghd_tree_fill_tokens", "ghd_copy_hidden", "ghd_gate_up",
]


class GhdError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        self.name = _STATUS[status] if 0 <= status < len(_STATUS) else str(status)
        super().__init__(f"{self.name}: {detail}" if detail else self.name)


class _Cfg(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("d_model", "n_heads", "n_kv_heads", "d_head", "d_ffn", "vocab", "n_layers",
                                          "max_kv_len", "max_nodes", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)]


class _LayerW(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("wqkv", "wo", "w_gate_up", "w_down", "rms1", "rms2")]


class _ModelW(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("layers", C.POINTER(_LayerW)), ("rms_final", C.c_void_p),
                ("lm_head", C.c_void_p)]


class _MedusaW(C.Structure):
    _fields_ = [("n_heads", C.c_int32), ("w1", C.c_void_p), ("w2", C.c_void_p)]


class _Kv(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("len", C.c_int32)]


class _Tree(C.Structure):
    _fields_ = [("n", C.c_int32), ("kv_len", C.c_int32), ("n_words", C.c_int32), ("has_parent", C.c_int32),
                ("mask", C.c_void_p), ("parent", C.c_void_p), ("depth", C.c_void_p), ("pos", C.c_void_p),
                ("rope", C.c_void_p), ("coo_ptr", C.c_void_p), ("coo_col", C.c_void_p), ("nnz", C.c_int32)]


_LIB = None


def load_library(path: str | Path | None = None):
    """Loads libghd.so (built by ``build.build()``); raises if it is not there."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    p = Path(path) if path else _build.LIB
    if not p.exists():
        raise RuntimeError(f"{p} is missing: build the CUDA library first "
                           "(python -m paper_2505_23219_b200.build); there is no fallback path")
    lib = C.CDLL(str(p))
    vp, i32 = C.c_void_p, C.c_int32
    sig = {
        "ghd_create": ([C.POINTER(_Cfg), vp, C.POINTER(vp)], C.c_int),
        "ghd_destroy": ([vp], None),
        "ghd_workspace_bytes": ([vp], C.c_size_t),
        "ghd_set_workspace": ([vp, vp, C.c_size_t], C.c_int),
        "ghd_set_option": ([vp, i32, i32], C.c_int),
        "ghd_path_count": ([vp, i32], C.c_int64),
        "ghd_tree_build": ([vp, vp, i32, i32, C.POINTER(_Tree)], C.c_int),
        "ghd_tree_from_mask": ([vp, vp, vp, vp, i32, i32, C.POINTER(_Tree)], C.c_int),
        "ghd_verify_layer": ([vp, C.POINTER(_LayerW), C.POINTER(_Kv), C.POINTER(_Tree), vp, vp], C.c_int),
        "ghd_verify_step": ([vp, C.POINTER(_ModelW), C.POINTER(_Kv), C.POINTER(_Tree), vp, vp, vp], C.c_int),
        "ghd_accept": ([vp, C.POINTER(_Tree), vp, vp, vp], C.c_int),
        "ghd_copy_hidden": ([vp, i32, vp], C.c_int),
        "ghd_kv_commit": ([vp, C.POINTER(_Kv), i32, i32, vp], C.c_int),
        "ghd_kv_len_set": ([vp, i32], C.c_int),
        "ghd_kv_len_get": ([vp, C.POINTER(i32)], C.c_int),
        "ghd_medusa_draft": ([vp, C.POINTER(_MedusaW), vp, vp, vp, vp], C.c_int),
        "ghd_tree_fill_tokens": ([vp, vp, vp, vp, vp, i32, vp], C.c_int),
        "ghd_linear": ([vp, vp, vp, i32, i32, i32, vp], C.c_int),
        "ghd_rmsnorm": ([vp, vp, vp, i32, vp], C.c_int),
        "ghd_gate_up": ([vp, vp, vp, i32, vp], C.c_int),
        "ghd_tree_attention": ([vp, vp, C.POINTER(_Kv), C.POINTER(_Tree), vp], C.c_int),
        "ghd_argmax": ([vp, vp, i32, i32, vp], C.c_int),
        "ghd_sync_status": ([vp], C.c_int),
        "ghd_status_str": ([C.c_int], C.c_char_p),
        "ghd_last_error": ([vp], C.c_char_p),
        "ghd_launch_count": ([vp], C.c_int64),
        "ghd_tree_attention_static": ([vp, i32, i32, i32, i32, vp, vp, vp, vp, i32, i32, vp, C.c_char_p, C.c_size_t],
                                      C.c_int),
    }
    for name, (args, res) in sig.items():
        fn = getattr(lib, name)
        fn.argtypes, fn.restype = args, res
    if path is None:
        _LIB = lib
    return lib


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


class ModelCfg:
    def __init__(self, d_model, n_heads, d_head, d_ffn, vocab, n_layers, max_kv_len, max_nodes, dtype,
                 rms_eps=1e-6, rope_theta=10000.0, n_kv_heads=None):
        self.c = _Cfg(d_model, n_heads, n_heads if n_kv_heads is None else n_kv_heads, d_head, d_ffn, vocab,
                      n_layers, max_kv_len, max_nodes, GHD_F32 if dtype in ("f32", GHD_F32) else GHD_F16,
                      rms_eps, rope_theta)

    @property
    def torch_dtype(self):
        return torch.float32 if self.c.dtype == GHD_F32 else torch.float16


class LayerWeights:
    """Device tensors of one layer (kept alive here)."""
    FIELDS = ("wqkv", "wo", "w_gate_up", "w_down", "rms1", "rms2")

    def __init__(self, **tensors):
        self.t = {k: tensors[k] for k in self.FIELDS}
        self.c = _LayerW(*[_ptr(self.t[k]) for k in self.FIELDS])


class ModelWeights:
    def __init__(self, embed, layers, rms_final, lm_head):
        self.embed, self.layers, self.rms_final, self.lm_head = embed, list(layers), rms_final, lm_head
        self._arr = (_LayerW * max(len(self.layers), 1))(*[l.c for l in self.layers])
        self.c = _ModelW(_ptr(embed), self._arr, _ptr(rms_final), _ptr(lm_head))


class MedusaWeights:
    """Drafting heads: w1 [n_heads][d_model][d_model], w2 [n_heads][vocab][d_model] (device tensors)."""

    def __init__(self, w1, w2):
        self.w1, self.w2 = w1, w2
        self.c = _MedusaW(int(w1.shape[0]), _ptr(w1), _ptr(w2))


class KvLayer:
    def __init__(self, k, v, length: int):
        self.k, self.v, self.len = k, v, int(length)

    @property
    def c(self):
        return _Kv(_ptr(self.k), _ptr(self.v), self.len)


class Tree:
    """Device buffers of a built tree plus the struct that describes them."""

    def __init__(self, ctx: "Ctx"):
        n, dev = ctx.cfg.c.max_nodes, ctx.device
        self.mask = torch.zeros(n * 4, dtype=torch.int64, device=dev)
        self.parent = torch.zeros(n, dtype=torch.int32, device=dev)
        self.depth = torch.zeros(n, dtype=torch.int32, device=dev)
        self.pos = torch.zeros(n, dtype=torch.int32, device=dev)
        self.rope = torch.zeros(n * ctx.cfg.c.d_head, dtype=torch.float32, device=dev)
        self.coo_ptr = torch.zeros(n + 1, dtype=torch.int32, device=dev)
        self.coo_col = torch.zeros(n * (n + 1) // 2, dtype=torch.int32, device=dev)
        self.c = _Tree(0, 0, 0, 0, _ptr(self.mask), _ptr(self.parent), _ptr(self.depth), _ptr(self.pos),
                       _ptr(self.rope), _ptr(self.coo_ptr), _ptr(self.coo_col), 0)

    @property
    def n(self):
        return self.c.n

    def coo(self):
        """-> (row pointers int32 [n + 1], visible node ids int32 [nnz]) on the host."""
        n = self.c.n
        ptr = self.coo_ptr[: n + 1].cpu().numpy()
        return ptr, self.coo_col[: int(ptr[n])].cpu().numpy()

    def mask_words(self) -> np.ndarray:
        """mask as uint64 [n][n_words] on the host."""
        n, w = self.c.n, self.c.n_words
        return self.mask[: n * w].cpu().numpy().view(np.uint64).reshape(n, w)


class Ctx:
    def __init__(self, cfg: ModelCfg, device="cuda:0"):
        self.lib = load_library()
        self.cfg = cfg
        self.device = torch.device(device)
        self.handle = C.c_void_p()
        with torch.cuda.device(self.device):
            self.stream = torch.cuda.current_stream(self.device)
            st = self.lib.ghd_create(C.byref(cfg.c), C.c_void_p(self.stream.cuda_stream), C.byref(self.handle))
            if st != 0:
                raise GhdError(st, "ghd_create")
            nbytes = self.lib.ghd_workspace_bytes(self.handle)
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self._check(self.lib.ghd_set_workspace(self.handle, self.workspace.data_ptr(), nbytes))

    def _check(self, st: int):
        if st != 0:
            raise GhdError(st, self.lib.ghd_last_error(self.handle).decode())

    def close(self):
        if self.handle:
            self.lib.ghd_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pack_mask(visible) -> np.ndarray:
    """bool [n][n] visibility matrix -> uint64 [n][ceil(n/64)] words, bit j of row i LSB first."""
    vis = np.asarray(visible, dtype=bool)
    n = vis.shape[0]
    w = (n + 63) // 64
    out = np.zeros((n, w), dtype=np.uint64)
    for i in range(n):
        for j in np.nonzero(vis[i])[0]:
            out[i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
    return out


# ---------------------------------------------------------------- same names as the C-ABI
def ghd_create(cfg: ModelCfg, device="cuda:0") -> Ctx:
    return Ctx(cfg, device)


def ghd_destroy(ctx: Ctx):
    ctx.close()


def ghd_set_option(ctx: Ctx, option: int, value: int):
    ctx._check(ctx.lib.ghd_set_option(ctx.handle, option, value))


def ghd_path_count(ctx: Ctx, path: int) -> int:
    """Launches so far that went to kernel family `path` (PATH_*)."""
    return int(ctx.lib.ghd_path_count(ctx.handle, path))


def ghd_tree_build(ctx: Ctx, parent, kv_len: int, tree: Tree | None = None) -> Tree:
    tree = tree or Tree(ctx)
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    ctx._check(ctx.lib.ghd_tree_build(ctx.handle, parent.ctypes.data if parent.size else None, parent.size, kv_len,
                                      C.byref(tree.c)))
    return tree


def ghd_tree_from_mask(ctx: Ctx, mask_words, kv_len: int, depth=None, parent=None, tree: Tree | None = None) -> Tree:
    tree = tree or Tree(ctx)
    mask_words = np.ascontiguousarray(mask_words, dtype=np.uint64)
    n = mask_words.shape[0]
    depth = None if depth is None else np.ascontiguousarray(depth, dtype=np.int32)
    parent = None if parent is None else np.ascontiguousarray(parent, dtype=np.int32)
    ctx._check(ctx.lib.ghd_tree_from_mask(ctx.handle, mask_words.ctypes.data,
                                          None if depth is None else depth.ctypes.data,
                                          None if parent is None else parent.ctypes.data, n, kv_len, C.byref(tree.c)))
    return tree


def ghd_verify_layer(ctx: Ctx, w: LayerWeights, kv: KvLayer, tree: Tree, x_in, x_out=None):
    x_out = torch.empty_like(x_in) if x_out is None else x_out
    kvc = kv.c
    ctx._check(ctx.lib.ghd_verify_layer(ctx.handle, C.byref(w.c), C.byref(kvc), C.byref(tree.c), x_in.data_ptr(),
                                        x_out.data_ptr()))
    return x_out


def ghd_verify_step(ctx: Ctx, w: ModelWeights, kvs, tree: Tree, tokens, logits=None, argmax=None):
    """-> (logits or None, argmax).  Pass ``logits=False`` to keep the logits in the workspace only."""
    n = tree.c.n
    if logits is None:
        logits = torch.empty((n, ctx.cfg.c.vocab), dtype=torch.float32, device=ctx.device)
    elif logits is False:
        logits = None
    if argmax is None:
        argmax = torch.empty(n, dtype=torch.int32, device=ctx.device)
    arr = (_Kv * max(len(kvs), 1))(*[kv.c for kv in kvs])
    ctx._check(ctx.lib.ghd_verify_step(ctx.handle, C.byref(w.c), arr, C.byref(tree.c), tokens.data_ptr(),
                                       _ptr(logits), argmax.data_ptr()))
    return logits, argmax


def ghd_copy_hidden(ctx: Ctx, n: int, out=None):
    """-> float32 device tensor [n][d_model]: the last layer's output of the last ghd_verify_step (before the final norm)."""
    if out is None:
        out = torch.empty((n, ctx.cfg.c.d_model), dtype=torch.float32, device=ctx.device)
    ctx._check(ctx.lib.ghd_copy_hidden(ctx.handle, n, out.data_ptr()))
    return out


def ghd_accept(ctx: Ctx, tree: Tree, tokens, argmax, out=None):
    """-> int32 device tensor laid out as ghd_accept_result: [n_matched, n_emitted, nodes[256], tokens[256]]."""
    if out is None:
        out = torch.zeros(2 + 2 * GHD_MAX_NODES, dtype=torch.int32, device=ctx.device)
    ctx._check(ctx.lib.ghd_accept(ctx.handle, C.byref(tree.c), tokens.data_ptr(), argmax.data_ptr(), out.data_ptr()))
    return out


def ghd_kv_commit(ctx: Ctx, kvs, kv_len: int, result):
    """Moves the cache rows of the accepted path (device struct `result` from ghd_accept) to slots
    kv_len .. kv_len + n_matched in every layer of `kvs`.  The layers' `len` fields are left alone."""
    arr = (_Kv * len(kvs))(*[kv.c for kv in kvs])
    ctx._check(ctx.lib.ghd_kv_commit(ctx.handle, arr, len(kvs), kv_len, result.data_ptr()))


def ghd_kv_len_set(ctx: Ctx, kv_len: int):
    """Writes the context's device word with the cache length (read by calls given KV_LEN_DEVICE)."""
    ctx._check(ctx.lib.ghd_kv_len_set(ctx.handle, int(kv_len)))


def ghd_kv_len_get(ctx: Ctx) -> int:
    """Waits for the stream and reads the device word back."""
    out = C.c_int32(0)
    ctx._check(ctx.lib.ghd_kv_len_get(ctx.handle, C.byref(out)))
    return int(out.value)


def ghd_medusa_draft(ctx: Ctx, w: MedusaWeights, result, topk, want_logits: bool = False):
    """Candidates of the drafting heads at the last accepted node of `result` (device struct of ghd_accept).
    -> int32 device tensor [n_heads][GHD_MAX_TOPK] (best first, -1 past a head's top-k) (+ float logits [n_heads][vocab])."""
    topk = np.ascontiguousarray(topk, dtype=np.int32)
    k = w.c.n_heads
    cand = torch.empty((k, GHD_MAX_TOPK), dtype=torch.int32, device=ctx.device)
    logits = torch.empty((k, ctx.cfg.c.vocab), dtype=torch.float32, device=ctx.device) if want_logits else None
    ctx._check(ctx.lib.ghd_medusa_draft(ctx.handle, C.byref(w.c), result.data_ptr(), topk.ctypes.data, cand.data_ptr(),
                                        logits.data_ptr() if want_logits else None))
    return (cand, logits) if want_logits else cand


def ghd_tree_fill_tokens(ctx: Ctx, cand, result, level, rank, tokens=None):
    """tokens[0] = bonus token of `result`; tokens[i] = cand[level[i] - 1][rank[i]] (level, rank: int32 device tensors)."""
    n = int(level.numel())
    if tokens is None:
        tokens = torch.empty(n, dtype=torch.int32, device=ctx.device)
    ctx._check(ctx.lib.ghd_tree_fill_tokens(ctx.handle, cand.data_ptr(), result.data_ptr(), level.data_ptr(), rank.data_ptr(), n,
                                            tokens.data_ptr()))
    return tokens


def ghd_linear(ctx: Ctx, x, w, y=None):
    n, k = x.shape
    m = w.shape[0]
    if y is None:
        y = torch.empty((n, m), dtype=torch.float32, device=ctx.device)
    ctx._check(ctx.lib.ghd_linear(ctx.handle, x.data_ptr(), w.data_ptr(), n, k, m, y.data_ptr()))
    return y


def ghd_gate_up(ctx: Ctx, h, w_gate_up, u=None):
    """u [n][d_ffn] = SiLU(h Wg^T) * (h Wu^T) with the layer's own kernel (gate rows first in w_gate_up)."""
    n = h.shape[0]
    if u is None:
        u = torch.empty((n, ctx.cfg.c.d_ffn), dtype=ctx.cfg.torch_dtype, device=ctx.device)
    ctx._check(ctx.lib.ghd_gate_up(ctx.handle, h.data_ptr(), w_gate_up.data_ptr(), n, u.data_ptr()))
    return u


def ghd_rmsnorm(ctx: Ctx, x, g, out=None):
    if out is None:
        out = torch.empty(x.shape, dtype=ctx.cfg.torch_dtype, device=ctx.device)
    ctx._check(ctx.lib.ghd_rmsnorm(ctx.handle, x.data_ptr(), g.data_ptr(), x.shape[0], out.data_ptr()))
    return out


def ghd_tree_attention(ctx: Ctx, q, kv: KvLayer, tree: Tree, out=None):
    out = torch.empty_like(q) if out is None else out
    kvc = kv.c
    ctx._check(ctx.lib.ghd_tree_attention(ctx.handle, q.data_ptr(), C.byref(kvc), C.byref(tree.c), out.data_ptr()))
    return out


def ghd_tree_attention_static(q, k_cache, v_cache, mask_dev, n_heads: int, d_head: int, kv_len: int, out=None):
    """Tree attention without a context or workspace, for callers that may not allocate device
    memory: the split partials live in an array inside the library (limits: 64 nodes,
    n_heads * d_head <= 4096).  Runs on torch's current stream; ``out`` is the caller's."""
    lib = load_library()
    n = q.shape[0]
    out = torch.empty_like(q) if out is None else out
    err = C.create_string_buffer(256)
    st = lib.ghd_tree_attention_static(C.c_void_p(torch.cuda.current_stream().cuda_stream),
                                       GHD_F32 if q.dtype == torch.float32 else GHD_F16, n_heads, d_head,
                                       k_cache.shape[1], q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                       mask_dev.data_ptr(), n, kv_len, out.data_ptr(), err, 256)
    if st != 0:
        raise GhdError(st, err.value.decode())
    return out


def ghd_argmax(ctx: Ctx, logits, out=None):
    n, v = logits.shape
    if out is None:
        out = torch.empty(n, dtype=torch.int32, device=ctx.device)
    ctx._check(ctx.lib.ghd_argmax(ctx.handle, logits.data_ptr(), n, v, out.data_ptr()))
    return out


def ghd_sync_status(ctx: Ctx):
    ctx._check(ctx.lib.ghd_sync_status(ctx.handle))


def ghd_launch_count(ctx: Ctx) -> int:
    return int(ctx.lib.ghd_launch_count(ctx.handle))
