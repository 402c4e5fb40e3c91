"""ctypes wrapper around the fp64 CPU oracle (``goose_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.  The oracle shares no code
with the CUDA path.  ``build()`` compiles the C file with gcc (``-O2 -fopenmp``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "goose_oracle.c")
_LIB = os.path.join(_HERE, "libgoose_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    import hashlib
    src_hash = hashlib.sha256(open(_SRC, "rb").read()).hexdigest()
    hash_file = _LIB + ".srchash"
    if not force and os.path.exists(_LIB) and os.path.exists(hash_file) and open(hash_file).read().strip() == src_hash:
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    with open(hash_file, "w") as f:
        f.write(src_hash + "\n")
    return _LIB


def _ptr(a: Optional[np.ndarray], ct):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ct))
    return a.ctypes.data_as(ctypes.POINTER(ct))


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
        for name in ("oracle_tree_attn", "oracle_tree_attn_rows", "oracle_tree_attn_gqa", "oracle_tree_attn_rows_gqa",
                     "oracle_node_topk", "oracle_accept",
                     "oracle_kv_compact", "oracle_check_parent", "oracle_harvest", "oracle_ancestors", "oracle_tree_attn_n",
                     "oracle_node_topk_n", "oracle_accept_n", "oracle_kv_compact_n"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _c(a, dt) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def _nn(n_nodes, S):
    """n_nodes [S] int32 or None (every sequence has all B nodes)."""
    return None if n_nodes is None else _c(n_nodes, np.int32).reshape(S)


def tree_attn(q, k_cache, v_cache, row_off, ctx_len, parent, scale: float, want_lse: bool = True, n_nodes=None
              ) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """q uint16 [S][B][H][D]; caches uint16 [rows][Hkv][D] (Hkv == H: multi-head attention; Hkv a divisor of H:
    grouped-query attention, query head h reads key/value head h // (H // Hkv)).
    n_nodes [S] (optional): nodes i >= n_nodes[s] do not exist; their output rows stay zero.
    Returns out fp64 [S][B][H][D], lse [S][B][H]."""
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    S, B, H, D = q.shape
    Hkv = k_cache.shape[1]
    if v_cache.shape != k_cache.shape or k_cache.shape[2] != D or Hkv < 1 or H % Hkv != 0:
        raise ValueError("cache shape %r does not fit q shape %r" % (k_cache.shape, q.shape))
    row_off = _c(row_off, np.int64).reshape(S); ctx_len = _c(ctx_len, np.int32).reshape(S)
    parent = _c(parent, np.int32).reshape(S, B)
    out = np.zeros((S, B, H, D), dtype=np.float64)
    lse = np.zeros((S, B, H), dtype=np.float64) if want_lse else None
    nn = _nn(n_nodes, S)
    rc = lib().oracle_tree_attn_n(_ptr(q, ctypes.c_uint16), _ptr(k_cache, ctypes.c_uint16), _ptr(v_cache, ctypes.c_uint16),
                                  _ptr(row_off, ctypes.c_int64), _ptr(ctx_len, ctypes.c_int32), _ptr(parent, ctypes.c_int32),
                                  _ptr(nn, ctypes.c_int32), ctypes.c_int(S), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(Hkv),
                                  ctypes.c_int(D), ctypes.c_double(scale), _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_tree_attn failed: rc=%d (invalid parent[]?)" % rc)
    return out, lse


def tree_attn_rows(q, k_cache, v_cache, row_off, ctx_len, parent, scale: float, ss, si, sh
                   ) -> Tuple[np.ndarray, np.ndarray]:
    """Same as :func:`tree_attn` for sampled (sequence, node, query head) rows only."""
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    S, B, H, D = q.shape
    Hkv = k_cache.shape[1]
    if v_cache.shape != k_cache.shape or k_cache.shape[2] != D or Hkv < 1 or H % Hkv != 0:
        raise ValueError("cache shape %r does not fit q shape %r" % (k_cache.shape, q.shape))
    row_off = _c(row_off, np.int64).reshape(S); ctx_len = _c(ctx_len, np.int32).reshape(S)
    parent = _c(parent, np.int32).reshape(S, B)
    ss = _c(ss, np.int32); si = _c(si, np.int32); sh = _c(sh, np.int32)
    n = len(ss)
    out = np.zeros((n, D), dtype=np.float64)
    lse = np.zeros((n,), dtype=np.float64)
    rc = lib().oracle_tree_attn_rows_gqa(_ptr(q, ctypes.c_uint16), _ptr(k_cache, ctypes.c_uint16), _ptr(v_cache, ctypes.c_uint16),
                                     _ptr(row_off, ctypes.c_int64), _ptr(ctx_len, ctypes.c_int32), _ptr(parent, ctypes.c_int32),
                                     ctypes.c_int(S), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D),
                                     ctypes.c_double(scale), ctypes.c_int(n), _ptr(ss, ctypes.c_int32),
                                     _ptr(si, ctypes.c_int32), _ptr(sh, ctypes.c_int32),
                                     _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_tree_attn_rows failed: rc=%d" % rc)
    return out, lse


def node_topk(logits, k: int, V: Optional[int] = None, n_nodes=None, B: int = 0
              ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """logits uint16 [rows][ldl] (first V columns used).  Returns argmax [rows], ids [rows][k], vals fp64 [rows][k].
    n_nodes [rows / B] with B (optional): rows of nodes that do not exist are skipped and stay zero."""
    logits = _c(logits, np.uint16)
    rows, ldl = logits.shape
    V = ldl if V is None else V
    argmax = np.zeros(rows, dtype=np.int32)
    ids = np.zeros((rows, k), dtype=np.int32)
    vals = np.zeros((rows, k), dtype=np.float64)
    nn = None if n_nodes is None else _nn(n_nodes, rows // B)
    rc = lib().oracle_node_topk_n(_ptr(logits, ctypes.c_uint16), ctypes.c_int(rows), ctypes.c_int(V),
                                  ctypes.c_int64(ldl), ctypes.c_int(k), _ptr(nn, ctypes.c_int32), ctypes.c_int(B),
                                  _ptr(argmax, ctypes.c_int32), _ptr(ids, ctypes.c_int32), _ptr(vals, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_node_topk failed: rc=%d" % rc)
    return argmax, ids, vals


def accept(draft_tok, parent, argmax, tag=None, n_nodes=None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Algorithm 3 walk.  Arrays [S][B].  Returns path [S][B], accept_len [S], bonus [S].  n_nodes [S] (optional)."""
    parent = _c(parent, np.int32)
    if parent.ndim == 1:
        parent = parent[None]
    S, B = parent.shape
    draft_tok = _c(draft_tok, np.int32).reshape(S, B)
    argmax = _c(argmax, np.int32).reshape(S, B)
    tag_a = None if tag is None else _c(np.asarray(tag).astype(np.uint8), np.uint8).reshape(S, B)
    path = np.zeros((S, B), dtype=np.int32)
    alen = np.zeros(S, dtype=np.int32)
    bonus = np.zeros(S, dtype=np.int32)
    rc = lib().oracle_accept_n(_ptr(draft_tok, ctypes.c_int32), _ptr(parent, ctypes.c_int32), _ptr(argmax, ctypes.c_int32),
                               _ptr(tag_a, ctypes.c_uint8), _ptr(_nn(n_nodes, S), ctypes.c_int32), ctypes.c_int(S), ctypes.c_int(B),
                               _ptr(path, ctypes.c_int32), _ptr(alen, ctypes.c_int32), _ptr(bonus, ctypes.c_int32))
    if rc != 0:
        raise ValueError("oracle_accept failed: rc=%d (invalid parent[]?)" % rc)
    return path, alen, bonus


def kv_compact(k_cache, v_cache, row_off, ctx_len, path, accept_len, n_nodes=None
               ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Out-of-place compaction.  Returns (k_out, v_out, new_ctx).  n_nodes [S] (optional): 0 = the sequence has left."""
    k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    rows, H, D = k_cache.shape
    path = _c(path, np.int32)
    if path.ndim == 1:
        path = path[None]
    S, B = path.shape
    row_off = _c(row_off, np.int64).reshape(S); ctx_len = _c(ctx_len, np.int32).reshape(S)
    accept_len = _c(accept_len, np.int32).reshape(S)
    k_out = k_cache.copy(); v_out = v_cache.copy()
    new_ctx = np.zeros(S, dtype=np.int32)
    rc = lib().oracle_kv_compact_n(_ptr(k_cache, ctypes.c_uint16), _ptr(v_cache, ctypes.c_uint16),
                                 _ptr(row_off, ctypes.c_int64), _ptr(ctx_len, ctypes.c_int32),
                                 _ptr(path, ctypes.c_int32), _ptr(accept_len, ctypes.c_int32), _ptr(_nn(n_nodes, S), ctypes.c_int32),
                                 ctypes.c_int(S), ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(D),
                                 _ptr(k_out, ctypes.c_uint16), _ptr(v_out, ctypes.c_uint16), _ptr(new_ctx, ctypes.c_int32))
    if rc != 0:
        raise ValueError("oracle_kv_compact failed: rc=%d" % rc)
    return k_out, v_out, new_ctx


def ancestors(parent) -> list:
    """Ancestor sets A(i) (Sec. 4 Stage 1: root-to-node path, node included) of every node as bitmasks, bit j = node j."""
    parent = _c(parent, np.int32).reshape(-1)
    B = len(parent)
    masks = []
    for i in range(B):
        vis = np.zeros(B, dtype=np.uint8)
        rc = lib().oracle_ancestors(_ptr(parent, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(i), _ptr(vis, ctypes.c_uint8))
        if rc != 0:
            raise ValueError("oracle_ancestors failed: rc=%d (invalid parent[]?)" % rc)
        masks.append(sum(1 << j for j in range(B) if vis[j]))
    return masks


def check_parent(parent) -> bool:
    parent = _c(parent, np.int32).reshape(-1)
    return lib().oracle_check_parent(_ptr(parent, ctypes.c_int32), ctypes.c_int(len(parent))) == 0


def harvest(logits, k: int, row_tok, adj_ids: np.ndarray, adj_scores: np.ndarray, V: Optional[int] = None
            ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Harvest every logits row into the Tier-1 adjacency table (ids int32 [table_rows][k], scores fp64
    [table_rows][k], both updated on copies).  Returns (adj_ids, adj_scores, row_lse)."""
    logits = _c(logits, np.uint16)
    rows, ldl = logits.shape
    V = ldl if V is None else V
    row_tok = _c(row_tok, np.int32).reshape(rows)
    ids = np.ascontiguousarray(adj_ids, dtype=np.int32).copy()
    sc = np.ascontiguousarray(adj_scores, dtype=np.float64).copy()
    lse = np.zeros(rows, dtype=np.float64)
    rc = lib().oracle_harvest(_ptr(logits, ctypes.c_uint16), ctypes.c_int(rows), ctypes.c_int(V), ctypes.c_int64(ldl),
                              ctypes.c_int(k), _ptr(row_tok, ctypes.c_int32), ctypes.c_int(ids.shape[0]),
                              _ptr(ids, ctypes.c_int32), _ptr(sc, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_harvest failed: rc=%d" % rc)
    return ids, sc, lse
