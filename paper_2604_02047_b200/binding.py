"""Thin Python binding of the C ABI in ``include/goose.h`` (argument marshalling only).

Every function takes torch CUDA tensors (or, for the ``*_host`` call, pinned CPU tensors),
passes their ``data_ptr()`` and the current CUDA stream to ``libgoose.so`` and returns the
output tensors.  No step of the method runs in Python or in torch ops; if the library is
missing or a call fails, an exception is raised -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgoose.so")

EXPORTS = [
    "goose_create", "goose_destroy", "goose_strerror", "goose_set_attn_impl", "goose_tree_attn",
    "goose_node_topk", "goose_accept", "goose_kv_compact", "goose_verify_step",
    "goose_verify_step_host", "goose_last_status", "goose_launch_count", "goose_node_topk_static", "goose_harvest",
    "goose_build_spine_tree", "goose_pad_tree", "goose_context_match", "goose_spine_ratio_tier", "goose_spine_ema",
    "goose_selftest_bounded_wait", "goose_tree_attn_gqa", "goose_verify_step_gqa", "goose_verify_step_host_gqa",
    "goose_verify_step_harvest",
]

ATTN_AUTO, ATTN_MMA, ATTN_UMMA = 0, 1, 2
ST_BAD_PARENT, ST_BAD_PATH, ST_TIMEOUT, ST_BAD_ROWS, ST_BAD_NODES = 1, 2, 4, 8, 16

_lib: Optional[ctypes.CDLL] = None


class GooseError(RuntimeError):
    pass


def load_library() -> ctypes.CDLL:
    """Load ``libgoose.so`` (built in-tree by :mod:`paper_2604_02047_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise GooseError("libgoose.so is missing at %s: run `python -m paper_2604_02047_b200.build` "
                         "(there is no fallback path)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    lib.goose_strerror.restype = ctypes.c_char_p
    lib.goose_strerror.argtypes = [ctypes.c_int]
    lib.goose_launch_count.restype = ctypes.c_int64
    lib.goose_launch_count.argtypes = [ctypes.c_void_p]
    for name in EXPORTS:
        if name not in ("goose_strerror", "goose_launch_count", "goose_spine_ratio_tier", "goose_spine_ema"):
            getattr(lib, name).restype = ctypes.c_int
    lib.goose_spine_ratio_tier.restype = ctypes.c_float
    lib.goose_spine_ratio_tier.argtypes = [ctypes.c_float]
    lib.goose_spine_ema.restype = ctypes.c_float
    lib.goose_spine_ema.argtypes = [ctypes.c_float, ctypes.c_int, ctypes.c_int]
    _lib = lib
    return lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        msg = load_library().goose_strerror(rc).decode()
        raise GooseError("%s failed: %s (rc=%d)" % (what, msg, rc))


def _p(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, dtype: torch.dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise GooseError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))
    return t


def _nn(n_nodes: Optional[torch.Tensor], S: int) -> Optional[torch.Tensor]:
    """Per-sequence node counts: a contiguous int32 CUDA tensor [S], or None (every tree has all B nodes)."""
    if n_nodes is None:
        return None
    _dev(n_nodes, torch.int32, "n_nodes")
    if n_nodes.numel() != S:
        raise GooseError("n_nodes must have one entry per sequence")
    return n_nodes


def _host_nn(h_n_nodes: Optional[torch.Tensor], S: int) -> Optional[torch.Tensor]:
    if h_n_nodes is None:
        return None
    if h_n_nodes.is_cuda or h_n_nodes.dtype != torch.int32 or not h_n_nodes.is_contiguous() or h_n_nodes.numel() != S:
        raise GooseError("h_n_nodes must be a contiguous int32 host tensor [S]")
    return h_n_nodes


def _kv_heads(k_cache: torch.Tensor, v_cache: torch.Tensor) -> int:
    if k_cache.dim() != 3 or tuple(k_cache.shape) != tuple(v_cache.shape):
        raise GooseError("k_cache and v_cache must both be [rows][Hkv][D]")
    return int(k_cache.shape[1])


def _same_heads(k_cache: torch.Tensor, v_cache: torch.Tensor, H: int, what: str) -> None:
    if _kv_heads(k_cache, v_cache) != H:
        raise GooseError("%s: the caches have %d heads, q has %d (grouped-query attention: use %s_gqa)"
                         % (what, k_cache.shape[1], H, what))


class Goose:
    """A context (workspace) on one CUDA device plus the calls of the verification step."""

    def __init__(self, max_S: int = 16, max_B: int = 128, max_H: int = 64, device: int = 0,
                 attn_impl: int = ATTN_AUTO):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise GooseError("no CUDA device: the tree-verification step only runs on the GPU")
        h = ctypes.c_void_p()
        _check(self.lib.goose_create(ctypes.byref(h), ctypes.c_int(device), ctypes.c_int(max_S),
                                     ctypes.c_int(max_B), ctypes.c_int(max_H), ctypes.c_int(128)), "goose_create")
        self.h = h
        self.device = torch.device("cuda", device)
        self.max_S, self.max_B, self.max_H = max_S, max_B, max_H
        if attn_impl != ATTN_AUTO:
            self.set_attn_impl(attn_impl)

    def close(self) -> None:
        if getattr(self, "h", None):
            torch.cuda.synchronize(self.device)
            self.lib.goose_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_attn_impl(self, impl: int) -> None:
        _check(self.lib.goose_set_attn_impl(self.h, ctypes.c_int(impl)), "goose_set_attn_impl")

    def launch_count(self) -> int:
        return int(self.lib.goose_launch_count(self.h))

    def selftest_bounded_wait(self, limit_cycles: int = 1_000_000) -> int:
        """Run the time-out self-test; returns the library's return code (0 = the wait gave up as designed)."""
        return int(self.lib.goose_selftest_bounded_wait(self.h, ctypes.c_int64(limit_cycles), _stream()))

    def last_status(self, S: int) -> torch.Tensor:
        st = torch.zeros(S, dtype=torch.int32)
        rc = self.lib.goose_last_status(self.h, _p(st), ctypes.c_int(S))
        if rc not in (0, -4):
            _check(rc, "goose_last_status")
        return st

    # ------------------------------------------------------------------ the four calls
    def tree_attn(self, q, k_cache, v_cache, row_off, ctx_len, parent, scale: float,
                  out: Optional[torch.Tensor] = None, want_lse: bool = False,
                  lse: Optional[torch.Tensor] = None, n_nodes: Optional[torch.Tensor] = None
                  ) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
        _dev(q, torch.bfloat16, "q"); _dev(k_cache, torch.bfloat16, "k_cache"); _dev(v_cache, torch.bfloat16, "v_cache")
        _dev(row_off, torch.int64, "row_off"); _dev(ctx_len, torch.int32, "ctx_len"); _dev(parent, torch.int32, "parent")
        S, B, H, D = q.shape
        _same_heads(k_cache, v_cache, H, "tree_attn")
        if out is None:
            out = torch.empty_like(q)
        if want_lse and lse is None:
            lse = torch.empty((S, B, H), dtype=torch.float32, device=q.device)
        _check(self.lib.goose_tree_attn(self.h, _p(q), _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]),
                                        _p(row_off), _p(ctx_len), _p(parent), _p(_nn(n_nodes, S)), ctypes.c_int(S), ctypes.c_int(B),
                                        ctypes.c_int(H), ctypes.c_int(D), ctypes.c_float(scale), _p(out), _p(lse),
                                        _stream()), "goose_tree_attn")
        return out, lse

    def tree_attn_gqa(self, q, k_cache, v_cache, row_off, ctx_len, parent, scale: float,
                      out: Optional[torch.Tensor] = None, want_lse: bool = False,
                      lse: Optional[torch.Tensor] = None, n_nodes: Optional[torch.Tensor] = None
                      ) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
        """Grouped-query attention: q [S][B][H][D], caches [rows][Hkv][D]; Hkv is read from the caches' shape."""
        _dev(q, torch.bfloat16, "q"); _dev(k_cache, torch.bfloat16, "k_cache"); _dev(v_cache, torch.bfloat16, "v_cache")
        _dev(row_off, torch.int64, "row_off"); _dev(ctx_len, torch.int32, "ctx_len"); _dev(parent, torch.int32, "parent")
        S, B, H, D = q.shape
        Hkv = _kv_heads(k_cache, v_cache)
        if out is None:
            out = torch.empty_like(q)
        if want_lse and lse is None:
            lse = torch.empty((S, B, H), dtype=torch.float32, device=q.device)
        _check(self.lib.goose_tree_attn_gqa(self.h, _p(q), _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]),
                                            _p(row_off), _p(ctx_len), _p(parent), _p(_nn(n_nodes, S)), ctypes.c_int(S), ctypes.c_int(B),
                                            ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_float(scale),
                                            _p(out), _p(lse), _stream()), "goose_tree_attn_gqa")
        return out, lse

    def node_topk(self, logits, k: int, V: Optional[int] = None, want_vals: bool = True,
                  n_nodes: Optional[torch.Tensor] = None, B: int = 0, outs=None):
        """``n_nodes`` [rows / B] with ``B``: rows of nodes that do not exist are skipped (not read, outputs untouched;
        pass ``outs`` = (argmax, ids, vals) to see what they held before)."""
        _dev(logits, torch.bfloat16, "logits")
        rows, ldl = logits.shape
        V = ldl if V is None else V
        if outs is not None:
            argmax, ids, vals = outs
        else:
            argmax = torch.empty(rows, dtype=torch.int32, device=logits.device)
            ids = torch.empty((rows, k), dtype=torch.int32, device=logits.device)
            vals = torch.empty((rows, k), dtype=torch.float32, device=logits.device) if want_vals else None
        nn = None if n_nodes is None else _nn(n_nodes, rows // max(B, 1))
        _check(self.lib.goose_node_topk(self.h, _p(logits), ctypes.c_int(rows), ctypes.c_int(V), ctypes.c_int64(ldl),
                                        ctypes.c_int(k), _p(nn), ctypes.c_int(B), _p(argmax), _p(ids), _p(vals), _stream()),
               "goose_node_topk")
        return argmax, ids, vals

    def harvest(self, logits, k: int, row_tok, adj_ids, adj_scores, V: Optional[int] = None):
        """Top-k + log-sum-exp of every row, then scatter into the adjacency table (updated in place)."""
        _dev(logits, torch.bfloat16, "logits"); _dev(row_tok, torch.int32, "row_tok")
        _dev(adj_ids, torch.int32, "adj_ids"); _dev(adj_scores, torch.float32, "adj_scores")
        rows, ldl = logits.shape
        V = ldl if V is None else V
        dev = logits.device
        argmax = torch.empty(rows, dtype=torch.int32, device=dev)
        ids = torch.empty((rows, k), dtype=torch.int32, device=dev)
        vals = torch.empty((rows, k), dtype=torch.float32, device=dev)
        lse = torch.empty(rows, dtype=torch.float32, device=dev)
        _check(self.lib.goose_harvest(self.h, _p(logits), ctypes.c_int(rows), ctypes.c_int(V), ctypes.c_int64(ldl),
                                      ctypes.c_int(k), _p(row_tok), ctypes.c_int(adj_ids.shape[0]), _p(adj_ids),
                                      _p(adj_scores), _p(argmax), _p(ids), _p(vals), _p(lse), _stream()),
               "goose_harvest")
        return argmax, ids, vals, lse

    def accept(self, draft_tok, parent, argmax, n_nodes: Optional[torch.Tensor] = None):
        _dev(draft_tok, torch.int32, "draft_tok"); _dev(parent, torch.int32, "parent"); _dev(argmax, torch.int32, "argmax")
        S, B = parent.shape
        path = torch.empty((S, B), dtype=torch.int32, device=parent.device)
        alen = torch.empty(S, dtype=torch.int32, device=parent.device)
        bonus = torch.empty(S, dtype=torch.int32, device=parent.device)
        _check(self.lib.goose_accept(self.h, _p(draft_tok), _p(parent), _p(_nn(n_nodes, S)), _p(argmax), ctypes.c_int(S), ctypes.c_int(B),
                                     _p(path), _p(alen), _p(bonus), _stream()), "goose_accept")
        return path, alen, bonus

    def kv_compact(self, k_cache, v_cache, row_off, ctx_len, path, accept_len, n_nodes: Optional[torch.Tensor] = None):
        _dev(k_cache, torch.bfloat16, "k_cache"); _dev(v_cache, torch.bfloat16, "v_cache")
        _dev(path, torch.int32, "path"); _dev(accept_len, torch.int32, "accept_len")
        rows, H, D = k_cache.shape
        S, B = path.shape
        new_ctx = torch.empty(S, dtype=torch.int32, device=path.device)
        _check(self.lib.goose_kv_compact(self.h, _p(k_cache), _p(v_cache), ctypes.c_int64(rows), _p(row_off),
                                         _p(ctx_len), _p(path), _p(accept_len), _p(_nn(n_nodes, S)), ctypes.c_int(S), ctypes.c_int(B),
                                         ctypes.c_int(H), ctypes.c_int(D), _p(new_ctx), _stream()), "goose_kv_compact")
        return new_ctx

    # ------------------------------------------------------------------ whole step
    def alloc_step_outputs(self, S: int, B: int, H: int, D: int, k: int, device=None) -> dict:
        dev = self.device if device is None else device
        return dict(
            out=torch.empty((S, B, H, D), dtype=torch.bfloat16, device=dev),
            argmax=torch.empty(S * B, dtype=torch.int32, device=dev),
            topk_ids=torch.empty((S * B, k), dtype=torch.int32, device=dev),
            topk_vals=torch.empty((S * B, k), dtype=torch.float32, device=dev),
            path=torch.empty((S, B), dtype=torch.int32, device=dev),
            accept_len=torch.empty(S, dtype=torch.int32, device=dev),
            bonus=torch.empty(S, dtype=torch.int32, device=dev),
            new_ctx_len=torch.empty(S, dtype=torch.int32, device=dev),
        )

    def verify_step(self, q, k_cache, v_cache, row_off, ctx_len, parent, draft_tok, logits, k: int, scale: float,
                    outs: Optional[dict] = None, V: Optional[int] = None, n_nodes: Optional[torch.Tensor] = None) -> dict:
        S, B, H, D = q.shape
        _same_heads(k_cache, v_cache, H, "verify_step")
        ldl = logits.shape[1]
        V = ldl if V is None else V
        if outs is None:
            outs = self.alloc_step_outputs(S, B, H, D, k, q.device)
        _check(self.lib.goose_verify_step(
            self.h, _p(q), _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]), _p(row_off), _p(ctx_len),
            _p(parent), _p(_nn(n_nodes, S)), _p(draft_tok), _p(logits), ctypes.c_int64(ldl), ctypes.c_int(S), ctypes.c_int(B),
            ctypes.c_int(H), ctypes.c_int(D), ctypes.c_int(V), ctypes.c_int(k), ctypes.c_float(scale),
            _p(outs["out"]), _p(outs.get("lse")), _p(outs["argmax"]), _p(outs["topk_ids"]), _p(outs["topk_vals"]),
            _p(outs["path"]), _p(outs["accept_len"]), _p(outs["bonus"]), _p(outs["new_ctx_len"]), _stream()),
            "goose_verify_step")
        return outs

    def verify_step_gqa(self, q, k_cache, v_cache, row_off, ctx_len, parent, draft_tok, logits, k: int, scale: float,
                        outs: Optional[dict] = None, V: Optional[int] = None, n_nodes: Optional[torch.Tensor] = None) -> dict:
        """The whole step with grouped-query attention (Hkv is read from the caches' shape)."""
        S, B, H, D = q.shape
        Hkv = _kv_heads(k_cache, v_cache)
        ldl = logits.shape[1]
        V = ldl if V is None else V
        if outs is None:
            outs = self.alloc_step_outputs(S, B, H, D, k, q.device)
        _check(self.lib.goose_verify_step_gqa(
            self.h, _p(q), _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]), _p(row_off), _p(ctx_len),
            _p(parent), _p(_nn(n_nodes, S)), _p(draft_tok), _p(logits), ctypes.c_int64(ldl), ctypes.c_int(S), ctypes.c_int(B),
            ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(V), ctypes.c_int(k), ctypes.c_float(scale),
            _p(outs["out"]), _p(outs.get("lse")), _p(outs["argmax"]), _p(outs["topk_ids"]), _p(outs["topk_vals"]),
            _p(outs["path"]), _p(outs["accept_len"]), _p(outs["bonus"]), _p(outs["new_ctx_len"]), _stream()),
            "goose_verify_step_gqa")
        return outs

    def verify_step_harvest(self, q, k_cache, v_cache, row_off, ctx_len, parent, draft_tok, logits, k: int, scale: float,
                            adj_ids, adj_scores, outs: Optional[dict] = None, V: Optional[int] = None,
                            n_nodes: Optional[torch.Tensor] = None) -> dict:
        """The whole step plus the harvest of its logits into the adjacency table (updated in place); multi-head or
        grouped-query (Hkv is read from the caches' shape).  ``outs`` gains ``row_lse`` [S*B]."""
        S, B, H, D = q.shape
        Hkv = _kv_heads(k_cache, v_cache)
        _dev(adj_ids, torch.int32, "adj_ids"); _dev(adj_scores, torch.float32, "adj_scores")
        ldl = logits.shape[1]
        V = ldl if V is None else V
        if outs is None:
            outs = self.alloc_step_outputs(S, B, H, D, k, q.device)
        if "row_lse" not in outs:
            outs["row_lse"] = torch.empty(S * B, dtype=torch.float32, device=q.device)
        _check(self.lib.goose_verify_step_harvest(
            self.h, _p(q), _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]), _p(row_off), _p(ctx_len),
            _p(parent), _p(_nn(n_nodes, S)), _p(draft_tok), _p(logits), ctypes.c_int64(ldl), ctypes.c_int(S), ctypes.c_int(B),
            ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(V), ctypes.c_int(k), ctypes.c_float(scale),
            _p(outs["out"]), _p(outs.get("lse")), _p(outs["argmax"]), _p(outs["topk_ids"]), _p(outs["topk_vals"]),
            _p(outs["path"]), _p(outs["accept_len"]), _p(outs["bonus"]), _p(outs["new_ctx_len"]), _p(outs["row_lse"]),
            ctypes.c_int(adj_ids.shape[0]), _p(adj_ids), _p(adj_scores), _stream()), "goose_verify_step_harvest")
        return outs

    def verify_step_host_gqa(self, k_cache, v_cache, h_q, h_k_new, h_v_new, h_row_off, h_ctx_len, h_parent,
                             h_draft_tok, h_logits, k: int, scale: float, h_outs: dict,
                             h_n_nodes: Optional[torch.Tensor] = None) -> dict:
        """End-to-end call with grouped-query attention: h_k_new / h_v_new are [S][B][Hkv][D]."""
        S, B, H, D = h_q.shape
        Hkv = _kv_heads(k_cache, v_cache)
        V = h_logits.shape[1]
        for t in (h_q, h_k_new, h_v_new, h_row_off, h_ctx_len, h_parent, h_draft_tok, h_logits, *h_outs.values()):
            if t.is_cuda or not t.is_contiguous():
                raise GooseError("verify_step_host_gqa takes contiguous host tensors")
        if tuple(h_k_new.shape) != (S, B, Hkv, D) or tuple(h_v_new.shape) != (S, B, Hkv, D):
            raise GooseError("h_k_new / h_v_new must be [S][B][Hkv][D]")
        _check(self.lib.goose_verify_step_host_gqa(
            self.h, _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]), _p(h_q), _p(h_k_new), _p(h_v_new),
            _p(h_row_off), _p(h_ctx_len), _p(h_parent), _p(_host_nn(h_n_nodes, S)), _p(h_draft_tok), _p(h_logits), ctypes.c_int(S),
            ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_int(V), ctypes.c_int(k),
            ctypes.c_float(scale), _p(h_outs["out"]), _p(h_outs["argmax"]), _p(h_outs["topk_ids"]),
            _p(h_outs["topk_vals"]), _p(h_outs["path"]), _p(h_outs["accept_len"]), _p(h_outs["bonus"]),
            _p(h_outs["new_ctx_len"]), _stream()), "goose_verify_step_host_gqa")
        return h_outs

    def verify_step_host(self, k_cache, v_cache, h_q, h_k_new, h_v_new, h_row_off, h_ctx_len, h_parent,
                         h_draft_tok, h_logits, k: int, scale: float, h_outs: dict,
                         h_n_nodes: Optional[torch.Tensor] = None) -> dict:
        """End-to-end call: per-step inputs and outputs are (pinned) host tensors; the prefix KV cache
        is device state.  Synchronises the current stream before returning."""
        S, B, H, D = h_q.shape
        _same_heads(k_cache, v_cache, H, "verify_step_host")
        V = h_logits.shape[1]
        for t in (h_q, h_k_new, h_v_new, h_row_off, h_ctx_len, h_parent, h_draft_tok, h_logits, *h_outs.values()):
            if t.is_cuda or not t.is_contiguous():
                raise GooseError("verify_step_host takes contiguous host tensors")
        _check(self.lib.goose_verify_step_host(
            self.h, _p(k_cache), _p(v_cache), ctypes.c_int64(k_cache.shape[0]), _p(h_q), _p(h_k_new), _p(h_v_new),
            _p(h_row_off), _p(h_ctx_len), _p(h_parent), _p(_host_nn(h_n_nodes, S)), _p(h_draft_tok), _p(h_logits), ctypes.c_int(S),
            ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(D), ctypes.c_int(V), ctypes.c_int(k),
            ctypes.c_float(scale), _p(h_outs["out"]), _p(h_outs["argmax"]), _p(h_outs["topk_ids"]),
            _p(h_outs["topk_vals"]), _p(h_outs["path"]), _p(h_outs["accept_len"]), _p(h_outs["bonus"]),
            _p(h_outs["new_ctx_len"]), _stream()), "goose_verify_step_host")
        return h_outs


def node_topk_static(logits: torch.Tensor, k: int, V: Optional[int] = None, want_vals: bool = True):
    """``goose_node_topk_static``: top-k without a context and without any device allocation inside the
    library (the output tensors are the caller's, allocated here by torch before the call)."""
    lib = load_library()
    _dev(logits, torch.bfloat16, "logits")
    rows, ldl = logits.shape
    V = ldl if V is None else V
    argmax = torch.empty(rows, dtype=torch.int32, device=logits.device)
    ids = torch.empty((rows, k), dtype=torch.int32, device=logits.device)
    vals = torch.empty((rows, k), dtype=torch.float32, device=logits.device) if want_vals else None
    with torch.cuda.device(logits.device):
        _check(lib.goose_node_topk_static(_p(logits), ctypes.c_int(rows), ctypes.c_int(V), ctypes.c_int64(ldl),
                                          ctypes.c_int(k), _p(argmax), _p(ids), _p(vals), _stream()),
               "goose_node_topk_static")
    return argmax, ids, vals


# ---------------------------------------------------------------------- host routines (numpy in, numpy out)
def build_spine_tree(anchor: int, chain, adj_ids, B: int, D: int, r: float, rho: float, pad: bool = False):
    """``goose_build_spine_tree`` (+ ``goose_pad_tree``).  adj_ids: int32 numpy [table_rows][K] on the host.
    Returns (draft_tok, parent, is_spine, n_nodes, n_spine); arrays have length B when ``pad`` else n_nodes."""
    import numpy as np
    lib = load_library()
    chain = np.ascontiguousarray(chain, dtype=np.int32)
    adj_ids = np.ascontiguousarray(adj_ids, dtype=np.int32)
    tok = np.zeros(B, np.int32); par = np.zeros(B, np.int32); sp = np.zeros(B, np.uint8)
    n = ctypes.c_int32(); ns = ctypes.c_int32()
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib.goose_build_spine_tree(ctypes.c_int32(anchor), vp(chain), ctypes.c_int(len(chain)), vp(adj_ids),
                                      ctypes.c_int(adj_ids.shape[0]), ctypes.c_int(adj_ids.shape[1]), ctypes.c_int(B),
                                      ctypes.c_int(D), ctypes.c_float(r), ctypes.c_float(rho), vp(tok), vp(par), vp(sp),
                                      ctypes.byref(n), ctypes.byref(ns)), "goose_build_spine_tree")
    if pad:
        _check(lib.goose_pad_tree(vp(tok), vp(par), n, ctypes.c_int(B)), "goose_pad_tree")
        return tok, par, sp.astype(bool), n.value, ns.value
    return tok[:n.value], par[:n.value], sp[:n.value].astype(bool), n.value, ns.value


def context_match(ctx, max_len: int = 20):
    """``goose_context_match``: returns (chain, consensus)."""
    import numpy as np
    lib = load_library()
    ctx = np.ascontiguousarray(ctx, dtype=np.int32)
    chain = np.zeros(max(1, max_len), np.int32)
    n = ctypes.c_int32(); c = ctypes.c_int32()
    vp = lambda a: a.ctypes.data_as(ctypes.c_void_p)
    _check(lib.goose_context_match(vp(ctx), ctypes.c_int(len(ctx)), ctypes.c_int(max_len), vp(chain), ctypes.byref(n),
                                   ctypes.byref(c)), "goose_context_match")
    return chain[:n.value].tolist(), bool(c.value)


# ---------------------------------------------------------------------- helpers for tests / bench
def to_device(x, device="cuda") -> dict:
    """Upload a ``synth.VerifyInputs`` (numpy, bf16 as uint16 bits) as torch tensors."""
    import numpy as np

    def bf(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)

    return dict(
        q=bf(x.q), k_cache=bf(x.k_cache), v_cache=bf(x.v_cache), logits=bf(x.logits),
        row_off=torch.from_numpy(x.row_off).to(device), ctx_len=torch.from_numpy(x.ctx_len).to(device),
        parent=torch.from_numpy(x.parent).to(device), draft_tok=torch.from_numpy(x.draft_tok).to(device),
    )


def bf16_to_bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
