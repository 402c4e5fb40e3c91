"""Seeded synthetic workloads for the Goose tree-verification step.

This module only *draws inputs*: spine trees, draft tokens, logits with planted
acceptances, and Q/K/V tensors.  It holds none of the method's arithmetic (no
attention, no top-k, no acceptance walk, no compaction), so both the CPU oracle's
tests and the CUDA path's tests/bench may import it without sharing any code of
the method itself.

Tensors are returned as numpy arrays.  bf16 values are carried as ``uint16`` bit
patterns so that every consumer reads identical bits.

Tree shape follows the paper's spine tree (Sec. 4.1, Algorithm 1): a deep chain
(the spine, node 0 = the anchor/root) plus short branch chains hung on spine
nodes, in topological order (``parent[i] < i``).  The acceptance structure follows
the heterogeneous acceptance model (Sec. 3): a spine child is "correct" with
probability ``p_spine`` and a branch child with probability ``p_branch``; a
correct child has +10 added to its parent's logit row at the child's token.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

HEAD_DIM = 128
VOCAB = 32000


@dataclass(frozen=True)
class VerifyConfig:
    """One workload of the benchmark table (index = position in ``CONFIGS``)."""

    name: str
    S: int                      # sequences in the batch
    H: int                      # query heads
    B: int                      # tree nodes per sequence, root included
    ctx: Tuple[int, int]        # prefix length range [lo, hi] (lo == hi: fixed)
    spine: Tuple[int, int]      # spine node count incl. root, range [lo, hi]
    branch_len_max: int         # longest branch chain
    p_spine: Tuple[float, float]
    p_branch: float
    V: int = VOCAB
    k: int = 8
    D: int = HEAD_DIM
    Hkv: Optional[int] = None   # key/value heads (None: multi-head attention, one per query head)


CONFIGS: List[VerifyConfig] = [
    VerifyConfig("tiny", S=1, H=32, B=16, ctx=(512, 512), spine=(6, 6), branch_len_max=2,
                 p_spine=(0.8, 0.8), p_branch=0.15),
    VerifyConfig("7b", S=1, H=32, B=80, ctx=(2048, 2048), spine=(16, 16), branch_len_max=3,
                 p_spine=(0.8, 0.8), p_branch=0.15),
    VerifyConfig("13b", S=1, H=40, B=80, ctx=(4096, 4096), spine=(20, 20), branch_len_max=3,
                 p_spine=(0.85, 0.85), p_branch=0.10),
    VerifyConfig("33b", S=1, H=52, B=128, ctx=(8192, 8192), spine=(24, 24), branch_len_max=3,
                 p_spine=(0.8, 0.8), p_branch=0.15),
    VerifyConfig("batch16", S=16, H=32, B=64, ctx=(1024, 16384), spine=(4, 20), branch_len_max=3,
                 p_spine=(0.5, 0.95), p_branch=0.15),
    # second workload: grouped-query attention and a large vocabulary, the shape of the 8B models of the
    # paper's evaluation (32 query heads over 8 key/value heads, 128 256 vocabulary entries)
    VerifyConfig("gqa8b", S=4, H=32, B=32, ctx=(4096, 16384), spine=(6, 12), branch_len_max=3,
                 p_spine=(0.5, 0.95), p_branch=0.15, V=128256, Hkv=8),
]

# stream ids: one independent generator per tensor
_ST_TREE, _ST_TOK, _ST_LOGIT, _ST_PLANT, _ST_Q, _ST_K, _ST_V, _ST_SHAPE = range(8)


def _rng(seed: int, config_id: int, seq_id: int, stream_id: int) -> np.random.Generator:
    return np.random.default_rng([seed, config_id, seq_id, stream_id])


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------- trees
def spine_tree(rng: np.random.Generator, B: int, n_spine: int, branch_len_max: int
               ) -> Tuple[np.ndarray, np.ndarray]:
    """Spine chain 0..n_spine-1, then branch chains on uniformly random spine nodes.

    Returns ``parent`` (int32, parent[0] = -1, parent[i] < i) and ``is_spine`` (bool).
    """
    n_spine = max(1, min(n_spine, B))
    parent = np.full(B, -1, dtype=np.int32)
    is_spine = np.zeros(B, dtype=bool)
    for i in range(n_spine):
        parent[i] = i - 1
        is_spine[i] = True
    n = n_spine
    while n < B:
        u = int(rng.integers(0, n_spine))
        L = int(rng.integers(1, branch_len_max + 1))
        L = min(L, B - n)
        prev = u
        for _ in range(L):
            parent[n] = prev
            prev = n
            n += 1
    return parent, is_spine


def chain_tree(B: int) -> np.ndarray:
    """Bypass mode (Sec. 4.3): the tree is a single linear chain."""
    p = np.arange(-1, B - 1, dtype=np.int32)
    return p


def star_tree(B: int) -> np.ndarray:
    p = np.zeros(B, dtype=np.int32)
    p[0] = -1
    return p


def kary_tree(B: int, k: int) -> np.ndarray:
    """Isotropic(k): balanced k-ary tree in BFS order (the paper's topology control)."""
    p = np.array([-1] + [(i - 1) // k for i in range(1, B)], dtype=np.int32)
    return p


def random_tree(rng: np.random.Generator, B: int) -> np.ndarray:
    """Uniformly random recursive tree: parent[i] uniform in [0, i)."""
    p = np.full(B, -1, dtype=np.int32)
    for i in range(1, B):
        p[i] = int(rng.integers(0, i))
    return p


def distinct_sibling_tokens(rng: np.random.Generator, parent: np.ndarray, V: int) -> np.ndarray:
    """Draft tokens uniform in [0, V), redrawn until distinct among siblings."""
    B = len(parent)
    if B > 1 and int(np.bincount(np.asarray(parent[1:], dtype=np.int64)).max()) > V:
        raise ValueError("a node has more children than there are tokens")
    tok = rng.integers(0, V, size=B).astype(np.int32)
    seen: Dict[int, set] = {}
    for i in range(B):
        s = seen.setdefault(int(parent[i]), set())
        while int(tok[i]) in s:
            tok[i] = int(rng.integers(0, V))
        s.add(int(tok[i]))
    return tok


def planted_logits(rng_val: np.random.Generator, rng_plant: np.random.Generator,
                   parent: np.ndarray, is_spine: np.ndarray, draft_tok: np.ndarray, V: int,
                   p_spine: float, p_branch: float) -> Tuple[np.ndarray, np.ndarray]:
    """N(0,1) logits [B][V]; with the class probability add +10 at the child's token in
    its parent's row; round to bf16.  Returns (bf16 bits, planted flags)."""
    B = len(parent)
    x = rng_val.standard_normal((B, V), dtype=np.float32)
    u = rng_plant.random(B)
    planted = np.zeros(B, dtype=bool)
    for i in range(1, B):
        p = p_spine if is_spine[i] else p_branch
        if u[i] < p:
            planted[i] = True
            x[int(parent[i]), int(draft_tok[i])] += np.float32(10.0)
    return f32_to_bf16_bits(x), planted


def normal_bf16(rng: np.random.Generator, shape, chunk_rows: int = 1 << 14) -> np.ndarray:
    """bf16 bits of N(0,1) samples, generated in row chunks to bound fp32 scratch."""
    shape = tuple(int(s) for s in shape)
    out = np.empty(shape, dtype=np.uint16)
    if len(shape) == 0 or shape[0] == 0:
        return out
    flat = out.reshape(shape[0], -1)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        flat[r0:r1] = f32_to_bf16_bits(rng.standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32))
    return out


# ----------------------------------------------------------------------------- workloads
@dataclass
class VerifyInputs:
    """All inputs of one verification step (host arrays)."""

    S: int
    B: int
    H: int
    D: int
    V: int
    k: int
    scale: float                       # 1/sqrt(D), python float (fp64)
    q: np.ndarray                      # uint16 [S][B][H][D]
    k_cache: np.ndarray                # uint16 [rows][Hkv][D]
    v_cache: np.ndarray                # uint16 [rows][Hkv][D]
    row_off: np.ndarray                # int64 [S]
    ctx_len: np.ndarray                # int32 [S]
    parent: np.ndarray                 # int32 [S][B]
    draft_tok: np.ndarray              # int32 [S][B]
    logits: np.ndarray                 # uint16 [S*B][V]
    is_spine: np.ndarray               # bool [S][B]   (generator metadata)
    planted: np.ndarray                # bool [S][B]   (generator metadata)
    p_spine: np.ndarray                # float64 [S]   (generator metadata)
    p_branch: float = 0.0
    name: str = ""
    meta: dict = field(default_factory=dict)

    @property
    def kv_rows(self) -> int:
        return int(self.k_cache.shape[0])

    @property
    def Hkv(self) -> int:
        return int(self.k_cache.shape[1])


def make_inputs(S: int, H: int, B: int, ctx_lens, parents, *, V: int = VOCAB, k: int = 8,
                seed: int = 0, config_id: int = 99, is_spine=None, p_spine=0.8, p_branch=0.15,
                D: int = HEAD_DIM, with_logits: bool = True, q_gain: float = 1.0,
                name: str = "custom", Hkv: Optional[int] = None) -> VerifyInputs:
    """Build a step's inputs from explicit prefix lengths and parent arrays.  ``Hkv`` key/value heads
    (default: H, multi-head attention)."""
    Hkv = H if Hkv is None else int(Hkv)
    if Hkv < 1 or H % Hkv != 0:
        raise ValueError("H must be a multiple of Hkv")
    ctx_lens = np.asarray(ctx_lens, dtype=np.int32).reshape(S)
    parents = np.asarray(parents, dtype=np.int32).reshape(S, B)
    if is_spine is None:
        is_spine = np.zeros((S, B), dtype=bool)
    is_spine = np.asarray(is_spine, dtype=bool).reshape(S, B)
    p_sp = np.broadcast_to(np.asarray(p_spine, dtype=np.float64), (S,)).copy()
    rows_per_seq = ctx_lens.astype(np.int64) + B
    row_off = np.concatenate([[0], np.cumsum(rows_per_seq)[:-1]]).astype(np.int64)
    total = int(rows_per_seq.sum())
    q = np.empty((S, B, H, D), dtype=np.uint16)
    kc = np.empty((total, Hkv, D), dtype=np.uint16)
    vc = np.empty((total, Hkv, D), dtype=np.uint16)
    tok = np.empty((S, B), dtype=np.int32)
    planted = np.zeros((S, B), dtype=bool)
    logits = np.empty((S * B, V), dtype=np.uint16) if with_logits else np.empty((0, V), dtype=np.uint16)
    for s in range(S):
        r0, n = int(row_off[s]), int(rows_per_seq[s])
        qf = _rng(seed, config_id, s, _ST_Q).standard_normal((B, H, D), dtype=np.float32)
        if q_gain != 1.0:
            qf = qf * np.float32(q_gain)
        q[s] = f32_to_bf16_bits(qf)
        kc[r0:r0 + n] = normal_bf16(_rng(seed, config_id, s, _ST_K), (n, Hkv, D))
        vc[r0:r0 + n] = normal_bf16(_rng(seed, config_id, s, _ST_V), (n, Hkv, D))
        tok[s] = distinct_sibling_tokens(_rng(seed, config_id, s, _ST_TOK), parents[s], V if with_logits else max(V, 4096))
        if with_logits:
            bits, pl = planted_logits(_rng(seed, config_id, s, _ST_LOGIT), _rng(seed, config_id, s, _ST_PLANT),
                                      parents[s], is_spine[s], tok[s], V, float(p_sp[s]), p_branch)
            logits[s * B:(s + 1) * B] = bits
            planted[s] = pl
    return VerifyInputs(S=S, B=B, H=H, D=D, V=V, k=k, scale=1.0 / float(np.sqrt(np.float64(D))),
                        q=q, k_cache=kc, v_cache=vc, row_off=row_off, ctx_len=ctx_lens,
                        parent=parents, draft_tok=tok, logits=logits, is_spine=is_spine,
                        planted=planted, p_spine=p_sp, p_branch=p_branch, name=name)


def config_shapes(config_id: int, seed: int = 0):
    """Per-sequence (ctx_len, parent, is_spine, p_spine) of a table config; cheap (no tensors)."""
    cfg = CONFIGS[config_id]
    ctxs, parents, spines, ps = [], [], [], []
    for s in range(cfg.S):
        rs = _rng(seed, config_id, s, _ST_SHAPE)
        ctx = int(rs.integers(cfg.ctx[0], cfg.ctx[1] + 1))
        n_sp = int(rs.integers(cfg.spine[0], cfg.spine[1] + 1))
        p_sp = float(rs.uniform(cfg.p_spine[0], cfg.p_spine[1])) if cfg.p_spine[0] != cfg.p_spine[1] else cfg.p_spine[0]
        par, sp = spine_tree(_rng(seed, config_id, s, _ST_TREE), cfg.B, n_sp, cfg.branch_len_max)
        ctxs.append(ctx); parents.append(par); spines.append(sp); ps.append(p_sp)
    return cfg, np.array(ctxs, np.int32), np.stack(parents), np.stack(spines), np.array(ps)


def make_config(config_id: int, seed: int = 0, *, with_logits: bool = True,
                ctx_override: Optional[int] = None) -> VerifyInputs:
    """Inputs of benchmark config ``config_id`` (0..5).  ``ctx_override`` shrinks the prefix
    (same tree / heads / vocabulary) for cases the oracle should finish quickly."""
    cfg, ctxs, parents, spines, ps = config_shapes(config_id, seed)
    if ctx_override is not None:
        ctxs = np.minimum(ctxs, np.int32(ctx_override))
    return make_inputs(cfg.S, cfg.H, cfg.B, ctxs, parents, V=cfg.V, k=cfg.k, seed=seed,
                       config_id=config_id, is_spine=spines, p_spine=ps, p_branch=cfg.p_branch,
                       D=cfg.D, with_logits=with_logits, name=cfg.name, Hkv=cfg.Hkv)


def algorithmic_bytes(S: int, H: int, B: int, D: int, V: int, ctx_lens, Hkv: Optional[int] = None) -> Dict[str, int]:
    """Bytes each part of the step must move at least once (bf16 = 2 bytes)."""
    ctx_lens = np.asarray(ctx_lens, dtype=np.int64)
    Hkv = H if Hkv is None else Hkv
    kv = int((2 * (ctx_lens + B) * Hkv * D * 2).sum())
    qo = int(2 * S * B * H * D * 2)
    logits = int(S * B * V * 2)
    return {"attn": kv + qo, "topk": logits, "total": kv + qo + logits}
