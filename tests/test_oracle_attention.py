"""Pins for the oracle's tree attention: things the paper and the mathematics fix,
none of which re-uses the oracle's own formula.

Sec. 4 (Stage 1) defines the tree attention mask: each node attends only to its
root-to-node ancestors (plus the shared prefix), so every root-to-leaf path is scored
as if it had been decoded sequentially -- the losslessness argument of the method.
"""
import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax

from paper_2604_02047_b200 import synth


def _f64(bits):
    return synth.bf16_bits_to_f64(bits)


def _small(S=1, H=3, B=9, ctx=(37,), parents=None, seed=3, **kw):
    if parents is None:
        rng = np.random.default_rng(seed)
        parents = [synth.random_tree(rng, B) for _ in range(S)]
    return synth.make_inputs(S, H, B, list(ctx), parents, V=16, with_logits=False, seed=seed, **kw)


def test_chain_tree_equals_library_causal_attention(oracle):
    """A chain-shaped tree (bypass mode, Sec. 4.3) must be ordinary causal attention."""
    x = _small(S=1, H=4, B=12, ctx=(29,), parents=[synth.chain_tree(12)])
    out, lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    n = 29 + 12
    K = torch.from_numpy(_f64(x.k_cache)).permute(1, 0, 2)        # [H][n][D]
    V = torch.from_numpy(_f64(x.v_cache)).permute(1, 0, 2)
    Q = torch.zeros(4, n, 128, dtype=torch.float64)
    Q[:, 29:, :] = torch.from_numpy(_f64(x.q[0])).permute(1, 0, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True, scale=x.scale)
    ref = ref[:, 29:, :].permute(1, 0, 2).numpy()                  # [B][H][D]
    assert np.abs(out[0] - ref).max() < 1e-12


def test_every_node_equals_sequential_decode_along_its_path(oracle):
    """out[i] == single-query attention of q_i over (prefix + K/V of the root-to-i path)."""
    x = _small(S=2, H=2, B=11, ctx=(23, 5), seed=11)
    out, lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    K, V, Q = _f64(x.k_cache), _f64(x.v_cache), _f64(x.q)
    for s in range(2):
        r0, ctx = int(x.row_off[s]), int(x.ctx_len[s])
        for i in range(11):
            chain, v = [], i
            while v != -1:
                chain.append(v); v = int(x.parent[s, v])
            rows = list(range(r0, r0 + ctx)) + [r0 + ctx + j for j in reversed(chain)]
            for h in range(2):
                sc = (K[rows, h, :] @ Q[s, i, h, :]) / np.sqrt(128.0)
                ref = softmax(sc) @ V[rows, h, :]
                assert np.abs(out[s, i, h] - ref).max() < 1e-12
                assert abs(lse[s, i, h] - logsumexp(sc)) < 1e-12


def test_root_only_tree_is_single_query_decode(oracle):
    """B = 1 is the autoregressive fallback (Algorithm 2): plain decode attention."""
    x = _small(S=1, H=2, B=1, ctx=(40,), parents=[np.array([-1], np.int32)])
    out, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    K, V, Q = _f64(x.k_cache), _f64(x.v_cache), _f64(x.q)
    for h in range(2):
        ref = softmax(K[:, h, :] @ Q[0, 0, h] * x.scale) @ V[:, h, :]
        assert np.abs(out[0, 0, h] - ref).max() < 1e-12


def test_empty_prefix(oracle):
    x = _small(S=1, H=1, B=5, ctx=(0,), parents=[synth.star_tree(5)])
    out, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    V = _f64(x.v_cache)
    assert np.abs(out[0, 0, 0] - V[0, 0]).max() < 1e-14         # root sees only itself


def test_relabelling_the_tree_permutes_the_outputs(oracle):
    """Another topological order of the same tree gives the same per-node results."""
    B = 10
    x = _small(S=1, H=2, B=B, ctx=(17,), seed=5)
    out, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    par = x.parent[0]
    # new order: DFS preorder (a valid topological order, generally different from the given one)
    kids = {i: [c for c in range(B) if par[c] == i] for i in range(B)}
    order, stack = [], [0]
    while stack:
        v = stack.pop(); order.append(v); stack.extend(reversed(kids[v]))
    assert order != list(range(B))
    new_of_old = {o: n for n, o in enumerate(order)}
    par2 = np.array([-1 if par[o] < 0 else new_of_old[int(par[o])] for o in order], np.int32)
    q2 = x.q[:, order]
    k2, v2 = x.k_cache.copy(), x.v_cache.copy()
    k2[17:] = x.k_cache[17:][order]; v2[17:] = x.v_cache[17:][order]
    out2, _ = oracle.tree_attn(q2, k2, v2, x.row_off, x.ctx_len, par2[None], x.scale)
    assert np.abs(out2[0] - out[0][order]).max() < 1e-13


def test_softmax_identities(oracle):
    x = _small(S=1, H=2, B=8, ctx=(19,), seed=9)
    one = np.full_like(x.v_cache, 0x3F80)                        # bf16 1.0
    out, _ = oracle.tree_attn(x.q, x.k_cache, one, x.row_off, x.ctx_len, x.parent, x.scale)
    assert np.abs(out - 1.0).max() < 1e-14                       # weights sum to one
    # all keys equal -> uniform weights over exactly the visible keys
    keq = np.broadcast_to(x.k_cache[:1], x.k_cache.shape).copy()
    out, lse = oracle.tree_attn(x.q, keq, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    V = _f64(x.v_cache)
    for i in range(8):
        anc, v = [], i
        while v != -1:
            anc.append(19 + v); v = int(x.parent[0, v])
        rows = list(range(19)) + anc
        assert np.abs(out[0, i] - V[rows].mean(axis=0)).max() < 1e-13
    # star tree: every non-root node sees the prefix, the root and itself only
    y = _small(S=1, H=1, B=6, ctx=(3,), parents=[synth.star_tree(6)], seed=2)
    out, _ = oracle.tree_attn(y.q, y.k_cache, y.v_cache, y.row_off, y.ctx_len, y.parent, y.scale)
    K, V, Q = _f64(y.k_cache), _f64(y.v_cache), _f64(y.q)
    for i in range(1, 6):
        rows = [0, 1, 2, 3, 3 + i]
        ref = softmax(K[rows, 0] @ Q[0, i, 0] * y.scale) @ V[rows, 0]
        assert np.abs(out[0, i, 0] - ref).max() < 1e-13


def test_scale_and_operand_roles(oracle):
    """Guards against a dropped scale, swapped K/V or a transposed operand."""
    x = _small(S=1, H=1, B=4, ctx=(6,), parents=[synth.chain_tree(4)])
    o1, l1 = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    o2, l2 = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, 0.0)
    V = _f64(x.v_cache)
    for i in range(4):                                            # scale 0 -> plain mean, lse = ln(n)
        assert np.abs(o2[0, i, 0] - V[:6 + i + 1, 0].mean(axis=0)).max() < 1e-13
        assert abs(l2[0, i, 0] - np.log(6 + i + 1)) < 1e-13
    assert np.abs(o1 - o2).max() > 1e-3
    o3, _ = oracle.tree_attn(x.q, x.v_cache, x.k_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    assert np.abs(o1 - o3).max() > 1e-3


def test_sampled_rows_match_full(oracle):
    x = _small(S=2, H=3, B=7, ctx=(11, 30), seed=21)
    out, lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    ss, si, sh = [0, 1, 1, 0], [6, 0, 3, 2], [2, 1, 0, 0]
    o, l = oracle.tree_attn_rows(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, ss, si, sh)
    for n in range(4):
        assert np.array_equal(o[n], out[ss[n], si[n], sh[n]]) and l[n] == lse[ss[n], si[n], sh[n]]


def test_invalid_parent_is_rejected(oracle):
    x = _small(S=1, H=1, B=4, ctx=(2,), parents=[synth.chain_tree(4)])
    bad = x.parent.copy(); bad[0, 2] = 3
    with pytest.raises(ValueError):
        oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, bad, x.scale)
    assert not oracle.check_parent(bad) and oracle.check_parent(x.parent)
    # every way parent[] can fail to be a rooted tree in topological order (parent[0] = -1, 0 <= parent[i] < i)
    for bad in ([0, 0, 1], [-1, 1, 0], [-1, -1, 0], [-1, 0, 2], [-1, 0, 3], [1, 0, 0], [-2, 0, 1]):
        assert not oracle.check_parent(np.array(bad, np.int32)), bad
        with pytest.raises(ValueError):
            oracle.ancestors(np.array(bad, np.int32))
    for good in ([-1], [-1, 0], [-1, 0, 0, 2, 1, 4]):
        assert oracle.check_parent(np.array(good, np.int32))
    assert oracle.ancestors([-1, 0, 0, 2, 1, 4]) == [0b1, 0b11, 0b101, 0b1101, 0b10011, 0b110011]


# ------------------------------------------------------------------ grouped-query attention
def test_gqa_equals_mha_on_replicated_kv_heads(oracle):
    """Query head h of a grouped-query model reads key/value head h // g (groups of g consecutive query heads):
    the result is that of multi-head attention over caches whose heads are each repeated g times in place."""
    for H, Hkv in ((8, 2), (6, 2), (4, 1), (3, 3)):
        g = H // Hkv
        x = _small(S=2, H=H, B=7, ctx=(19, 4), seed=5 + H, Hkv=Hkv)
        assert x.k_cache.shape[1] == Hkv
        out, lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
        k_rep, v_rep = np.repeat(x.k_cache, g, axis=1), np.repeat(x.v_cache, g, axis=1)
        ref, ref_lse = oracle.tree_attn(x.q, k_rep, v_rep, x.row_off, x.ctx_len, x.parent, x.scale)
        assert np.array_equal(out, ref) and np.array_equal(lse, ref_lse)
        if g > 1 and Hkv > 1:
            # the interleaved assignment (h % Hkv) is a different function
            k_til, v_til = np.tile(x.k_cache, (1, g, 1)), np.tile(x.v_cache, (1, g, 1))
            other, _ = oracle.tree_attn(x.q, k_til, v_til, x.row_off, x.ctx_len, x.parent, x.scale)
            assert np.abs(other - ref).max() > 1e-3


def test_gqa_rows_by_direct_formula(oracle):
    """Every (node, query head) row written out with numpy: softmax over prefix + ancestors of the group's KV head."""
    H, Hkv, B = 6, 3, 10
    x = _small(S=1, H=H, B=B, ctx=(21,), seed=23, Hkv=Hkv)
    out, lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    K, V, Q = _f64(x.k_cache), _f64(x.v_cache), _f64(x.q)
    for i in range(B):
        chain, v = [], i
        while v != -1:
            chain.append(v); v = int(x.parent[0, v])
        rows = list(range(21)) + [21 + j for j in sorted(chain)]
        for h in range(H):
            hk = h // (H // Hkv)
            sc = (K[rows, hk, :] @ Q[0, i, h, :]) / np.sqrt(128.0)
            assert np.abs(out[0, i, h] - softmax(sc) @ V[rows, hk, :]).max() < 1e-12
            assert abs(lse[0, i, h] - logsumexp(sc)) < 1e-12
    # sampled-row entry point agrees with the full one
    ss = np.zeros(5, np.int32); si = np.array([0, 3, 9, 4, 7], np.int32); sh = np.array([5, 0, 2, 3, 4], np.int32)
    o2, l2 = oracle.tree_attn_rows(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, ss, si, sh)
    assert np.array_equal(o2, out[ss, si, sh]) and np.array_equal(l2, lse[ss, si, sh])


def test_gqa_rejects_heads_that_do_not_divide(oracle):
    x = _small(S=1, H=4, B=5, ctx=(8,), seed=2)
    with pytest.raises(ValueError):
        oracle.tree_attn(x.q, x.k_cache[:, :3], x.v_cache[:, :3], x.row_off, x.ctx_len, x.parent, x.scale)
