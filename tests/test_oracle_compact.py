"""Pins for the oracle's KV compaction.  The paper is silent on cache handling after acceptance;
the reading is: the accepted nodes' K/V rows follow the prefix in path order, so that the next
cycle sees exactly the cache a sequential decode of the accepted tokens would have produced."""
import numpy as np

from paper_2604_02047_b200 import synth


def test_compaction_equals_regather_and_sequential_cache(oracle):
    rng = np.random.default_rng(5)
    B, H = 10, 2
    parents = [synth.random_tree(rng, B) for _ in range(3)]
    x = synth.make_inputs(3, H, B, [9, 0, 21], parents, V=8, with_logits=False, seed=4)
    # accepted paths: walk down random children
    path = np.full((3, B), -1, np.int32); alen = np.zeros(3, np.int32)
    for s in range(3):
        v, L = 0, 0
        path[s, 0] = 0
        while True:
            kids = [c for c in range(B) if parents[s][c] == v]
            if not kids or rng.random() < 0.2:
                break
            v = int(rng.choice(kids)); L += 1; path[s, L] = v
        alen[s] = L
    ko, vo, new_ctx = oracle.kv_compact(x.k_cache, x.v_cache, x.row_off, x.ctx_len, path, alen)
    for s in range(3):
        r0, ctx, L = int(x.row_off[s]), int(x.ctx_len[s]), int(alen[s])
        assert new_ctx[s] == ctx + 1 + L
        rows = [r0 + ctx + int(path[s, j]) for j in range(L + 1)]
        assert np.array_equal(ko[r0 + ctx:r0 + ctx + L + 1], x.k_cache[rows])
        assert np.array_equal(vo[r0 + ctx:r0 + ctx + L + 1], x.v_cache[rows])
        assert np.array_equal(ko[r0:r0 + ctx], x.k_cache[r0:r0 + ctx])          # prefix untouched
        assert np.array_equal(ko[r0 + ctx + L + 1:r0 + ctx + B], x.k_cache[r0 + ctx + L + 1:r0 + ctx + B])
        # the compacted cache is the one a sequential decode would hold: the last accepted node's
        # tree-attention output equals plain decode attention of its query over the compacted rows
        last = int(path[s, L])
        o_tree, _ = oracle.tree_attn_rows(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale,
                                          [s] * H, [last] * H, list(range(H)))
        q1 = x.q[s:s + 1, last:last + 1]
        n = ctx + L + 1
        o_seq, _ = oracle.tree_attn(q1, ko[r0:r0 + n], vo[r0:r0 + n], [0], [n - 1], [[-1]], x.scale)
        assert np.abs(o_seq[0, 0] - o_tree).max() < 1e-13


def test_identity_path_is_a_noop_and_overlapping_moves(oracle):
    B, H = 6, 1
    x = synth.make_inputs(1, H, B, [4], [synth.chain_tree(B)], V=8, with_logits=False)
    path = np.arange(B, dtype=np.int32)[None]
    ko, vo, nc = oracle.kv_compact(x.k_cache, x.v_cache, x.row_off, x.ctx_len, path, [B - 1])
    assert np.array_equal(ko, x.k_cache) and np.array_equal(vo, x.v_cache) and nc[0] == 4 + B
    # path [0,2,3]: row ctx+2 is both a destination and a source -> must read the ORIGINAL row 3
    y = synth.make_inputs(1, H, 4, [2], [np.array([-1, 0, 0, 2], np.int32)], V=8, with_logits=False)
    ko, vo, nc = oracle.kv_compact(y.k_cache, y.v_cache, y.row_off, y.ctx_len, [[0, 2, 3, -1]], [2])
    assert np.array_equal(ko[3], y.k_cache[4]) and np.array_equal(ko[4], y.k_cache[5]) and nc[0] == 5
