"""Pins for the per-sequence node counts n_nodes[s] <= B (a batch whose sequences carry trees of different sizes, and
sequences that have left the batch: the paper's batched prototype pads finished requests and pays for them, App.
"Batch-Size Sweep").  The definition is "the result on the tree cut to its first n nodes": every function with n_nodes
is compared with the same function WITHOUT n_nodes (pinned elsewhere) run on inputs that were cut by hand, sequence by
sequence; rows and values of nodes that do not exist are poisoned to show that they are never read."""
import numpy as np
import pytest

from paper_2604_02047_b200 import synth

NAN16 = 0x7FC0          # bf16 NaN


def _batch(seed=3, S=5, H=3, B=12, V=257):
    rng = np.random.default_rng(seed)
    parents = [synth.random_tree(rng, B) if s % 2 else synth.spine_tree(rng, B, 5, 2)[0] for s in range(S)]
    x = synth.make_inputs(S, H, B, [37, 0, 130, 5, 64][:S], parents, V=V, k=4, seed=seed, p_spine=0.9, p_branch=0.6,
                          is_spine=np.ones((S, B), bool))
    n_nodes = np.array([B, 1, 7, 0, B - 1][:S], np.int32)
    return x, n_nodes


def _poison(x, n_nodes):
    """Copies of the inputs in which everything that belongs to a node that does not exist is garbage."""
    q, kc, vc = x.q.copy(), x.k_cache.copy(), x.v_cache.copy()
    par, tok, lg = x.parent.copy(), x.draft_tok.copy(), x.logits.copy()
    for s in range(x.S):
        n = int(n_nodes[s])
        q[s, n:] = NAN16; par[s, n:] = 99; tok[s, n:] = -7
        r = int(x.row_off[s]) + int(x.ctx_len[s])
        kc[r + n:r + x.B] = NAN16; vc[r + n:r + x.B] = NAN16
        lg[s * x.B + n:(s + 1) * x.B] = NAN16
    return q, kc, vc, par, tok, lg


def test_attention_equals_the_cut_tree_sequence_by_sequence(oracle):
    x, n_nodes = _batch()
    q, kc, vc, par, tok, lg = _poison(x, n_nodes)
    out, lse = oracle.tree_attn(q, kc, vc, x.row_off, x.ctx_len, par, x.scale, n_nodes=n_nodes)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    for s in range(x.S):
        n = int(n_nodes[s])
        assert np.all(out[s, n:] == 0) and np.all(lse[s, n:] == 0)          # never written
        if n == 0:
            continue
        r0, ctx = int(x.row_off[s]), int(x.ctx_len[s])
        ref, ref_lse = oracle.tree_attn(x.q[s:s + 1, :n], x.k_cache[r0:r0 + ctx + n], x.v_cache[r0:r0 + ctx + n], [0], [ctx],
                                        x.parent[s:s + 1, :n], x.scale)
        assert np.array_equal(out[s, :n], ref[0]) and np.array_equal(lse[s, :n], ref_lse[0])
    with pytest.raises(ValueError):
        oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, n_nodes=[x.B + 1, 1, 1, 1, 1])
    # n_nodes = B everywhere is the plain call
    a, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, n_nodes=[x.B] * x.S)
    b, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
    assert np.array_equal(a, b)


def test_topk_walk_and_compaction_equal_the_cut_tree(oracle):
    x, n_nodes = _batch(seed=4)
    q, kc, vc, par, tok, lg = _poison(x, n_nodes)
    B, S, k = x.B, x.S, x.k
    am, ids, vals = oracle.node_topk(lg, k, n_nodes=n_nodes, B=B)
    path, alen, bonus = oracle.accept(tok, par, am.reshape(S, B), n_nodes=n_nodes)
    ko, vo, new_ctx = oracle.kv_compact(kc, vc, x.row_off, x.ctx_len, path, alen, n_nodes=n_nodes)
    assert alen.max() >= 2                                                   # the generator planted real acceptances
    for s in range(S):
        n = int(n_nodes[s])
        rows = slice(s * B, s * B + n)
        assert np.all(ids[s * B + n:(s + 1) * B] == 0) and np.all(am[s * B + n:(s + 1) * B] == 0)   # never written
        if n == 0:                                                           # left the batch
            assert alen[s] == 0 and bonus[s] == -1 and np.all(path[s] == -1) and new_ctx[s] == x.ctx_len[s]
            continue
        ram, rids, rvals = oracle.node_topk(x.logits[rows], k)
        assert np.array_equal(am[rows], ram) and np.array_equal(ids[rows], rids) and np.array_equal(vals[rows], rvals)
        rp, rl, rb = oracle.accept(x.draft_tok[s:s + 1, :n], x.parent[s:s + 1, :n], ram[None])
        assert alen[s] == rl[0] and bonus[s] == rb[0]
        assert np.array_equal(path[s, :n], rp[0]) and np.all(path[s, n:] == -1)
        r0, ctx = int(x.row_off[s]), int(x.ctx_len[s])
        rk, rv, rn = oracle.kv_compact(x.k_cache[r0:r0 + ctx + n], x.v_cache[r0:r0 + ctx + n], [0], [ctx], rp, rl)
        assert new_ctx[s] == rn[0] == ctx + 1 + alen[s]
        assert np.array_equal(ko[r0:r0 + rn[0]], rk[:rn[0]]) and np.array_equal(vo[r0:r0 + rn[0]], rv[:rn[0]])
    # the batch without the sequence that left gives the same results for the others
    keep = [s for s in range(S) if n_nodes[s] > 0]
    am2, _, _ = oracle.node_topk(np.concatenate([lg[s * B:(s + 1) * B] for s in keep]), k, n_nodes=n_nodes[keep], B=B)
    p2, l2, b2 = oracle.accept(tok[keep], par[keep], am2.reshape(len(keep), B), n_nodes=n_nodes[keep])
    assert np.array_equal(p2, path[keep]) and np.array_equal(l2, alen[keep]) and np.array_equal(b2, bonus[keep])


def test_a_cut_inside_the_accepted_path_shortens_it(oracle):
    """Chain 0-1-2-3-4 with every child accepted: with n nodes the walk accepts n - 1 of them and the bonus is the
    prediction at node n - 1."""
    B = 5
    par = synth.chain_tree(B)[None]; tok = np.array([[10, 11, 12, 13, 14]], np.int32)
    am = np.array([[11, 12, 13, 14, 99]], np.int32)
    for n in range(1, B + 1):
        p, l, b = oracle.accept(tok, par, am, n_nodes=[n])
        assert l[0] == n - 1 and b[0] == am[0, n - 1] and p[0].tolist() == list(range(n)) + [-1] * (B - n)
