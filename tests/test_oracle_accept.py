"""Pins for the oracle's greedy acceptance walk (Algorithm 3, UnifiedGreedyWalk)."""
import os

import numpy as np
import pytest

from paper_2604_02047_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "accept_hand_example.txt")


def _load_hand_example():
    ex = {"cases": []}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(None, 1)
        if key == "case":
            name, am, path, alen, bonus = [t.strip() for t in rest.split("|")]
            ex["cases"].append((name, [int(t) for t in am.split()], [int(t) for t in path.split()], int(alen), int(bonus)))
        elif key == "anc":
            ex["anc"] = [int(t, 2) for t in rest.split()]
        elif key == "B":
            ex["B"] = int(rest)
        else:
            ex[key] = [int(t) for t in rest.split()]
    return ex


def test_hand_example(oracle):
    ex = _load_hand_example()
    B = ex["B"]
    assert oracle.ancestors(ex["parent"]) == ex["anc"]          # the ancestor sets behind the tree attention mask
    for name, am, path, alen, bonus in ex["cases"]:
        p, l, b = oracle.accept(ex["draft_tok"], ex["parent"], am)
        assert l[0] == alen and b[0] == bonus, name
        assert p[0].tolist() == path + [-1] * (B - len(path)), name


def _root_to_leaf_paths(parent):
    B = len(parent)
    kids = {i: [c for c in range(B) if parent[c] == i] for i in range(B)}
    paths = []

    def rec(v, acc):
        if not kids[v]:
            paths.append(acc)
        for c in kids[v]:
            rec(c, acc + [c])
    rec(0, [0])
    return paths


def test_brute_force_over_all_root_to_leaf_paths(oracle):
    """The walk 'automatically discovers the longest accepted path' (Sec. 4.2): enumerate every
    root-to-leaf path, count its matching prefix, and compare the best one with the walk."""
    rng = np.random.default_rng(7)
    for trial in range(300):
        B = int(rng.integers(1, 11))
        parent = synth.random_tree(rng, B)
        tok = synth.distinct_sibling_tokens(rng, parent, 4 if B < 6 else 12)
        am = rng.integers(0, 5, size=B).astype(np.int32)
        best = [0]
        for path in _root_to_leaf_paths(parent):
            n = 1
            while n < len(path) and tok[path[n]] == am[path[n - 1]]:
                n += 1
            if n > len(best):
                best = path[:n]
            elif n == len(best):
                assert path[:n] == best                    # distinct siblings: the accepted prefix is unique
        p, l, b = oracle.accept(tok, parent, am)
        assert l[0] == len(best) - 1
        assert p[0, :len(best)].tolist() == best and np.all(p[0, len(best):] == -1)
        assert b[0] == am[best[-1]]


def test_source_priority_never_changes_the_path_with_distinct_siblings(oracle):
    rng = np.random.default_rng(8)
    for trial in range(100):
        B = 12
        parent, is_spine = synth.spine_tree(rng, B, 5, 2)
        tok = synth.distinct_sibling_tokens(rng, parent, 16)
        am = rng.integers(0, 16, size=B).astype(np.int32)
        a = oracle.accept(tok, parent, am)
        b = oracle.accept(tok, parent, am, tag=is_spine[None])
        assert all(np.array_equal(u, v) for u, v in zip(a, b))


def test_duplicate_siblings_are_defined(oracle):
    parent = np.array([-1, 0, 0, 0], np.int32)
    tok = np.array([1, 5, 5, 5], np.int32)
    am = np.array([5, 9, 8, 7], np.int32)
    p, l, b = oracle.accept(tok, parent, am)
    assert p[0].tolist() == [0, 1, -1, -1] and b[0] == 9        # lowest index wins without tags
    p, l, b = oracle.accept(tok, parent, am, tag=np.array([[0, 0, 1, 0]]))
    assert p[0].tolist() == [0, 2, -1, -1] and b[0] == 8        # Algorithm 3: spine child first


def test_full_chain_accepted_and_single_node(oracle):
    B = 9
    parent = synth.chain_tree(B)
    tok = np.arange(100, 100 + B, dtype=np.int32)
    am = np.concatenate([tok[1:], [42]]).astype(np.int32)
    p, l, b = oracle.accept(tok, parent, am)
    assert l[0] == B - 1 and p[0].tolist() == list(range(B)) and b[0] == 42
    p, l, b = oracle.accept([3], [-1], [17])
    assert l[0] == 0 and p[0].tolist() == [0] and b[0] == 17
    with pytest.raises(ValueError):
        oracle.accept([1, 2, 3], [-1, 2, 0], [0, 0, 0])


def test_expected_yield_matches_eq1_when_branches_are_independent_chains(oracle):
    """Eq. (1): E[tau] >= sum_{i=1..m} ps^i + sum_{i=0..m-1} ps^i (1-ps) phi_i (1 + lbar) + 1, tight when
    the branches are independent chains.  Draw the target's argmax from exactly that acceptance model
    (Sec. 3) and let the walk count tokens; the Monte-Carlo mean must sit on the closed form."""
    ps, pt, m, D = 0.6, 0.25, 4, 4
    w = [3, 2, 1, 1]                                           # branch widths at spine nodes 0..m-1
    # build the tree: spine 0..m, then for spine node i: w_i branch chains of D-1+1 nodes
    parent = [-1] + list(range(0, m))
    heads = {i: [] for i in range(m)}
    for i in range(m):
        for _ in range(w[i]):
            prev = i
            for d in range(D):                                  # branch token + D-1 extension tokens
                parent.append(prev); prev = len(parent) - 1
                if d == 0:
                    heads[i].append(prev)
    parent = np.array(parent, np.int32)
    B = len(parent)
    kids = {i: [c for c in range(B) if parent[c] == i] for i in range(B)}
    tok = np.arange(1000, 1000 + B, dtype=np.int32)            # all distinct
    N = 40000
    rng = np.random.default_rng(123)
    am = np.full((N, B), -5, np.int32)                          # -5 matches nothing
    for v in range(B):
        if v < m:                                               # spine node with a spine child v+1
            u = rng.random(N)
            spine_ok = u < ps
            phi = 1 - (1 - pt) ** w[v]
            branch_ok = (~spine_ok) & (rng.random(N) < phi)
            pick = np.array(heads[v])[rng.integers(0, w[v], size=N)]
            am[spine_ok, v] = tok[v + 1]
            am[branch_ok, v] = tok[pick[branch_ok]]
        elif kids[v]:                                           # inside a branch chain
            ok = rng.random(N) < pt
            am[ok, v] = tok[kids[v][0]]
    _, alen, _ = oracle.accept(np.broadcast_to(tok, (N, B)), np.broadcast_to(parent, (N, B)), am)
    tau = alen.astype(np.float64) + 1.0
    lbar = sum(pt ** k for k in range(1, D))
    eq1 = sum(ps ** i for i in range(1, m + 1)) \
        + sum(ps ** i * (1 - ps) * (1 - (1 - pt) ** w[i]) * (1 + lbar) for i in range(m)) + 1.0
    se = tau.std() / np.sqrt(N)
    assert abs(tau.mean() - eq1) < 5 * se + 1e-3, (tau.mean(), eq1, se)


def _expected_accept_len(parent, is_spine, p_spine, p_branch):
    """Exact E[accept_len] under the generator: a reached node's accepted child is its planted
    child with the largest N(0,1)+10 value, i.e. uniform among the planted siblings."""
    B = len(parent)
    reach = np.zeros(B); reach[0] = 1.0
    total = 0.0
    for c in range(1, B):
        sib = [x for x in range(1, B) if parent[x] == parent[c] and x != c]
        dist = np.array([1.0])                                  # distribution of #planted other siblings
        for x in sib:
            p = p_spine if is_spine[x] else p_branch
            dist = np.convolve(dist, [1 - p, p])
        pc = p_spine if is_spine[c] else p_branch
        win = pc * sum(dist[n] / (1 + n) for n in range(len(dist)))
        reach[c] = reach[parent[c]] * win
        total += reach[c]
    return total


def test_generator_acceptance_statistics(oracle):
    """End to end over seeds: generator logits -> oracle top-k -> oracle walk; the mean accepted
    length must match the exact per-tree expectation of the planted-acceptance model."""
    B, V, n_seeds = 16, 2048, 400
    got, exp = [], []
    for seed in range(n_seeds):
        rng = np.random.default_rng([seed, 77])
        parent, is_spine = synth.spine_tree(rng, B, 6, 2)
        tok = synth.distinct_sibling_tokens(rng, parent, V)
        bits, _ = synth.planted_logits(np.random.default_rng([seed, 78]), np.random.default_rng([seed, 79]),
                                       parent, is_spine, tok, V, 0.8, 0.15)
        am, _, _ = oracle.node_topk(bits, 1)
        _, alen, _ = oracle.accept(tok, parent, am)
        got.append(float(alen[0])); exp.append(_expected_accept_len(parent, is_spine, 0.8, 0.15))
    got, exp = np.array(got), np.array(exp)
    se = got.std() / np.sqrt(n_seeds)
    assert abs(got.mean() - exp.mean()) < 4 * se + 0.03, (got.mean(), exp.mean(), se)
    assert 1.5 < got.mean() < 4.5                               # tau = mean+1 lands in the paper's measured range
