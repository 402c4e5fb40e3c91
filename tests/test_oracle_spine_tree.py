"""Pins for the host-side oracle: Algorithm 1 (BuildSpineTree), ContextMatch, spine-ratio tiers."""
import numpy as np

from _golden import load_spine_tree_example
from oracle import spine_tree as st


def _table(V, K, rng):
    ids = np.stack([rng.permutation(V)[:K] for _ in range(V)]).astype(np.int32)
    return ids


def test_budget_identities_and_the_papers_root_share():
    for B in (16, 60, 64, 80, 128):
        for m in (0, 1, 5, 18, 40):
            for r in (0.15, 0.30, 0.50):
                b_s, b_r, b_rho = st.budget_split(m, B, r, 0.5)
                assert b_s + b_r + b_rho == B - 1 and b_s == min(m, int(B * r)) and b_r >= 0 and b_rho >= 0
    # default hyper-parameters (B = 60, rho = 0.5) at the middle tier r = 0.30: the root's share of the branch
    # budget is 20/41 = 0.488 -- the paper quotes "about 0.49" for the deployed rule (App. power-law allocation)
    b_s, b_r, b_rho = st.budget_split(40, 60, 0.30, 0.5)
    assert (b_s, b_r, b_rho) == (18, 20, 21) and abs(b_r / (b_r + b_rho) - 0.49) < 0.005


def test_harmonic_allocation_worked_by_hand():
    # b_s = 18, b_rho = 21: H_18 = 3.49511; 21/H = 6.008 -> a = floor(6.008 / i)
    assert st.harmonic_allocation(18, 21) == [6, 3, 2, 1, 1, 1] + [0] * 12
    assert st.harmonic_allocation(1, 7) == [7] and st.harmonic_allocation(0, 5) == []
    a = st.harmonic_allocation(9, 30)
    assert all(a[i] >= a[i + 1] for i in range(len(a) - 1)) and sum(a) <= 30      # monotone, within budget


def test_tree_invariants_on_random_tables():
    rng = np.random.default_rng(0)
    V, K = 200, 10
    for trial in range(200):
        adj = _table(V, K, rng)
        adj[rng.random(adj.shape) < 0.2] = -1                           # empty slots
        B = int(rng.choice([8, 16, 60, 128])); D = int(rng.integers(1, 7))
        m = int(rng.integers(0, 25)); d = rng.integers(0, V, m).tolist()
        r = float(rng.choice([0.15, 0.3, 0.5])); rho = 0.5
        tok, parent, spine, info = st.build_spine_tree(int(rng.integers(0, V)), d, adj, B, D, r, rho)
        n = len(tok)
        assert 1 <= n <= B and parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n))
        b_s = info["b_s"]
        assert spine[:b_s + 1] == [True] * (b_s + 1) and not any(spine[b_s + 1:])
        assert tok[1:b_s + 1] == d[:b_s] and all(parent[i] == i - 1 for i in range(1, b_s + 1))
        for p in range(n):                                               # no duplicate siblings
            kids = [tok[c] for c in range(n) if parent[c] == p]
            assert len(kids) == len(set(kids))
        for i in range(b_s + 1, n):                                      # a branch is at most D nodes from its fork
            dep, v = 0, i
            while not spine[v]:
                v = parent[v]; dep += 1
            assert 1 <= dep <= D
            assert tok[i] in [x for x in adj[tok[parent[i]]] if x >= 0]  # every branch token is a listed successor
        root_kids = [c for c in range(b_s + 1, n) if parent[c] == 0]
        assert len(root_kids) <= info["b_r"]
        for i in range(1, b_s + 1):
            assert len([c for c in range(b_s + 1, n) if parent[c] == i]) <= info["a"][i - 1]


def test_hand_worked_tree():
    """The hand-worked example fixes what the invariants above leave open: the chain is cut to floor(B r) nodes, the
    rank order of the attached successors, the duplicate skip taking the next-ranked entry without using up the
    allocation, a_i = 0, and step 4 extending the leaves breadth first, in creation order, by their TOP-ranked successor
    up to D nodes per branch."""
    ex = load_spine_tree_example()
    assert st.budget_split(len(ex["chain"]), ex["B"], ex["r"], ex["rho"]) == tuple(ex["budget"])
    assert st.harmonic_allocation(ex["budget"][0], ex["budget"][2]) == ex["alloc"]
    for D, tok, parent, n_spine in ex["cases"]:
        otok, opar, ospine, info = st.build_spine_tree(ex["anchor"], ex["chain"], ex["adj"], ex["B"], D, ex["r"], ex["rho"])
        assert otok == tok and opar == parent, D
        assert ospine == [True] * n_spine + [False] * (len(tok) - n_spine) and info["a"] == ex["alloc"]


def test_special_trees():
    rng = np.random.default_rng(1)
    adj = _table(50, 10, rng)
    # no context match: the spine vanishes, a transition-only tree remains (Sec. 4)
    tok, parent, spine, info = st.build_spine_tree(3, [], adj, 16, 6, 0.3, 0.5)
    assert info["b_s"] == 0 and spine == [True] + [False] * (len(tok) - 1) and len(tok) > 1
    # empty table: only the spine (a chain) remains
    empty = np.full((50, 10), -1, np.int32)
    tok, parent, spine, info = st.build_spine_tree(3, [4, 5, 6, 7, 8, 9], empty, 16, 6, 0.5, 0.5)
    assert tok == [3, 4, 5, 6, 7, 8, 9] and parent == [-1, 0, 1, 2, 3, 4, 5] and all(spine)
    # the spine continuation is not attached a second time as a branch
    adj2 = np.full((50, 3), -1, np.int32); adj2[3] = [4, 11, 12]
    tok, parent, spine, _ = st.build_spine_tree(3, [4], adj2, 8, 1, 0.5, 0.5)
    assert [tok[c] for c in range(len(tok)) if parent[c] == 0] == [4, 11, 12]


def test_context_match():
    ctx = [1, 2, 3, 4, 5, 6, 7, 1, 2, 3, 4, 5]
    d, c = st.context_match(ctx)
    assert d == [6, 7, 1, 2, 3, 4, 5] and c                             # all of n = 3, 4, 5 agree on token 6
    d, c = st.context_match([9, 8, 7, 6])
    assert d == [] and not c
    ctx = [5, 1, 2, 3, 9, 9, 4, 1, 2, 3, 7, 0, 1, 2, 3]
    d, c = st.context_match(ctx)                                        # only n = 3 matches; most recent occurrence wins
    assert d == [7, 0, 1, 2, 3] and not c
    d, _ = st.context_match(list(range(6)) * 10, max_len=20)
    assert d == [0, 1, 2, 3, 4, 5]                                      # most recent occurrence: the continuation ends with the context
    d, _ = st.context_match(list(range(30)) + [7, 8, 9, 10, 11], max_len=4)
    assert d == [12, 13, 14, 15]                                        # max_len caps the chain


def test_tiers_and_ema():
    assert [st.spine_ratio_tier(p) for p in (0.0, 0.19, 0.2, 0.39, 0.4, 0.9)] == [0.15, 0.15, 0.30, 0.30, 0.50, 0.50]
    p = 0.3                                                             # the paper's initial estimate
    for _ in range(5):
        p = st.ema_update(p, 9, 10)
    assert abs(p - (0.9 - 0.6 * 0.7 ** 5)) < 1e-12                      # EMA closed form, coefficient 0.3
    assert st.spine_ratio_tier(p) == 0.50                               # deepens the spine within 3-5 cycles
    assert st.ema_update(0.3, 0, 0) == 0.3
