"""Plain Python oracle of the host side of Goose's loop.  TEST INFRASTRUCTURE ONLY.

Written from Algorithm 1 (BuildSpineTree), the ContextMatch paragraph after Algorithm 2, and the
hyper-parameter table (spine-ratio tiers, EMA coefficient, bypass threshold); pure Python loops,
no sharing with the C++ host routines of the library.

Readings where the paper leaves room (also listed in the design notes):
  * A(t) lists token t's successors in rank order; empty slots (id < 0) are skipped.
  * "Duplicate entries are excluded during attachment": a successor whose token already is a child of
    the node (for instance the spine continuation) is skipped, and the next-ranked one is taken.
  * Step 4 extends every branch leaf by its single top-scoring successor, level by level (breadth
    first) in creation order, while nodes remain in the budget; a branch is at most D nodes long
    measured from the spine/root node it hangs on.
  * Node order: spine 0..b_s, root branches, spine branches (spine index ascending, rank ascending),
    then the extensions in the order they are created; hence parent[i] < i.
  * ContextMatch: for each n in (5, 4, 3) the last n tokens are looked up at their most recent earlier
    occurrence that has a continuation; the draft chain is the continuation (at most max_len tokens)
    of the longest n that matched; consensus = at least two n's matched and agree on the first token.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def budget_split(m: int, B: int, r: float, rho: float) -> Tuple[int, int, int]:
    """Algorithm 1, lines 1-3."""
    b_s = min(m, int(B * r))
    b_r = int((B - 1 - b_s) * (1 - rho))
    b_rho = B - 1 - b_s - b_r
    return b_s, b_r, b_rho


def harmonic_allocation(b_s: int, b_rho: int) -> List[int]:
    """Algorithm 1, step 3: a_i = floor(b_rho * (1/i) / sum_{j=1..b_s} 1/j), i = 1..b_s."""
    if b_s == 0:
        return []
    H = sum(1.0 / j for j in range(1, b_s + 1))
    return [int(b_rho * (1.0 / i) / H) for i in range(1, b_s + 1)]


def build_spine_tree(t_anc: int, d: Sequence[int], adj_ids, B: int, D: int, r: float, rho: float):
    """Returns (tok, parent, is_spine, info).  adj_ids[t] = ranked successor ids of token t (negative = empty)."""
    m = len(d)
    b_s, b_r, b_rho = budget_split(m, B, r, rho)
    tok, parent, is_spine, depth = [int(t_anc)], [-1], [True], [0]     # depth = nodes from the fork, 0 on the spine
    children = {0: set()}

    def add(p: int, t: int, spine: bool, dep: int) -> int:
        tok.append(int(t)); parent.append(p); is_spine.append(spine); depth.append(dep)
        children[p].add(int(t)); children[len(tok) - 1] = set()
        return len(tok) - 1

    def successors(t: int):
        if t < 0 or t >= len(adj_ids):
            return []
        return [int(x) for x in adj_ids[t] if int(x) >= 0]

    spine_nodes = [0]
    for i in range(1, b_s + 1):                                          # step 1: the spine
        spine_nodes.append(add(spine_nodes[-1], d[i - 1], True, 0))
    branch_nodes: List[int] = []

    def attach(node: int, count: int):
        got = 0
        for t in successors(tok[node]):
            if got >= count or len(tok) >= B:
                break
            if t in children[node]:
                continue
            branch_nodes.append(add(node, t, False, 1)); got += 1

    attach(0, b_r)                                                       # step 2: root branches
    a = harmonic_allocation(b_s, b_rho)
    for i in range(1, b_s + 1):                                          # step 3: spine branches
        attach(spine_nodes[i], a[i - 1])
    frontier = list(branch_nodes)                                        # step 4: breadth-first extension
    while frontier and len(tok) < B:
        nxt = []
        for leaf in frontier:
            if len(tok) >= B:
                break
            if depth[leaf] >= D:
                continue
            for t in successors(tok[leaf]):
                if t not in children[leaf]:
                    nxt.append(add(leaf, t, False, depth[leaf] + 1))
                    break
        frontier = nxt
    return tok, parent, is_spine, {"b_s": b_s, "b_r": b_r, "b_rho": b_rho, "a": a}


def context_match(ctx: Sequence[int], ns=(5, 4, 3), max_len: int = 20) -> Tuple[List[int], bool]:
    chains = {}
    L = len(ctx)
    for n in ns:
        if L <= n:
            continue
        query = list(ctx[L - n:])
        for p in range(L - n - 1, -1, -1):                               # most recent earlier occurrence
            if list(ctx[p:p + n]) == query:
                chains[n] = list(ctx[p + n:p + n + max_len])
                break
    if not chains:
        return [], False
    best = chains[max(chains)]
    firsts = [c[0] for c in chains.values() if c]
    consensus = any(firsts.count(f) >= 2 for f in firsts)
    return best, consensus


def spine_ratio_tier(p_hat: float) -> float:
    """p_hat < 0.2 -> 0.15, < 0.4 -> 0.30, else 0.50."""
    return 0.15 if p_hat < 0.2 else (0.30 if p_hat < 0.4 else 0.50)


def ema_update(p_hat: float, accepted_spine: int, drafted_spine: int, coeff: float = 0.3) -> float:
    if drafted_spine <= 0:
        return p_hat
    return (1.0 - coeff) * p_hat + coeff * (accepted_spine / drafted_spine)
