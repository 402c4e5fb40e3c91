"""The C++ host routines of the loop (BuildSpineTree, ContextMatch, tiers) against the Python oracle.  CPU only."""
import numpy as np
import pytest

from _golden import load_spine_tree_example
from oracle import spine_tree as st


@pytest.fixture(scope="module")
def binding():
    from paper_2604_02047_b200 import binding as b, build
    build.build()
    b.load_library()
    return b


def test_build_spine_tree_matches_the_oracle(binding):
    rng = np.random.default_rng(0)
    V, K = 300, 10
    for trial in range(300):
        adj = np.stack([rng.permutation(V)[:K] for _ in range(V)]).astype(np.int32)
        adj[rng.random(adj.shape) < 0.25] = -1
        B = int(rng.choice([1, 2, 8, 16, 60, 64, 80, 128])); D = int(rng.integers(1, 8))
        m = int(rng.integers(0, 30)); d = rng.integers(0, V, m).astype(np.int32)
        r = float(rng.choice([0.15, 0.30, 0.50])); rho = float(rng.choice([0.25, 0.5, 0.75]))
        anchor = int(rng.integers(0, V))
        tok, par, sp, n, ns = binding.build_spine_tree(anchor, d, adj, B, D, r, rho)
        otok, opar, osp, info = st.build_spine_tree(anchor, d.tolist(), adj, B, D, r, rho)
        assert n == len(otok) and ns == info["b_s"] + 1
        assert tok.tolist() == otok and par.tolist() == opar and sp.tolist() == osp


def test_build_spine_tree_matches_the_hand_worked_example(binding):
    """goose_build_spine_tree against the tree worked out by hand from Algorithm 1 (not against the oracle)."""
    ex = load_spine_tree_example()
    for D, tok, parent, n_spine in ex["cases"]:
        gtok, gpar, gsp, n, ns = binding.build_spine_tree(ex["anchor"], ex["chain"], ex["adj"], ex["B"], D, ex["r"], ex["rho"])
        assert n == len(tok) and ns == n_spine, D
        assert gtok.tolist() == tok and gpar.tolist() == parent
        assert gsp.tolist() == [True] * n_spine + [False] * (n - n_spine)


def test_padding_nodes_can_never_be_accepted(binding, oracle):
    adj = np.full((20, 4), -1, np.int32); adj[3] = [5, 6, -1, 7]
    tok, par, sp, n, ns = binding.build_spine_tree(3, [9, 8], adj, 16, 3, 0.5, 0.5, pad=True)
    assert len(tok) == 16 and n < 16
    assert all(par[i] == 0 and tok[i] < 0 for i in range(n, 16)) and len(set(tok[n:].tolist())) == 16 - n
    assert oracle.check_parent(par)
    am = np.full(16, 9, np.int32); am[1] = 8                               # argmax follows the spine 3 -> 9 -> 8
    path, alen, bonus = oracle.accept(tok, par, am)
    assert path[0, :3].tolist() == [0, 1, 2] and alen[0] == 2


def test_context_match_matches_the_oracle(binding):
    rng = np.random.default_rng(1)
    for trial in range(500):
        L = int(rng.integers(0, 60)); voc = int(rng.choice([2, 3, 5, 50]))
        ctx = rng.integers(0, voc, L).tolist()
        max_len = int(rng.choice([0, 1, 8, 20]))
        d, c = binding.context_match(ctx, max_len)
        od, oc = st.context_match(ctx, max_len=max_len)
        assert d == od
        if max_len > 0:
            assert c == oc


def test_tiers_and_ema_match_the_oracle(binding):
    lib = binding.load_library()
    for p in np.linspace(0, 1, 101):
        assert abs(lib.goose_spine_ratio_tier(float(p)) - st.spine_ratio_tier(float(np.float32(p)))) < 1e-7
    p_c, p_o = 0.3, 0.3
    rng = np.random.default_rng(2)
    for _ in range(50):
        dr = int(rng.integers(0, 12)); ac = int(rng.integers(0, dr + 1))
        p_c = lib.goose_spine_ema(p_c, ac, dr); p_o = st.ema_update(p_o, ac, dr)
        assert abs(p_c - p_o) < 1e-5


def test_argument_errors(binding):
    lib = binding.load_library()
    import ctypes
    n = ctypes.c_int32()
    buf = (ctypes.c_int32 * 8)()
    buf2 = (ctypes.c_int32 * 8)()
    assert lib.goose_build_spine_tree(0, None, 0, None, 0, 0, 129, 6, ctypes.c_float(0.3), ctypes.c_float(0.5), buf, buf, None,
                                      ctypes.byref(n), None) == -1         # B > 128
    assert lib.goose_build_spine_tree(0, None, 0, None, 0, 0, 8, 6, ctypes.c_float(1.0), ctypes.c_float(0.5), buf, buf, None,
                                      ctypes.byref(n), None) == -1         # r must be in (0, 1)
    assert lib.goose_build_spine_tree(7, None, 0, None, 0, 0, 8, 6, ctypes.c_float(0.3), ctypes.c_float(0.5), buf, buf2, None,
                                      ctypes.byref(n), None) == 0 and n.value == 1 and buf[0] == 7 and buf2[0] == -1
