"""Properties of the seeded input generator (no method arithmetic is tested here)."""
import numpy as np
import torch

from paper_2604_02047_b200 import synth


def test_bf16_rounding_matches_library():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(100000, dtype=np.float32) * np.float32(7.0)
    x[:4] = [0.0, -0.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]   # exact ties -> even
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    back = synth.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_tree_shapes_and_tokens():
    for cid, cfg in enumerate(synth.CONFIGS):
        _, ctxs, parents, spines, ps = synth.config_shapes(cid, seed=0)
        assert parents.shape == (cfg.S, cfg.B)
        for s in range(cfg.S):
            p = parents[s]
            assert p[0] == -1 and all(0 <= p[i] < i for i in range(1, cfg.B))
            n_sp = int(spines[s].sum())
            assert cfg.spine[0] <= n_sp <= cfg.spine[1]
            assert all(p[i] == i - 1 for i in range(1, n_sp))
            # branch chains hang on spine nodes and are at most branch_len_max deep
            for i in range(n_sp, cfg.B):
                d, v = 0, i
                while not spines[s][v]:
                    v = p[v]; d += 1
                assert 1 <= d <= cfg.branch_len_max
            assert cfg.ctx[0] <= ctxs[s] <= cfg.ctx[1]
            assert cfg.p_spine[0] <= ps[s] <= cfg.p_spine[1]


def test_config0_tensors_and_determinism():
    a = synth.make_config(0, seed=0)
    b = synth.make_config(0, seed=0)
    c = synth.make_config(0, seed=1)
    assert a.q.shape == (1, 16, 32, 128) and a.k_cache.shape == (512 + 16, 32, 128)
    assert a.logits.shape == (16, 32000) and a.logits.dtype == np.uint16
    for f in ("q", "k_cache", "v_cache", "logits", "draft_tok", "parent"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert not np.array_equal(a.q, c.q)
    # distinct sibling tokens
    for par in set(a.parent[0].tolist()):
        toks = a.draft_tok[0][a.parent[0] == par]
        assert len(set(toks.tolist())) == len(toks)
    # a planted child is worth about +10 in its parent's row
    lg = synth.bf16_bits_to_f32(a.logits)
    for i in range(1, a.B):
        v = lg[a.parent[0, i], a.draft_tok[0, i]]
        assert (v > 5.5) == bool(a.planted[0, i])
    # value distribution ~ N(0,1)
    kf = synth.bf16_bits_to_f32(a.k_cache)
    assert abs(kf.mean()) < 0.01 and abs(kf.std() - 1.0) < 0.01


def test_ragged_batch_layout():
    x = synth.make_inputs(3, 2, 8, [5, 0, 130], [synth.chain_tree(8), synth.star_tree(8), synth.kary_tree(8, 3)],
                          V=64, with_logits=True)
    assert x.row_off.tolist() == [0, 13, 21] and x.kv_rows == 13 + 8 + 138
    assert x.logits.shape == (24, 64)


def test_algorithmic_bytes_table():
    # the per-config byte counts the roofline is computed from
    exp = {0: 9.94e6, 1: 41.30e6, 2: 92.29e6, 3: 233.12e6}
    for cid, total in exp.items():
        cfg, ctxs, *_ = synth.config_shapes(cid)
        b = synth.algorithmic_bytes(cfg.S, cfg.H, cfg.B, cfg.D, cfg.V, ctxs)
        assert abs(b["total"] - total) / total < 2e-3
