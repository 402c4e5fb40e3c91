"""Seeded random shapes against the oracle: top-k over random (rows, V, row stride, k, tie density) and tree attention
over random (query heads, key/value heads, tree size and shape, batch, prefix lengths).  The fixed-shape tests pin the
corners; these sweep the partition arithmetic of the persistent kernels (items per CTA, rows across CTA ranges, M tiles,
ragged tiles) with many combinations nobody wrote down."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth
from test_gpu_parity import ATTN_TOL, LSE_TOL, attn_row_err, goose  # noqa: F401

pytestmark = pytest.mark.gpu


def _bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_topk_random_shapes(goose, oracle, seed):
    rng = np.random.default_rng(seed)
    for it in range(12):
        V = int(rng.choice([rng.integers(1, 200), rng.integers(200, 40000), rng.integers(32000, 70000),
                            rng.integers(60000, 262145)]))
        rows = int(rng.integers(1, max(1, min(2048, int(3e7 // V))) + 1))
        k = int(rng.integers(1, min(16, V) + 1))
        ldl = (V + 7) // 8 * 8 + 8 * int(rng.integers(0, 3))
        x = rng.standard_normal((rows, ldl), dtype=np.float32)
        mode = it % 4
        if mode == 1:
            x = np.round(x * 2) / 2                            # exact ties
        if mode == 2:
            x = np.round(x)                                    # very heavy ties: the slow path on many items
        if mode == 3:
            x[rng.integers(0, rows, max(1, rows // 7))] = rng.integers(-3, 4)   # some constant rows
        bits = synth.f32_to_bf16_bits(x.astype(np.float32))
        bits[:, V:] = 0x7F00                                   # the padding behind V must be ignored
        am, ids, vals = goose.node_topk(_bf16(bits), k, V=V)
        ram, rids, rvals = oracle.node_topk(bits, k, V=V)
        where = "rows=%d V=%d ldl=%d k=%d mode=%d" % (rows, V, ldl, k, mode)
        assert np.array_equal(am.cpu().numpy(), ram), where
        assert np.array_equal(ids.cpu().numpy(), rids), where
        assert np.array_equal(vals.cpu().numpy().astype(np.float64), rvals), where


@pytest.mark.parametrize("seed", [21, 22])
def test_attention_random_shapes(goose, oracle, seed):
    from paper_2604_02047_b200 import binding
    rng = np.random.default_rng(seed)
    done = 0
    while done < 10:
        Hkv = int(rng.choice([1, 2, 3, 4, 8]))
        group = int(rng.choice([1, 1, 2, 3, 4, 8, 16]))
        H = Hkv * group
        if H > 64:
            continue
        done += 1
        B = int(rng.integers(1, 129))
        S = int(rng.integers(1, 5))
        ctxs = [int(rng.choice([0, rng.integers(1, 300), rng.integers(100, 3000)])) for _ in range(S)]
        trees = []
        for _ in range(S):
            kind = rng.choice(["chain", "star", "random", "spine"])
            trees.append({"chain": lambda: synth.chain_tree(B), "star": lambda: synth.star_tree(B),
                          "random": lambda: synth.random_tree(rng, B),
                          "spine": lambda: synth.spine_tree(rng, B, max(1, B // 4), 3)[0]}[kind]())
        x = synth.make_inputs(S, H, B, ctxs, trees, V=8, with_logits=False, seed=int(rng.integers(1 << 30)), Hkv=Hkv,
                              q_gain=float(rng.choice([1.0, 1.0, 6.0])))
        d = binding.to_device(x)
        ref, ref_lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
        where = "H=%d Hkv=%d B=%d S=%d ctx=%s" % (H, Hkv, B, S, ctxs)
        try:
            for impl in (binding.ATTN_MMA, binding.ATTN_UMMA):
                goose.set_attn_impl(impl)
                out, lse = goose.tree_attn_gqa(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"],
                                               x.scale, want_lse=True)
                torch.cuda.synchronize()
                assert not goose.last_status(S).any(), where
                got = out.float().cpu().numpy().astype(np.float64)
                assert attn_row_err(got, ref).max() <= ATTN_TOL, where
                assert np.abs(lse.cpu().numpy() - ref_lse).max() <= LSE_TOL, where
        finally:
            goose.set_attn_impl(binding.ATTN_AUTO)


@pytest.mark.parametrize("seed", [31, 32])
def test_step_with_harvest_random_shapes(oracle, seed):
    """The whole step plus harvest on random batches (multi-head and grouped, 1-5 sequences, tree sizes 2-128, vocabularies
    64-70000, k 1-16, a few padding-style negative tokens): every integer result and the compacted cache rows bit-exact,
    table scores within 1e-5, attention within the usual bar."""
    from paper_2604_02047_b200 import binding, build
    build.build()
    g = binding.Goose(max_S=8, max_B=128, max_H=64)
    rng = np.random.default_rng(seed)
    for _ in range(6):
        Hkv = int(rng.choice([1, 2, 4, 8])); H = Hkv * int(rng.choice([1, 1, 2, 4]))
        B = int(rng.integers(2, 129)); S = int(rng.integers(1, 6))
        V = (int(rng.choice([64, 1000, 4096, 32000, 50000, 70000])) + 7) // 8 * 8
        k = min(int(rng.integers(1, 17)), V)
        ctxs = [int(rng.choice([0, rng.integers(1, 200), rng.integers(100, 1500)])) for _ in range(S)]
        trees = [synth.spine_tree(rng, B, max(1, B // int(rng.integers(2, 6))), 3) for _ in range(S)]
        x = synth.make_inputs(S, H, B, ctxs, [t[0] for t in trees], V=V, k=k, seed=int(rng.integers(1 << 30)), Hkv=Hkv,
                              is_spine=[t[1] for t in trees], p_spine=0.8, p_branch=0.3)
        for s in range(S):
            for i in rng.integers(1, B, 2):
                x.draft_tok[s, i] = -1 - int(i)                 # never matched, never harvested
        where = "S=%d B=%d H=%d Hkv=%d V=%d k=%d ctx=%s" % (S, B, H, Hkv, V, k, ctxs)
        d = binding.to_device(x)
        ids = torch.full((V, k), -7, dtype=torch.int32, device="cuda"); sc = torch.full((V, k), -1.0, device="cuda")
        o = g.verify_step_harvest(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                                  d["logits"], k, x.scale, ids, sc)
        torch.cuda.synchronize()
        assert not g.last_status(S).any(), where
        ram, rids, _ = oracle.node_topk(x.logits, k)
        rp, rl, rb = oracle.accept(x.draft_tok, x.parent, ram.reshape(S, B))
        rk, rv, rn = oracle.kv_compact(x.k_cache, x.v_cache, x.row_off, x.ctx_len, rp, rl)
        hids, hsc, _ = oracle.harvest(x.logits, k, x.draft_tok.reshape(-1), np.full((V, k), -7, np.int32), np.full((V, k), -1.0))
        ref, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale)
        assert np.array_equal(o["argmax"].cpu().numpy(), ram) and np.array_equal(o["topk_ids"].cpu().numpy(), rids), where
        assert np.array_equal(o["path"].cpu().numpy(), rp) and np.array_equal(o["accept_len"].cpu().numpy(), rl), where
        assert np.array_equal(o["bonus"].cpu().numpy(), rb) and np.array_equal(o["new_ctx_len"].cpu().numpy(), rn), where
        gk, gv = binding.bf16_to_bits(d["k_cache"]), binding.bf16_to_bits(d["v_cache"])
        for s in range(S):
            r0, n = int(x.row_off[s]), int(rn[s])
            assert np.array_equal(gk[r0:r0 + n], rk[r0:r0 + n]) and np.array_equal(gv[r0:r0 + n], rv[r0:r0 + n]), where
        assert np.array_equal(ids.cpu().numpy(), hids), where
        assert np.all(np.abs(sc.cpu().numpy() - hsc) <= 1e-5 * np.abs(hsc) + 1e-9), where
        got = o["out"].float().cpu().numpy().astype(np.float64)
        assert attn_row_err(got, ref).max() <= ATTN_TOL, where
    g.close()
