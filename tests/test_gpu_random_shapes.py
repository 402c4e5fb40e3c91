"""Seeded random shapes against the oracle: top-k over random (rows, V, row stride, k, tie density) and tree attention
over random (query heads, key/value heads, tree size and shape, batch, prefix lengths).  The fixed-shape tests pin the
corners; these sweep the partition arithmetic of the persistent kernels (items per CTA, rows across CTA ranges, M tiles,
ragged tiles) with many combinations nobody wrote down."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth
from test_gpu_parity import ATTN_TOL, attn_row_err, goose  # noqa: F401

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
                assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 3e-3, where
        finally:
            goose.set_attn_impl(binding.ATTN_AUTO)
