"""GPU parity of the grouped-query workload: H query heads over Hkv key/value heads (query head h reads key/value
head h // (H // Hkv)) and a large vocabulary.  Same bars as the multi-head tests: attention within 1e-2 of the fp64
oracle per (sequence, node, head) row, integer results bit-exact."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth
from test_gpu_parity import ATTN_TOL, LSE_TOL, _check_attn_full, _check_step, _impl_ids, _impls, _run_attn, attn_row_err, goose  # noqa: F401

pytestmark = pytest.mark.gpu


def _tree(rng, B, kind):
    return {"chain": lambda: synth.chain_tree(B), "star": lambda: synth.star_tree(B),
            "kary3": lambda: synth.kary_tree(B, 3), "random": lambda: synth.random_tree(rng, B),
            "spine": lambda: synth.spine_tree(rng, B, max(1, B // 4), 3)[0]}[kind]()


# (H, Hkv, B): group sizes 1..16, trees that fill the 128-row tile exactly, leave it ragged, or need several tiles
# (B * g > 128), and a group size that does not divide 128
GQA_SHAPES = [(8, 2, 32), (8, 2, 16), (8, 2, 33), (8, 2, 128), (6, 2, 50), (16, 1, 20), (4, 4, 20), (2, 1, 64),
              (2, 1, 65), (32, 8, 32), (10, 2, 26), (12, 4, 1), (16, 1, 128), (64, 4, 128)]   # last two: the limits


@pytest.mark.parametrize("impl", _impls(), ids=_impl_ids())
@pytest.mark.parametrize("H,Hkv,B", GQA_SHAPES)
def test_gqa_attention_shapes(goose, oracle, impl, H, Hkv, B):
    rng = np.random.default_rng([H, Hkv, B])
    kinds = ["spine", "random", "kary3"] if B > 1 else ["chain"] * 3
    ctxs = [300, 0, 129]
    x = synth.make_inputs(3, H, B, ctxs, [_tree(rng, B, k) for k in kinds], V=8, with_logits=False,
                          seed=H * 1000 + Hkv * 100 + B, Hkv=Hkv)
    _check_attn_full(goose, oracle, x, impl)


@pytest.mark.parametrize("impl", _impls(), ids=_impl_ids())
def test_gqa_long_prefix_split_over_all_ctas(goose, oracle, impl):
    """One key/value head, two M tiles, a prefix long enough that every CTA holds a piece of each."""
    B, H = 40, 4
    x = synth.make_inputs(1, H, B, [30000], [synth.kary_tree(B, 3)], V=8, with_logits=False, seed=77, Hkv=1)
    out, lse, st = _run_attn(goose, x, impl)
    rng = np.random.default_rng(3)
    n = 24
    ss = np.zeros(n, np.int32); si = rng.integers(0, B, n).astype(np.int32); sh = rng.integers(0, H, n).astype(np.int32)
    si[:4] = [0, 31, 32, B - 1]                                # both sides of the M-tile boundary
    ref, ref_lse = oracle.tree_attn_rows(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, ss, si, sh)
    assert not st.any() and attn_row_err(out[ss, si, sh], ref).max() <= ATTN_TOL
    assert np.abs(lse[ss, si, sh] - ref_lse).max() <= LSE_TOL


def test_gqa_equals_multi_head_on_replicated_caches(goose):
    """The grouped kernel against the multi-head kernel run on caches whose heads are repeated in place: both go
    through the same arithmetic per row, so the outputs agree to the last bit of the bf16 output or one ulp of it
    (the split points of the key range differ, hence the order of the fp32 partial sums)."""
    from paper_2604_02047_b200 import binding
    rng = np.random.default_rng(9)
    H, Hkv, B = 8, 2, 32
    x = synth.make_inputs(2, H, B, [1000, 257], [synth.random_tree(rng, B), synth.chain_tree(B)], V=8,
                          with_logits=False, seed=12, Hkv=Hkv)
    d = binding.to_device(x)
    out_g, _ = goose.tree_attn_gqa(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], x.scale)
    k_rep = d["k_cache"].repeat_interleave(H // Hkv, dim=1).contiguous()
    v_rep = d["v_cache"].repeat_interleave(H // Hkv, dim=1).contiguous()
    out_m, _ = goose.tree_attn(d["q"], k_rep, v_rep, d["row_off"], d["ctx_len"], d["parent"], x.scale)
    torch.cuda.synchronize()
    a, b = out_g.float(), out_m.float()
    assert (a - b).abs().max() <= 2.0 ** -7 * b.abs().max()


def test_gqa_determinism_and_invalid_tree(goose):
    from paper_2604_02047_b200 import binding
    rng = np.random.default_rng(4)
    H, Hkv, B = 8, 2, 48                                       # two M tiles
    x = synth.make_inputs(2, H, B, [2000, 900], [synth.random_tree(rng, B), synth.random_tree(rng, B)], V=8,
                          with_logits=False, seed=8, Hkv=Hkv)
    a, la, _ = _run_attn(goose, x, binding.ATTN_UMMA)
    b, lb, _ = _run_attn(goose, x, binding.ATTN_UMMA)
    assert np.array_equal(a, b) and np.array_equal(la, lb)
    x.parent[1, 40] = 44                                       # parent[i] >= i, in the second M tile's nodes
    for impl in _impls():
        out, _, st = _run_attn(goose, x, impl)
        assert st.tolist() == [0, 1] and np.all(out[1] == 0) and np.abs(out[0]).max() > 0


def test_gqa_step_small_prefix_full_check(goose, oracle):
    """The gqa8b workload (32 query heads over 8 key/value heads, V = 128256) with the prefixes cut to 700 rows:
    every attention row, every top-k row, the walk and the compacted cache rows."""
    from paper_2604_02047_b200 import binding
    x = synth.make_config(5, seed=0, ctx_override=700)
    assert x.Hkv == 8 and x.H == 32 and x.V == 128256
    _check_step(goose, oracle, x)
    for impl in _impls():
        _check_attn_full(goose, oracle, x, impl)


def test_gqa_step_full_size(goose, oracle):
    x = synth.make_config(5, seed=0)
    _check_step(goose, oracle, x)


def test_gqa_step_host_buffers(goose, oracle):
    x = synth.make_inputs(2, 8, 20, [100, 260], [synth.kary_tree(20, 3), synth.chain_tree(20)], V=40000, seed=6, Hkv=2)
    _check_step(goose, oracle, x, host=True)


def test_gqa_argument_errors(goose):
    from paper_2604_02047_b200 import binding
    x = synth.make_inputs(1, 6, 8, [50], [synth.chain_tree(8)], V=8, with_logits=False, seed=1, Hkv=3)
    d = binding.to_device(x)
    with pytest.raises(binding.GooseError):                    # multi-head entry point with grouped caches
        goose.tree_attn(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], x.scale)
    bad = torch.zeros((58, 4, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.GooseError):                    # 6 query heads over 4 key/value heads
        goose.tree_attn_gqa(d["q"], bad, bad, d["row_off"], d["ctx_len"], d["parent"], x.scale)
    q34 = torch.zeros((1, 8, 34, 128), dtype=torch.bfloat16, device="cuda")
    kv1 = torch.zeros((58, 1, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.GooseError):                    # group of 34 > GOOSE_MAX_GROUP
        goose.tree_attn_gqa(q34, kv1, kv1, d["row_off"], d["ctx_len"], d["parent"], x.scale)
