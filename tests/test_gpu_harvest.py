"""GPU parity of goose_harvest (top-k + row log-sum-exp + scatter into the Tier-1 adjacency table) against
the oracle: ids bit-exact, softmax scores within 1e-5 relative (fp32 sum of exp2 vs fp64), lse within 2e-5."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def goose():
    from paper_2604_02047_b200 import binding, build
    build.build()
    g = binding.Goose(max_S=16, max_B=128, max_H=8)
    yield g
    g.close()


def _bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def _check(goose, oracle, bits, k, tok, table_rows, V=None):
    ids0 = np.full((table_rows, k), -7, np.int32); sc0 = np.full((table_rows, k), -1.0, np.float32)
    adj_ids = torch.from_numpy(ids0).cuda(); adj_sc = torch.from_numpy(sc0).cuda()
    am, ids, vals, lse = goose.harvest(_bf16(bits), k, torch.from_numpy(np.asarray(tok, np.int32)).cuda(), adj_ids, adj_sc, V=V)
    torch.cuda.synchronize()
    rids, rsc, rlse = oracle.harvest(bits, k, tok, ids0, sc0.astype(np.float64), V=V)
    ram, rtop, rvals = oracle.node_topk(bits, k, V=V)
    assert np.array_equal(am.cpu().numpy(), ram) and np.array_equal(ids.cpu().numpy(), rtop)
    assert np.array_equal(vals.cpu().numpy().astype(np.float64), rvals)
    assert np.abs(lse.cpu().numpy().astype(np.float64) - rlse).max() <= 2e-5
    assert np.array_equal(adj_ids.cpu().numpy(), rids)                       # incl. untouched rows and last-writer rule
    got = adj_sc.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - rsc) <= 1e-5 * np.abs(rsc) + 1e-12)


def test_harvest_tree_logits(goose, oracle):
    for cid in (0, 1):
        x = synth.make_config(cid)
        _check(goose, oracle, x.logits, x.k, x.draft_tok.reshape(-1), x.V)


def test_harvest_duplicates_and_bad_tokens(goose, oracle):
    rng = np.random.default_rng(8)
    rows, V, k = 300, 4096, 10
    bits = synth.f32_to_bf16_bits((rng.standard_normal((rows, V)) * 2).astype(np.float32))
    tok = rng.integers(0, 60, rows).astype(np.int32)                          # heavy duplication: 60 tokens, 300 rows
    tok[5] = -1; tok[17] = V; tok[rows - 1] = tok[0]
    _check(goose, oracle, bits, k, tok, V)


def test_harvest_long_rows_and_row_stride(goose, oracle):
    rng = np.random.default_rng(9)
    rows, V, ldl, k = 9, 100001, 100008, 16                                   # four 32768-element chunks, ragged tail
    bits = synth.f32_to_bf16_bits(rng.standard_normal((rows, ldl), dtype=np.float32))
    bits[:, V:] = 0x7F00                                                     # padding must not enter the sums
    _check(goose, oracle, bits, k, np.arange(rows, dtype=np.int32) * 11111, V, V=V)
    const = np.full((2, 40000), 0x4040, np.uint16)                            # constant rows: slow path + lse = 3 + ln V
    _check(goose, oracle, const, 8, [1, 2], 40000)


def test_harvest_more_items_than_sms(goose, oracle):
    """Rows of three chunks, more items than SMs: the row log-sum-exp is merged over chunks inside a CTA and over CTAs."""
    rng = np.random.default_rng(31)
    rows, V, k = 200, 70000, 8
    bits = synth.f32_to_bf16_bits((rng.standard_normal((rows, V)) * 3).astype(np.float32))
    tok = rng.permutation(V)[:rows].astype(np.int32)
    _check(goose, oracle, bits, k, tok, V, V=V)


def test_step_with_harvest_equals_step_then_harvest(oracle):
    """goose_verify_step_harvest reads the logits once; its step outputs equal goose_verify_step's and its table equals
    goose_harvest's with row_tok = draft_tok, which in turn equals the oracle's."""
    from paper_2604_02047_b200 import binding, build
    build.build()
    g = binding.Goose(max_S=4, max_B=128, max_H=64)
    for x in (synth.make_config(0, seed=3),
              synth.make_inputs(3, 8, 20, [100, 7, 260], [synth.kary_tree(20, 3), synth.chain_tree(20), synth.star_tree(20)],
                                V=40000, seed=4, Hkv=2)):
        x.draft_tok[0, 1] = -5                                         # a padding-style token: its row is skipped
        d1, d2 = binding.to_device(x), binding.to_device(x)
        step = g.verify_step if x.Hkv == x.H else g.verify_step_gqa
        o1 = step(d1["q"], d1["k_cache"], d1["v_cache"], d1["row_off"], d1["ctx_len"], d1["parent"], d1["draft_tok"],
                  d1["logits"], x.k, x.scale)
        ids1 = torch.full((x.V, x.k), -7, dtype=torch.int32, device="cuda"); sc1 = torch.full((x.V, x.k), -1.0, device="cuda")
        g.harvest(d1["logits"], x.k, d1["draft_tok"].view(-1), ids1, sc1)
        ids2 = torch.full((x.V, x.k), -7, dtype=torch.int32, device="cuda"); sc2 = torch.full((x.V, x.k), -1.0, device="cuda")
        o2 = g.verify_step_harvest(d2["q"], d2["k_cache"], d2["v_cache"], d2["row_off"], d2["ctx_len"], d2["parent"],
                                   d2["draft_tok"], d2["logits"], x.k, x.scale, ids2, sc2)
        torch.cuda.synchronize()
        assert not g.last_status(x.S).any()
        for key in ("out", "argmax", "topk_ids", "topk_vals", "path", "accept_len", "bonus", "new_ctx_len"):
            assert torch.equal(o1[key], o2[key]), key
        assert torch.equal(d1["k_cache"], d2["k_cache"]) and torch.equal(d1["v_cache"], d2["v_cache"])
        assert torch.equal(ids1, ids2) and torch.equal(sc1, sc2)
        rids, rsc, rlse = oracle.harvest(x.logits, x.k, x.draft_tok.reshape(-1), np.full((x.V, x.k), -7, np.int32),
                                         np.full((x.V, x.k), -1.0, np.float64))
        assert np.array_equal(ids2.cpu().numpy(), rids)
        assert np.abs(sc2.cpu().numpy() - rsc).max() <= 1e-5 * max(1.0, np.abs(rsc).max())
        assert np.abs(o2["row_lse"].cpu().numpy() - rlse).max() <= 2e-5 * max(1.0, np.abs(rlse).max())
    g.close()


def test_harvest_argument_errors(goose):
    from paper_2604_02047_b200 import binding
    lg = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.GooseError):
        goose.harvest(lg, 17, tok, torch.zeros((64, 17), dtype=torch.int32, device="cuda"),
                      torch.zeros((64, 17), dtype=torch.float32, device="cuda"))


def test_step_with_harvest_argument_errors():
    """A harvest needs all of row_lse, adj_ids, adj_scores and topk_vals; nothing is enqueued otherwise."""
    import ctypes
    from paper_2604_02047_b200 import binding, build
    build.build()
    g = binding.Goose(max_S=1, max_B=128, max_H=64)
    x = synth.make_config(0, seed=5)
    d = binding.to_device(x)
    o = g.alloc_step_outputs(x.S, x.B, x.H, x.D, x.k, "cuda")
    lse = torch.empty(x.S * x.B, dtype=torch.float32, device="cuda")
    ids = torch.zeros((x.V, x.k), dtype=torch.int32, device="cuda"); sc = torch.zeros((x.V, x.k), device="cuda")
    P = binding._p

    def call(row_lse, adj_ids, adj_sc, vals, table_rows):
        return g.lib.goose_verify_step_harvest(
            g.h, P(d["q"]), P(d["k_cache"]), P(d["v_cache"]), ctypes.c_int64(d["k_cache"].shape[0]), P(d["row_off"]),
            P(d["ctx_len"]), P(d["parent"]), P(None), P(d["draft_tok"]), P(d["logits"]), ctypes.c_int64(x.V), ctypes.c_int(x.S),
            ctypes.c_int(x.B), ctypes.c_int(x.H), ctypes.c_int(x.H), ctypes.c_int(128), ctypes.c_int(x.V), ctypes.c_int(x.k),
            ctypes.c_float(x.scale), P(o["out"]), None, P(o["argmax"]), P(o["topk_ids"]), P(vals), P(o["path"]),
            P(o["accept_len"]), P(o["bonus"]), P(o["new_ctx_len"]), P(row_lse), ctypes.c_int(table_rows), P(adj_ids), P(adj_sc),
            ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))

    n0 = g.launch_count()
    assert call(lse, ids, None, o["topk_vals"], x.V) == -1          # scores missing
    assert call(None, ids, sc, o["topk_vals"], x.V) == -1           # row_lse missing
    assert call(lse, ids, sc, None, x.V) == -1                      # topk_vals missing
    assert call(lse, ids, sc, o["topk_vals"], 0) == -1              # empty table
    assert g.launch_count() == n0                                   # nothing was enqueued
    assert call(lse, ids, sc, o["topk_vals"], x.V) == 0
    assert call(None, None, None, None, 0) == 0                     # no harvest: the plain step, topk_vals optional
    torch.cuda.synchronize()
    g.close()
