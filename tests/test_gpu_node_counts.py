"""Per-sequence node counts on the GPU: one batch whose sequences carry trees of B, 1, 17, 0 and B - 1 nodes, everything
that belongs to a node that does not exist poisoned (NaN in q, K/V rows and logits rows, garbage parents and tokens),
against the oracle with the same n_nodes.  Outputs of absent nodes must keep the sentinel they held before the call."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth
from test_gpu_parity import ATTN_TOL, LSE_TOL, _impl_ids, _impls, attn_row_err, goose  # noqa: F401

pytestmark = pytest.mark.gpu
NAN16 = 0x7FC0


def _mixed_batch(B=32, H=4, Hkv=None, V=2048, k=8, seed=11, ctxs=(300, 0, 129, 77, 1000)):
    rng = np.random.default_rng(seed)
    S = len(ctxs)
    parents = [synth.spine_tree(rng, B, max(2, B // 4), 3)[0] if s % 2 == 0 else synth.random_tree(rng, B) for s in range(S)]
    x = synth.make_inputs(S, H, B, list(ctxs), parents, V=V, k=k, seed=seed, p_spine=0.9, p_branch=0.5,
                          is_spine=np.ones((S, B), bool), Hkv=Hkv)
    n_nodes = np.array([B, 1, min(17, B), 0, B - 1][:S], np.int32)
    for s in range(S):                                       # poison what belongs to nodes that do not exist
        n = int(n_nodes[s])
        x.q[s, n:] = NAN16; x.parent[s, n:] = 99; x.draft_tok[s, n:] = 12345
        r = int(x.row_off[s]) + int(x.ctx_len[s])
        x.k_cache[r + n:r + B] = NAN16; x.v_cache[r + n:r + B] = NAN16
        x.logits[s * B + n:(s + 1) * B] = NAN16
    return x, n_nodes


def _step_outputs_with_sentinels(goose, x):
    o = goose.alloc_step_outputs(x.S, x.B, x.H, x.D, x.k)
    o["out"].fill_(7.0); o["argmax"].fill_(-5); o["topk_ids"].fill_(-5); o["topk_vals"].fill_(-5.0)
    o["path"].fill_(-9); o["accept_len"].fill_(-9); o["bonus"].fill_(-9); o["new_ctx_len"].fill_(-9)
    o["lse"] = torch.full((x.S, x.B, x.H), 7.0, dtype=torch.float32, device="cuda")
    return o


def _check_against_oracle(oracle, x, n_nodes, o, d, check_cache=True, untouched=True):
    from paper_2604_02047_b200 import binding
    B, S = x.B, x.S
    ram, rids, rvals = oracle.node_topk(x.logits, x.k, n_nodes=n_nodes, B=B)
    rp, rl, rb = oracle.accept(x.draft_tok, x.parent, ram.reshape(S, B), n_nodes=n_nodes)
    rk, rv, rn = oracle.kv_compact(x.k_cache, x.v_cache, x.row_off, x.ctx_len, rp, rl, n_nodes=n_nodes)
    ref, ref_lse = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, n_nodes=n_nodes)
    got = o["out"].float().cpu().numpy().astype(np.float64)
    am, ids, vals = o["argmax"].cpu().numpy(), o["topk_ids"].cpu().numpy(), o["topk_vals"].cpu().numpy()
    for s in range(S):
        n = int(n_nodes[s])
        rows = slice(s * B, s * B + n)
        assert np.array_equal(am[rows], ram[rows]) and np.array_equal(ids[rows], rids[rows]), s
        assert np.array_equal(vals[rows].astype(np.float64), rvals[rows]), s
        if untouched:                                        # rows of nodes that do not exist keep what they held
            assert np.all(am[s * B + n:(s + 1) * B] == -5) and np.all(ids[s * B + n:(s + 1) * B] == -5)
            assert np.all(got[s, n:] == 7.0), s
        if n:
            assert np.isfinite(got[s, :n]).all()
            assert attn_row_err(got[s, :n], ref[s, :n]).max() <= ATTN_TOL, s
            if "lse" in o:
                assert np.abs(o["lse"][s, :n].cpu().numpy() - ref_lse[s, :n]).max() <= LSE_TOL
    assert np.array_equal(o["path"].cpu().numpy(), rp) and np.array_equal(o["accept_len"].cpu().numpy(), rl)
    assert np.array_equal(o["bonus"].cpu().numpy(), rb) and np.array_equal(o["new_ctx_len"].cpu().numpy(), rn)
    assert rl.max() >= 2 and rn[3] == x.ctx_len[3]
    if check_cache:
        gk, gv = binding.bf16_to_bits(d["k_cache"]), binding.bf16_to_bits(d["v_cache"])
        for s in range(S):
            r0, n = int(x.row_off[s]), int(rn[s])
            assert np.array_equal(gk[r0:r0 + n], rk[r0:r0 + n]) and np.array_equal(gv[r0:r0 + n], rv[r0:r0 + n])


@pytest.mark.parametrize("impl", _impls(), ids=_impl_ids())
def test_step_with_mixed_node_counts(goose, oracle, impl):
    from paper_2604_02047_b200 import binding
    x, n_nodes = _mixed_batch()
    d = binding.to_device(x)
    nn = torch.from_numpy(n_nodes).cuda()
    o = _step_outputs_with_sentinels(goose, x)
    goose.set_attn_impl(impl)
    try:
        goose.verify_step(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                          d["logits"], x.k, x.scale, outs=o, n_nodes=nn)
        torch.cuda.synchronize()
    finally:
        goose.set_attn_impl(binding.ATTN_AUTO)
    assert not goose.last_status(x.S).any()
    _check_against_oracle(oracle, x, n_nodes, o, d)


def test_step_with_mixed_node_counts_large_tree_long_prefix_and_grouped_heads(goose, oracle):
    """B = 128 (full tile), prefixes long enough that every CTA holds pieces of several heads, then the grouped-query form
    with two M tiles (B * g > 128), where a short tree leaves a whole M tile without rows."""
    from paper_2604_02047_b200 import binding
    for kw in (dict(B=128, H=8, V=32000, ctxs=(5000, 64, 3000, 900, 8000)),
               dict(B=48, H=8, Hkv=2, V=4096, ctxs=(2000, 10, 700, 300, 1500))):
        x, n_nodes = _mixed_batch(seed=21, **kw)
        d = binding.to_device(x)
        nn = torch.from_numpy(n_nodes).cuda()
        o = _step_outputs_with_sentinels(goose, x)
        call = goose.verify_step if x.Hkv == x.H else goose.verify_step_gqa
        call(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"], d["logits"],
             x.k, x.scale, outs=o, n_nodes=nn)
        torch.cuda.synchronize()
        assert not goose.last_status(x.S).any()
        _check_against_oracle(oracle, x, n_nodes, o, d)


def test_the_four_calls_with_node_counts(goose, oracle):
    """Stand-alone entry points, long rows for the top-k (three chunks per row, rows spread over CTAs)."""
    from paper_2604_02047_b200 import binding
    x, n_nodes = _mixed_batch(B=20, H=2, V=70000, k=5, seed=31)
    d = binding.to_device(x)
    nn = torch.from_numpy(n_nodes).cuda()
    B, S = x.B, x.S
    outs = (torch.full((S * B,), -5, dtype=torch.int32, device="cuda"), torch.full((S * B, x.k), -5, dtype=torch.int32, device="cuda"),
            torch.full((S * B, x.k), -5.0, dtype=torch.float32, device="cuda"))
    am, ids, vals = goose.node_topk(d["logits"], x.k, n_nodes=nn, B=B, outs=outs)
    ram, rids, rvals = oracle.node_topk(x.logits, x.k, n_nodes=n_nodes, B=B)
    for s in range(S):
        n = int(n_nodes[s]); rows = slice(s * B, s * B + n); rest = slice(s * B + n, (s + 1) * B)
        assert np.array_equal(am.cpu().numpy()[rows], ram[rows]) and np.array_equal(ids.cpu().numpy()[rows], rids[rows])
        assert np.array_equal(vals.cpu().numpy()[rows].astype(np.float64), rvals[rows])
        assert np.all(am.cpu().numpy()[rest] == -5) and np.all(ids.cpu().numpy()[rest] == -5)
    am_full = torch.from_numpy(ram.reshape(S, B)).cuda()
    p, l, b = goose.accept(d["draft_tok"], d["parent"], am_full, n_nodes=nn)
    rp, rl, rb = oracle.accept(x.draft_tok, x.parent, ram.reshape(S, B), n_nodes=n_nodes)
    assert np.array_equal(p.cpu().numpy(), rp) and np.array_equal(l.cpu().numpy(), rl) and np.array_equal(b.cpu().numpy(), rb)
    for impl in _impls():
        goose.set_attn_impl(impl)
        try:
            out = torch.full((S, B, x.H, 128), 7.0, dtype=torch.bfloat16, device="cuda")
            goose.tree_attn(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], x.scale, out=out, n_nodes=nn)
            torch.cuda.synchronize()
        finally:
            goose.set_attn_impl(binding.ATTN_AUTO)
        ref, _ = oracle.tree_attn(x.q, x.k_cache, x.v_cache, x.row_off, x.ctx_len, x.parent, x.scale, n_nodes=n_nodes)
        got = out.float().cpu().numpy().astype(np.float64)
        for s in range(S):
            n = int(n_nodes[s])
            assert np.all(got[s, n:] == 7.0) and (n == 0 or attn_row_err(got[s, :n], ref[s, :n]).max() <= ATTN_TOL)
    new_ctx = goose.kv_compact(d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], p, l, n_nodes=nn)
    rk, rv, rn = oracle.kv_compact(x.k_cache, x.v_cache, x.row_off, x.ctx_len, rp, rl, n_nodes=n_nodes)
    assert np.array_equal(new_ctx.cpu().numpy(), rn)
    gk = binding.bf16_to_bits(d["k_cache"])
    for s in range(S):
        r0, n = int(x.row_off[s]), int(rn[s])
        assert np.array_equal(gk[r0:r0 + n], rk[r0:r0 + n])
    assert not goose.last_status(S).any()


def test_host_buffer_step_and_harvest_with_node_counts(goose, oracle):
    from paper_2604_02047_b200 import binding
    x, n_nodes = _mixed_batch(B=16, H=4, V=1024, k=4, seed=41)
    d = binding.to_device(x)
    S, B = x.S, x.B
    # ---- harvest: rows of nodes that do not exist never reach the table
    nn = torch.from_numpy(n_nodes).cuda()
    adj_ids = torch.full((x.V, x.k), -1, dtype=torch.int32, device="cuda"); adj_sc = torch.zeros((x.V, x.k), device="cuda")
    dd = {k_: v.clone() for k_, v in d.items()}
    o = goose.verify_step_harvest(dd["q"], dd["k_cache"], dd["v_cache"], dd["row_off"], dd["ctx_len"], dd["parent"],
                                  dd["draft_tok"], dd["logits"], x.k, x.scale, adj_ids, adj_sc, n_nodes=nn)
    torch.cuda.synchronize()
    row_tok = x.draft_tok.copy()
    for s in range(S):
        row_tok[s, int(n_nodes[s]):] = -1                    # input preparation for the oracle: those rows are not harvested
    lg = x.logits.copy(); lg[lg == NAN16] = 0                # (the oracle's harvest computes every row's lse before it skips)
    rid, rsc, _ = oracle.harvest(lg, x.k, row_tok.reshape(-1), np.full((x.V, x.k), -1, np.int32), np.zeros((x.V, x.k)))
    assert np.array_equal(adj_ids.cpu().numpy(), rid)
    assert np.abs(adj_sc.cpu().numpy() - rsc).max() <= 1e-5 * max(1e-30, np.abs(rsc).max())
    # ---- host buffers
    houts = {k_: v.pin_memory() for k_, v in goose.alloc_step_outputs(S, B, x.H, x.D, x.k, device="cpu").items()}
    houts["out"].fill_(7.0); houts["argmax"].fill_(-5); houts["topk_ids"].fill_(-5)
    hin = {k_: v.cpu().pin_memory() for k_, v in d.items()}
    rows = np.concatenate([np.arange(x.row_off[s] + x.ctx_len[s], x.row_off[s] + x.ctx_len[s] + B) for s in range(S)])
    rows_t = torch.from_numpy(rows).cuda()
    k_new = d["k_cache"][rows_t].reshape(S, B, x.Hkv, x.D).cpu().pin_memory()
    v_new = d["v_cache"][rows_t].reshape(S, B, x.Hkv, x.D).cpu().pin_memory()
    goose.verify_step_host(d["k_cache"], d["v_cache"], hin["q"], k_new, v_new, hin["row_off"], hin["ctx_len"], hin["parent"],
                           hin["draft_tok"], hin["logits"], x.k, x.scale, houts, h_n_nodes=torch.from_numpy(n_nodes))
    assert not goose.last_status(S).any()
    ho = {k_: v.cuda() for k_, v in houts.items()}
    # (the host-buffer call copies whole output arrays back: rows of absent nodes are unspecified there)
    _check_against_oracle(oracle, x, n_nodes, ho, d, untouched=False)
    with pytest.raises(binding.GooseError):                  # host data: validated on the host
        goose.verify_step_host(d["k_cache"], d["v_cache"], hin["q"], k_new, v_new, hin["row_off"], hin["ctx_len"], hin["parent"],
                               hin["draft_tok"], hin["logits"], x.k, x.scale, houts,
                               h_n_nodes=torch.tensor([B + 1, 1, 1, 1, 1], dtype=torch.int32))


def test_node_count_outside_the_tree_is_flagged_and_the_sequence_skipped(goose, oracle):
    from paper_2604_02047_b200 import binding
    x, n_nodes = _mixed_batch(B=16, H=2, V=256, k=4, seed=51)
    d = binding.to_device(x)
    bad = n_nodes.copy(); bad[2] = x.B + 3; bad[4] = -1      # device data: read as 0, reported
    o = _step_outputs_with_sentinels(goose, x)
    goose.verify_step(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                      d["logits"], x.k, x.scale, outs=o, n_nodes=torch.from_numpy(bad).cuda())
    torch.cuda.synchronize()
    assert goose.last_status(x.S).tolist() == [0, 0, 16, 0, 16]
    as_zero = n_nodes.copy(); as_zero[2] = 0; as_zero[4] = 0
    _, rl, _ = oracle.accept(x.draft_tok, x.parent, oracle.node_topk(x.logits, x.k, n_nodes=as_zero, B=x.B)[0].reshape(x.S, x.B),
                             n_nodes=as_zero)
    assert np.array_equal(o["accept_len"].cpu().numpy(), rl)
    assert o["new_ctx_len"].cpu().tolist()[2] == int(x.ctx_len[2]) and torch.all(o["out"][2] == 7.0)
