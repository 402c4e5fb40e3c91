"""Several verification steps enqueued back to back on one stream with NO host synchronisation in between: step t+1
consumes step t's new_ctx_len (a device array) and the cache step t compacted.  This is the situation the kernels' reads
ahead of their dependency wait were argued for (the top-k streams the step's logits early, the walk/compaction launch
loads parent[], the draft tokens, ctx_len[] and row_off[] early), so the results of all steps are compared with the
oracle run step by step.  new_ctx_len must not alias ctx_len (rejected on the host): the steps ping-pong two arrays."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth
from test_gpu_parity import ATTN_TOL, attn_row_err, goose  # noqa: F401

pytestmark = pytest.mark.gpu


def _bf16(a, dev="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(dev)


def _draw_steps(n_steps, S, H, B, V, k, trees, seed, full_accept):
    """Per-step inputs: make_inputs with an empty prefix draws q, the B tree rows of K/V, tokens and planted logits."""
    steps = []
    for t in range(n_steps):
        parents = [trees(t, s) for s in range(S)]
        sp = np.ones((S, B), bool) if full_accept else None
        steps.append(synth.make_inputs(S, H, B, [0] * S, parents, V=V, k=k, seed=seed + t, is_spine=sp,
                                       p_spine=1.0 if full_accept else 0.8, p_branch=0.5))
    return steps


def _run_chain(goose, oracle, S, H, B, V, k, ctx0, trees, seed, full_accept, prewrite):
    n_steps = 3
    steps = _draw_steps(n_steps, S, H, B, V, k, trees, seed, full_accept)
    cap = np.asarray(ctx0, np.int64) + n_steps * B + 8                  # rows per sequence: room for every step's tree
    row_off = np.concatenate([[0], np.cumsum(cap)[:-1]]).astype(np.int64)
    total = int(cap.sum())
    rng = np.random.default_rng(seed)
    ck = synth.normal_bf16(rng, (total, H, 128)); cv = synth.normal_bf16(rng, (total, H, 128))
    scale = steps[0].scale

    # ---- oracle, step by step on the host
    ref = []
    ok_, ov_, ctx = ck.copy(), cv.copy(), np.asarray(ctx0, np.int32).copy()
    for x in steps:
        for s in range(S):
            r = int(row_off[s]) + int(ctx[s])
            ok_[r:r + B] = x.k_cache[s * B:(s + 1) * B]; ov_[r:r + B] = x.v_cache[s * B:(s + 1) * B]
        out, _ = oracle.tree_attn(x.q, ok_, ov_, row_off, ctx, x.parent, scale, want_lse=False)
        am, ids, vals = oracle.node_topk(x.logits, k)
        path, alen, bonus = oracle.accept(x.draft_tok, x.parent, am.reshape(S, B))
        ok_, ov_, new_ctx = oracle.kv_compact(ok_, ov_, row_off, ctx, path, alen)
        ref.append(dict(out=out, argmax=am, ids=ids, path=path, alen=alen, bonus=bonus, new_ctx=new_ctx, ctx=ctx.copy()))
        ctx = new_ctx
    if full_accept:
        assert all((r["alen"] == B - 1).all() for r in ref)

    # ---- GPU: everything enqueued on the current stream, one synchronisation at the very end
    dk, dv = _bf16(ck), _bf16(cv)
    d_off = torch.from_numpy(row_off).cuda()
    ctx_bufs = [torch.from_numpy(np.asarray(ctx0, np.int32)).cuda(), torch.zeros(S, dtype=torch.int32, device="cuda")]
    dev = [dict(q=_bf16(x.q), kn=_bf16(x.k_cache).view(S, B, H, 128), vn=_bf16(x.v_cache).view(S, B, H, 128),
                parent=torch.from_numpy(x.parent).cuda(), tok=torch.from_numpy(x.draft_tok).cuda(),
                logits=_bf16(x.logits)) for x in steps]
    outs = [goose.alloc_step_outputs(S, B, H, 128, k) for _ in steps]
    ar = torch.arange(B, device="cuda")
    if prewrite:                                                        # rows known up front (every chain is accepted whole)
        for t, d in enumerate(dev):
            for s in range(S):
                r = int(row_off[s]) + int(ctx0[s]) + t * B
                dk[r:r + B] = d["kn"][s]; dv[r:r + B] = d["vn"][s]
    torch.cuda.synchronize()
    for t, d in enumerate(dev):
        cur, nxt = ctx_bufs[t & 1], ctx_bufs[(t + 1) & 1]
        if not prewrite:                                                # the caller's K/V append, addressed on the device
            rows = (d_off[:, None] + cur[:, None].long() + ar[None, :]).reshape(-1)
            dk.index_copy_(0, rows, d["kn"].reshape(S * B, H, 128)); dv.index_copy_(0, rows, d["vn"].reshape(S * B, H, 128))
        o = outs[t]; o["new_ctx_len"] = nxt
        goose.verify_step(d["q"], dk, dv, d_off, cur, d["parent"], d["tok"], d["logits"], k, scale, outs=o)
    torch.cuda.synchronize()
    assert not goose.last_status(S).any()
    for t, (r, o) in enumerate(zip(ref, outs)):
        assert np.array_equal(o["argmax"].cpu().numpy(), r["argmax"]) and np.array_equal(o["topk_ids"].cpu().numpy(), r["ids"]), t
        assert np.array_equal(o["path"].cpu().numpy(), r["path"]) and np.array_equal(o["accept_len"].cpu().numpy(), r["alen"]), t
        assert np.array_equal(o["bonus"].cpu().numpy(), r["bonus"]), t
        got = o["out"].float().cpu().numpy().astype(np.float64)
        assert attn_row_err(got, r["out"]).max() <= ATTN_TOL, t
    assert np.array_equal(ctx_bufs[n_steps & 1].cpu().numpy(), ref[-1]["new_ctx"])
    from paper_2604_02047_b200 import binding
    gk, gv = binding.bf16_to_bits(dk), binding.bf16_to_bits(dv)
    for s in range(S):                                                  # the cache after three compactions, rows < new_ctx
        r0, n = int(row_off[s]), int(ref[-1]["new_ctx"][s])
        assert np.array_equal(gk[r0:r0 + n], ok_[r0:r0 + n]) and np.array_equal(gv[r0:r0 + n], ov_[r0:r0 + n])
    return ref


def test_three_steps_without_host_sync_random_trees(goose, oracle):
    rng = np.random.default_rng(3)
    S, H, B, V, k = 3, 4, 24, 2048, 8
    trees = lambda t, s: synth.spine_tree(rng, B, 8, 3)[0]
    ref = _run_chain(goose, oracle, S, H, B, V, k, [300, 5, 1100], trees, seed=50, full_accept=False, prewrite=False)
    assert any(r["alen"].max() > 0 for r in ref)                        # something was accepted, so rows did move


def test_three_steps_back_to_back_fully_accepted_chains(goose, oracle):
    """Chains accepted whole: step t+1's rows sit right behind step t's, so all tree rows are in place before the first
    launch and the twelve kernels of the three steps follow one another with nothing in between."""
    S, H, B, V, k = 2, 8, 16, 4096, 4
    _run_chain(goose, oracle, S, H, B, V, k, [700, 129], lambda t, s: synth.chain_tree(B), seed=60, full_accept=True,
               prewrite=True)


def test_new_ctx_len_must_not_alias_ctx_len(goose):
    from paper_2604_02047_b200 import binding
    x = synth.make_inputs(1, 2, 8, [40], [synth.chain_tree(8)], V=64, seed=1)
    d = binding.to_device(x)
    o = goose.alloc_step_outputs(1, 8, 2, 128, 4)
    o["new_ctx_len"] = d["ctx_len"]
    with pytest.raises(binding.GooseError):
        goose.verify_step(d["q"], d["k_cache"], d["v_cache"], d["row_off"], d["ctx_len"], d["parent"], d["draft_tok"],
                          d["logits"], 4, x.scale, outs=o)
    lib = goose.lib
    import ctypes
    path = torch.zeros((1, 8), dtype=torch.int32, device="cuda"); alen = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.goose_kv_compact(goose.h, binding._p(d["k_cache"]), binding._p(d["v_cache"]), ctypes.c_int64(48),
                              binding._p(d["row_off"]), binding._p(d["ctx_len"]), binding._p(path), binding._p(alen),
                              binding._p(None), ctypes.c_int(1), ctypes.c_int(8), ctypes.c_int(2), ctypes.c_int(128),
                              binding._p(d["ctx_len"]), binding._stream())
    assert rc == -1
