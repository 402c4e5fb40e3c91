"""End to end: the Goose decoding loop (Algorithm 2) driven by the library must emit exactly the tokens of
greedy autoregressive decoding (losslessness), on a synthetic deterministic target whose logits depend on the
last two tokens.  Every cycle uses the host routines (ContextMatch, BuildSpineTree, tiers/EMA), the verification
step on the GPU (tree attention over a growing KV cache, top-k, acceptance walk, compaction, with ctx_len chained
on the device) and the harvest into the adjacency table.  The KV cache must stay equal to the cache a sequential
decode of the same tokens would hold."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

V, K, B, D_MAX, H, HD = 512, 8, 32, 6, 2, 128


class ToyTarget:
    """logits(prev, cur) = noise[cur] + 10 at favoured(prev, cur): a bigram model with a small common vocabulary,
    so that generated text repeats (context matches exist) and transitions are learnable."""

    def __init__(self, seed=0):
        g = torch.Generator().manual_seed(seed)
        self.noise = torch.randn((V, V), generator=g).to(torch.bfloat16).cuda()
        self.kv = torch.randn((V, 2, H, HD), generator=g).to(torch.bfloat16).cuda()     # per-token K and V

    @staticmethod
    def favoured(prev, cur):
        return (cur * 7 + (prev % 3) * 5 + 1) % 23 if cur % 11 else (prev * 3 + cur + 2) % 40

    def logits(self, prev, cur):
        """prev, cur: int64 tensors [n] -> bf16 [n][V] (test-side model, not part of the library)."""
        rows = self.noise[cur.clamp(min=0)].float()
        fav = torch.tensor([self.favoured(int(p), int(c)) for p, c in zip(prev.tolist(), cur.tolist())], device="cuda")
        rows[torch.arange(len(cur), device="cuda"), fav] += 10.0
        return rows.to(torch.bfloat16)

    def kv_rows(self, tok, pos):
        """K and V rows of tokens at positions: bf16 [n][H][HD] each, a deterministic function of (token, position)."""
        t = self.kv[tok.clamp(min=0) % V]
        shift = (pos % 7).to(torch.bfloat16).view(-1, 1, 1) * 0.25
        return (t[:, 0] + shift).contiguous(), (t[:, 1] - shift).contiguous()


def greedy_ar(model, prompt, n_new):
    y = list(prompt)
    for _ in range(n_new):
        lg = model.logits(torch.tensor([y[-2]], device="cuda"), torch.tensor([y[-1]], device="cuda"))
        y.append(int(np.argmax(lg.float().cpu().numpy()[0])))
    return y


def test_goose_loop_is_lossless_and_keeps_the_cache_consistent():
    from paper_2604_02047_b200 import binding, build
    build.build()
    lib = binding.load_library()
    g = binding.Goose(max_S=1, max_B=B, max_H=H)
    model = ToyTarget()
    prompt = [3, 17, 4, 9, 30, 2, 5, 12]
    n_new = 160
    ref = greedy_ar(model, prompt, n_new + B)                             # the last cycle may overshoot n_new

    cap = len(prompt) + n_new + 2 * B
    k_cache = torch.zeros((cap, H, HD), dtype=torch.bfloat16, device="cuda")
    v_cache = torch.zeros_like(k_cache)
    adj_ids = torch.full((V, K), -1, dtype=torch.int32, device="cuda")
    adj_sc = torch.zeros((V, K), dtype=torch.float32, device="cuda")
    row_off = torch.zeros(1, dtype=torch.int64, device="cuda")

    # prefill: cache of the prompt except its last token (the first anchor), table from the prompt's logits
    y = list(prompt)
    pt = torch.tensor(prompt, device="cuda")
    kp, vp = model.kv_rows(pt[:-1], torch.arange(len(prompt) - 1, device="cuda"))
    k_cache[:len(prompt) - 1] = kp; v_cache[:len(prompt) - 1] = vp
    pl = model.logits(pt[:-2], pt[1:-1])
    g.harvest(pl, K, pt[1:-1].to(torch.int32), adj_ids, adj_sc)
    ctx_len = torch.tensor([len(prompt) - 1], dtype=torch.int32, device="cuda")

    p_hat, cycles, modes = 0.3, 0, {"bypass": 0, "tree": 0, "ar": 0}
    scale = 1.0 / np.sqrt(HD)
    while len(y) < len(prompt) + n_new:
        ctx = len(y) - 1
        assert int(ctx_len.item()) == ctx                                  # chained on the device from the last step
        anchor = y[-1]
        d, consensus = binding.context_match(y, 20)
        table = adj_ids.cpu().numpy()
        if d and (len(d) >= 8 or consensus):                               # bypass: verify the chain linearly
            chain = d[:B - 1]
            tok = np.array([anchor] + chain, np.int32); par = np.arange(-1, len(chain), dtype=np.int32)
            n, n_spine = len(tok), len(tok)
            tok = np.concatenate([tok, np.zeros(B - n, np.int32)]); par = np.concatenate([par, np.zeros(B - n, np.int32)])
            assert lib.goose_pad_tree(tok.ctypes.data_as(__import__("ctypes").c_void_p),
                                      par.ctypes.data_as(__import__("ctypes").c_void_p), n, B) == 0
            modes["bypass"] += 1
        elif d or (table[anchor] >= 0).any():                              # spine tree
            r = float(lib.goose_spine_ratio_tier(p_hat))
            tok, par, sp, n, n_spine = binding.build_spine_tree(anchor, d, table, B, D_MAX, r, 0.5, pad=True)
            modes["tree"] += 1
        else:                                                              # autoregressive fallback: a root-only tree
            tok, par, sp, n, n_spine = binding.build_spine_tree(anchor, [], np.full((1, 1), -1, np.int32), B, 1, 0.3, 0.5, pad=True)
            modes["ar"] += 1
        # the "forward": K/V of the tree nodes at rows ctx+i, their logits rows
        depth = np.zeros(B, np.int64)
        for i in range(1, B):
            depth[i] = depth[par[i]] + 1
        tok_t = torch.from_numpy(tok).cuda().long()
        par_t = torch.from_numpy(par).cuda()
        prev = torch.where(par_t >= 0, tok_t[par_t.clamp(min=0).long()], torch.tensor(y[-2], device="cuda"))
        logits = model.logits(prev, tok_t)
        kn, vn = model.kv_rows(tok_t, torch.from_numpy(ctx + depth).cuda())
        k_cache[ctx:ctx + B] = kn; v_cache[ctx:ctx + B] = vn
        q = kn.unsqueeze(0).contiguous()                                   # any finite queries
        # one call per cycle: verify the tree and harvest the forward's logits (read once) into the table
        o = g.verify_step_harvest(q, k_cache, v_cache, row_off, ctx_len, par_t.view(1, B).contiguous(),
                                  torch.from_numpy(tok).cuda().view(1, B), logits, K, scale, adj_ids, adj_sc)
        torch.cuda.synchronize()
        assert torch.isfinite(o["out"].float()).all() and not g.last_status(1).any()
        L = int(o["accept_len"].item()); path = o["path"].cpu().numpy()[0]
        accepted = [int(tok[path[j]]) for j in range(1, L + 1)]
        assert all(path[j] < n for j in range(L + 1))                      # padding is never accepted
        y += accepted + [int(o["bonus"].item())]
        p_hat = float(lib.goose_spine_ema(p_hat, int(sum(1 for j in range(1, L + 1) if path[j] < n_spine)), n_spine - 1))
        ctx_len = o["new_ctx_len"]
        cycles += 1

    assert len(y) >= len(prompt) + n_new and y == ref[:len(y)]              # identical to greedy autoregressive output
    assert cycles < 0.6 * n_new and modes["tree"] > 0                      # speculation really saved target calls
    # the compacted cache is the sequential cache of the emitted tokens
    n_ctx = int(ctx_len.item())
    assert n_ctx == len(y) - 1
    toks = torch.tensor(y[:n_ctx], device="cuda")
    ke, ve = model.kv_rows(toks, torch.arange(n_ctx, device="cuda"))
    assert torch.equal(k_cache[:n_ctx], ke) and torch.equal(v_cache[:n_ctx], ve)
    g.close()
