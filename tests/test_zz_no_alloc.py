"""goose_node_topk_static: the top-k entry point for callers that must not allocate device memory.

It is checked against goose_node_topk (same kernel, context-owned scratch) on two calls in a row:
the static scratch array is shared by all calls and keeps the previous call's contents, so the second
call proves that nothing stale leaks into a result.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth

pytestmark = pytest.mark.gpu


def _bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def test_static_topk_matches_the_context_entry_point_twice():
    from paper_2604_02047_b200 import binding, build
    build.build()
    g = binding.Goose(max_S=1, max_B=128, max_H=8)
    rng = np.random.default_rng(5)
    # rows longer than one 32768-element chunk: this is the case that needs the scratch array
    for call, (rows, V, k) in enumerate([(37, 100000, 8), (64, 151936, 16)]):
        bits = synth.f32_to_bf16_bits(rng.standard_normal((rows, V), dtype=np.float32))
        bits[:, ::977] = bits[:, :1]                          # plant exact ties across chunks
        lg = _bf16(bits)
        ref = g.node_topk(lg, k)
        got = binding.node_topk_static(lg, k)
        torch.cuda.synchronize()
        for a, b in zip(got, ref):
            assert torch.equal(a, b), "call %d" % call        # bit-exact: ids, argmax and exact values
    # single-chunk rows do not touch the scratch but go through the same entry point
    x = synth.make_config(0)
    lg = _bf16(x.logits)
    for a, b in zip(binding.node_topk_static(lg, x.k), g.node_topk(lg, x.k)):
        assert torch.equal(a, b)
    g.close()


def test_static_topk_rejects_sizes_beyond_its_scratch():
    from paper_2604_02047_b200 import binding
    lg = torch.zeros((2049, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.GooseError):
        binding.node_topk_static(lg, 4)                       # rows > GOOSE_STATIC_TOPK_MAX_ROWS
    with pytest.raises(binding.GooseError):
        binding.node_topk_static(lg[:8], 17)                  # k > 16
