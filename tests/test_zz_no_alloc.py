"""goose_node_topk_static: the top-k entry point for callers that must not allocate device memory.

It is checked on two calls in a row against the fp64 oracle (bit-exact ids, argmax and values) and against
goose_node_topk (same kernel, context-owned scratch): the static scratch array is shared by all calls and
keeps the previous call's contents, so the second call proves that nothing stale leaks into a result.
A further test checks that a call leaves the amount of free device memory unchanged.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2604_02047_b200 import synth

pytestmark = pytest.mark.gpu


def _bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def _assert_equals_oracle(oracle, got, bits, k):
    ram, rids, rvals = oracle.node_topk(bits, k)
    am, ids, vals = got
    assert np.array_equal(am.cpu().numpy(), ram) and np.array_equal(ids.cpu().numpy(), rids)
    assert np.array_equal(vals.cpu().numpy().astype(np.float64), rvals)


def test_static_topk_matches_the_oracle_and_the_context_entry_point_twice(oracle):
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
        _assert_equals_oracle(oracle, got, bits, k)
    # single-chunk rows do not touch the scratch but go through the same entry point
    x = synth.make_config(0)
    lg = _bf16(x.logits)
    got = binding.node_topk_static(lg, x.k)
    for a, b in zip(got, g.node_topk(lg, x.k)):
        assert torch.equal(a, b)
    _assert_equals_oracle(oracle, got, x.logits, x.k)
    g.close()


def test_static_topk_leaves_free_device_memory_unchanged(oracle):
    """The point of the entry point: once its first call on the device has run, a call (multi-chunk rows, so the
    static scratch is in use) changes the free device memory by nothing.  The outputs are the caller's."""
    from paper_2604_02047_b200 import binding
    rng = np.random.default_rng(6)
    rows, V, k = 50, 70000, 8
    bits = synth.f32_to_bf16_bits(rng.standard_normal((rows, V), dtype=np.float32))
    lg = _bf16(bits)
    binding.node_topk_static(lg, k)                           # first call on this device: set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    lib = binding.load_library()
    import ctypes
    am = torch.empty(rows, dtype=torch.int32, device="cuda")
    ids = torch.empty((rows, k), dtype=torch.int32, device="cuda")
    vals = torch.empty((rows, k), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    rc = lib.goose_node_topk_static(binding._p(lg), ctypes.c_int(rows), ctypes.c_int(V), ctypes.c_int64(V), ctypes.c_int(k),
                                    binding._p(am), binding._p(ids), binding._p(vals), binding._stream())
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert rc == 0 and free1 == free0
    _assert_equals_oracle(oracle, (am, ids, vals), bits, k)


def test_static_topk_rejects_sizes_beyond_its_scratch():
    from paper_2604_02047_b200 import binding
    lg = torch.zeros((2049, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.GooseError):
        binding.node_topk_static(lg, 4)                       # rows > GOOSE_STATIC_TOPK_MAX_ROWS
    with pytest.raises(binding.GooseError):
        binding.node_topk_static(lg[:8], 17)                  # k > 16
