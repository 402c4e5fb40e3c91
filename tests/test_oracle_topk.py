"""Pins for the oracle's per-node argmax / top-k (Algorithm 3 step 2; App. logit harvesting)."""
import numpy as np

from paper_2604_02047_b200 import synth


def _ref_topk(bits, k):
    """Library cross-check: stable argsort of the negated values = (value desc, index asc)."""
    v = synth.bf16_bits_to_f32(bits).astype(np.float64) + 0.0     # -0.0 + 0.0 == +0.0
    order = np.argsort(-v, axis=1, kind="stable")[:, :k]
    return order.astype(np.int32), np.take_along_axis(v, order, axis=1)


def test_topk_matches_stable_argsort_with_many_ties(oracle):
    rng = np.random.default_rng(0)
    # coarse values -> massive exact ties, incl. at the maximum
    x = np.round(rng.standard_normal((40, 3000)) * 4).astype(np.float32) / 4
    bits = synth.f32_to_bf16_bits(x)
    am, ids, vals = oracle.node_topk(bits, 8)
    rid, rval = _ref_topk(bits, 8)
    assert np.array_equal(ids, rid) and np.array_equal(vals, rval) and np.array_equal(am, rid[:, 0])


def test_topk_on_generator_logits(oracle):
    x = synth.make_config(0)
    am, ids, vals = oracle.node_topk(x.logits, x.k)
    rid, rval = _ref_topk(x.logits, x.k)
    assert np.array_equal(ids, rid) and np.array_equal(vals, rval)
    # a planted child token is its parent's argmax unless a larger planted sibling exists
    lg = synth.bf16_bits_to_f32(x.logits)
    assert np.array_equal(am, np.argmax(lg, axis=1))              # numpy argmax: first maximum


def test_special_rows(oracle):
    V, k = 100, 8
    const = np.full((1, V), 0x4000, np.uint16)                    # all 2.0 -> ids 0..k-1
    am, ids, _ = oracle.node_topk(const, k)
    assert ids[0].tolist() == list(range(k)) and am[0] == 0
    zeros = np.zeros((1, V), np.uint16); zeros[0, ::2] = 0x8000   # mix of -0.0 and +0.0: all equal
    _, ids, vals = oracle.node_topk(zeros, k)
    assert ids[0].tolist() == list(range(k)) and np.all(vals == 0)
    row = synth.f32_to_bf16_bits(np.linspace(-1, 1, V, dtype=np.float32))[None].copy()
    row[0, 0] = row[0, V - 1]                                     # maximum duplicated at both ends
    am, ids, _ = oracle.node_topk(row, 3)
    assert am[0] == 0 and ids[0].tolist() == [0, V - 1, V - 2]
    neg = synth.f32_to_bf16_bits(-np.arange(1, V + 1, dtype=np.float32))[None]
    _, ids, vals = oracle.node_topk(neg, 4)
    assert ids[0].tolist() == [0, 1, 2, 3] and vals[0].tolist() == [-1, -2, -3, -4]


def test_row_stride_and_k_equals_v(oracle):
    rng = np.random.default_rng(4)
    full = synth.f32_to_bf16_bits(rng.standard_normal((5, 48), dtype=np.float32))
    am, ids, vals = oracle.node_topk(full, 16, V=16)              # ldl = 48, only first 16 columns count
    rid, rval = _ref_topk(full[:, :16], 16)
    assert np.array_equal(ids, rid) and np.array_equal(vals, rval)
