"""Pins for the oracle's logit harvest into the Tier-1 adjacency table (App. "Aggressive logit
harvesting"; "Dense GPU bigram adjacency table", Tier 1)."""
import numpy as np
from scipy.special import logsumexp, softmax

from paper_2604_02047_b200 import synth


def _table(V, k):
    return np.full((V, k), -7, np.int32), np.full((V, k), -1.0, np.float64)


def test_scores_are_softmax_probabilities_of_the_topk(oracle):
    rng = np.random.default_rng(2)
    V, k, rows = 500, 10, 6
    bits = synth.f32_to_bf16_bits((rng.standard_normal((rows, V)) * 3).astype(np.float32))
    tok = np.array([3, 499, 17, 0, 250, 8], np.int32)                  # distinct tokens
    ids, sc, lse = oracle.harvest(bits, k, tok, *_table(V, k))
    x = synth.bf16_bits_to_f64(bits)
    assert np.abs(lse - logsumexp(x, axis=1)).max() < 1e-12
    p = softmax(x, axis=1)
    order = np.argsort(-x, axis=1, kind="stable")[:, :k]
    for r in range(rows):
        assert np.array_equal(ids[tok[r]], order[r])
        assert np.abs(sc[tok[r]] - p[r, order[r]]).max() < 1e-14
    untouched = np.setdiff1d(np.arange(V), tok)
    assert np.all(ids[untouched] == -7) and np.all(sc[untouched] == -1.0)   # other tokens keep their entries


def test_closed_forms(oracle):
    V = 64
    const = np.full((1, V), 0x4040, np.uint16)                         # every logit 3.0
    ids, sc, lse = oracle.harvest(const, V, [5], *_table(V, V))
    assert ids[5].tolist() == list(range(V))                           # ties: lowest index first
    assert np.abs(sc[5] - 1.0 / V).max() < 1e-15 and abs(lse[0] - (3.0 + np.log(V))) < 1e-13
    rng = np.random.default_rng(3)
    bits = synth.f32_to_bf16_bits(rng.standard_normal((4, V), dtype=np.float32))
    ids, sc, _ = oracle.harvest(bits, V, [0, 1, 2, 3], *_table(V, V))
    assert np.abs(sc[:4].sum(axis=1) - 1.0).max() < 1e-13             # k = V: the scores of a row sum to one
    one_hot = np.full((1, V), 0xC2C8, np.uint16); one_hot[0, 9] = 0x42C8   # -100 everywhere, +100 at 9
    ids, sc, lse = oracle.harvest(one_hot, 2, [1], *_table(V, 2))
    assert ids[1, 0] == 9 and abs(sc[1, 0] - 1.0) < 1e-15 and abs(lse[0] - 100.0) < 1e-12


def test_last_row_with_a_token_wins_and_bad_tokens_are_skipped(oracle):
    rng = np.random.default_rng(4)
    V, k = 40, 4
    bits = synth.f32_to_bf16_bits(rng.standard_normal((5, V), dtype=np.float32))
    tok = np.array([7, 2, 7, -1, 40], np.int32)                        # 7 twice; -1 and 40 are out of range
    ids, sc, lse = oracle.harvest(bits, k, tok, *_table(V, k))
    ids2, sc2, _ = oracle.harvest(bits[2:3], k, [7], *_table(V, k))
    assert np.array_equal(ids[7], ids2[7]) and np.array_equal(sc[7], sc2[7])
    ids1, _, _ = oracle.harvest(bits[0:1], k, [7], *_table(V, k))
    assert not np.array_equal(ids1[7], ids2[7])
    touched = [7, 2]
    rest = np.setdiff1d(np.arange(V), touched)
    assert np.all(ids[rest] == -7)
    assert len(lse) == 5 and np.isfinite(lse).all()                    # lse is still reported for skipped rows
