"""Pins for the drop metrics of the CPU checker ("Order", "Reverse Order", "Random", "Score"):
closed forms for the positional metrics, agreement of the Score metric with the score-based
drop, uniformity and seed behaviour of the random keys."""
import numpy as np
import pytest

import oracle
from paper_2503_05066_b200 import synth
from tests.util import mask_to_dense


def _routing(N, E, k, seed, q=0.0):
    s = oracle.softmax(synth.synthetic_logits(N, E, seed, bias=-np.log(np.arange(E) + 1.0), quantum=q))
    idx, _, load = oracle.topk(s, k)
    return s, idx, load


def test_score_metric_is_the_score_based_drop():
    N, E, k, D = 800, 16, 4, 4
    s, idx, _ = _routing(N, E, k, 1, q=0.25)
    keys = oracle.drop_keys("score", 0, s, None, E)
    assert np.array_equal(keys, s.view(np.uint32))
    C = oracle.capacity(N, E, k, 1.0)
    a = oracle.drop_keyed(keys, idx, C)
    b = oracle.token_drop(s, idx, C)
    for key in ("keep_mask", "kept", "offsets", "slot_row"):
        assert np.array_equal(a[key], b[key]), key
    a = oracle.drop_keyed(keys, idx, C, D, True)
    b = oracle.expanded_drop(s, idx, C, D)
    for key in ("keep_mask", "cand", "kept", "offsets", "slot_row"):
        assert np.array_equal(a[key], b[key]), key
    # sparse [N,k] form: keys of the top-k entries only
    kk = oracle.drop_keys("score", 0, np.take_along_axis(s, idx, 1), idx, E)
    assert np.array_equal(kk, np.take_along_axis(keys, idx, 1))


def test_order_keeps_the_first_and_reverse_order_the_last_candidates():
    N, E, k = 600, 8, 2
    s, idx, load = _routing(N, E, k, 2)
    C = oracle.capacity(N, E, k, 1.0)
    topk_mask = np.zeros((N, E), bool)
    np.put_along_axis(topk_mask, idx, True, axis=1)
    for metric in ("order", "reverse_order"):
        keys = oracle.drop_keys(metric, 0, s, None, E)
        r = oracle.drop_keyed(keys, idx, C)
        dense = mask_to_dense(r["keep_mask"], E).astype(bool)
        assert np.array_equal(r["kept"], np.minimum(load, C))
        for e in range(E):
            cands = np.nonzero(topk_mask[:, e])[0]
            want = cands[:C] if metric == "order" else cands[len(cands) - min(C, len(cands)):]
            assert np.array_equal(np.nonzero(dense[:, e])[0], want), (metric, e)


def test_random_keys_are_uniform_seeded_and_position_based():
    N, E = 4000, 16
    s = np.zeros((N, E), np.float32)
    k1 = oracle.drop_keys("random", 7, s, None, E)
    k2 = oracle.drop_keys("random", 7, s + 1.0, None, E)         # independent of the scores
    k3 = oracle.drop_keys("random", 8, s, None, E)
    assert np.array_equal(k1, k2) and not np.array_equal(k1, k3)
    u = k1.astype(np.float64).ravel() / 2.0 ** 32
    n = u.size
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / n) and abs(u.var() - 1 / 12) < 0.002
    assert len(np.unique(k1)) > 0.999 * n                          # 64k draws from 2^32: almost no collisions
    # bit balance: every bit of the key is set about half the time
    bits = ((k1.ravel()[:, None] >> np.arange(32, dtype=np.uint32)) & 1).mean(0)
    assert np.all(np.abs(bits - 0.5) < 0.01)
    # the key of an entry depends on (t, e) only: the sparse [N,k] form picks the same values
    idx = np.stack([np.arange(N) % E, (np.arange(N) * 7 + 3) % E], 1).astype(np.int32)
    ks = oracle.drop_keys("random", 7, np.zeros((N, 2), np.float32), idx, E)
    assert np.array_equal(ks, np.take_along_axis(k1, idx, 1))


def test_random_drop_has_no_positional_or_score_preference():
    N, E, k = 6000, 4, 1
    s, idx, load = _routing(N, E, k, 3)
    C = int(load.max() // 2)
    keys = oracle.drop_keys("random", 123, s, None, E)
    r = oracle.drop_keyed(keys, idx, C)
    dense = mask_to_dense(r["keep_mask"], E).astype(bool)
    e = int(load.argmax())
    cands = np.nonzero(idx[:, 0] == e)[0]
    kept = dense[cands, e]
    assert kept.sum() == C
    frac = C / len(cands)
    half = len(cands) // 2
    sd = np.sqrt(frac * (1 - frac) / half)
    assert abs(kept[:half].mean() - frac) < 5 * sd                 # early and late tokens alike
    hi = s[cands, e] > np.median(s[cands, e])
    assert abs(kept[hi].mean() - frac) < 5 * sd                    # high and low scores alike
