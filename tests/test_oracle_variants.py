"""Pins for the CPU checker's variants of the drop: priority classes (modality-first dropping,
Expanded Drop as substitution only), the 'w/ max' limit on experts per token, global top-(k+m)
expansion, and the rebuild of counts / offsets / rows from a keep mask.  Each is checked against a
brute-force restatement in plain Python and against the properties the paper states for it."""
import numpy as np
import pytest

import oracle
from paper_2503_05066_b200 import synth
from tests.util import mask_to_dense


def _routing(N, E, k, seed, q=0.0, s_bias=1.0):
    s = oracle.softmax(synth.synthetic_logits(N, E, seed, bias=-s_bias * np.log(np.arange(E) + 1.0), quantum=q))
    idx, _, load = oracle.topk(s, k)
    return s, idx, load


def _dense_topk(idx, E):
    m = np.zeros((idx.shape[0], E), bool)
    np.put_along_axis(m, idx, True, axis=1)
    return m


def _brute_select(cand_mask, rank_key, C):
    """Per expert: the C candidates with the largest rank_key tuple, ties to the lower token.
    rank_key(t, e) -> tuple.  Returns a dense bool keep matrix."""
    N, E = cand_mask.shape
    keep = np.zeros((N, E), bool)
    for e in range(E):
        ts = [t for t in range(N) if cand_mask[t, e]]
        ts.sort(key=lambda t: (tuple(-x for x in rank_key(t, e)), t))
        for t in ts[:C]:
            keep[t, e] = True
    return keep


def test_priority_bits_sit_above_an_unchanged_score_key():
    N, E, k = 50, 8, 2
    s, idx, _ = _routing(N, E, k, 3)
    base = oracle.drop_keys("score", 0, s, None, E)
    assert int(base.max()) <= 0x3F800000 < 2 ** 30          # scores lie in [0, 1]
    cls = (np.arange(N) % 3 == 0).astype(np.uint8)
    keys = oracle.priority_keys(base, None, E, True, token_class=cls, topk_idx=idx)
    tk = _dense_topk(idx, E)
    assert np.array_equal(keys & np.uint32(0x3FFFFFFF), base)
    assert np.array_equal(keys >> np.uint32(30), (2 * tk + cls[:, None]).astype(np.uint32))
    # no class given: nothing changes
    assert np.array_equal(oracle.priority_keys(base, None, E, True), base)
    # inexact bodies lose their two low bits, exact ones must fit
    rnd = oracle.drop_keys("random", 5, s, None, E)
    shifted = oracle.priority_keys(rnd, None, E, False, token_class=cls)
    assert np.array_equal(shifted & np.uint32(0x3FFFFFFF), rnd >> np.uint32(2))
    with pytest.raises(ValueError):
        oracle.priority_keys(rnd | np.uint32(1 << 31), None, E, True)
    # sparse [N,k] layout with expert ids
    sp = oracle.priority_keys(np.take_along_axis(base, idx, 1), idx, E, True, token_class=cls, topk_idx=idx)
    assert np.array_equal(sp, np.take_along_axis(keys, idx, 1))


@pytest.mark.parametrize("protect_text", [True, False])
def test_modality_first_dropping_matches_brute_force(protect_text):
    """Image First = text tokens are protected: an expert drops image tokens before any text token."""
    N, E, k = 240, 6, 2
    s, idx, load = _routing(N, E, k, 11, q=0.25, s_bias=1.5)
    is_image = (np.arange(N) * 7 % 10) < 6
    cls = (~is_image if protect_text else is_image).astype(np.uint8)
    C = oracle.capacity(N, E, k, 0.75)
    keys = oracle.priority_keys(oracle.drop_keys("score", 0, s, None, E), None, E, True, token_class=cls)
    r = oracle.drop_keyed(keys, idx, C)
    got = mask_to_dense(r["keep_mask"], E).astype(bool)
    tk = _dense_topk(idx, E)
    want = _brute_select(tk, lambda t, e: (int(cls[t]), float(s[t, e])), C)
    assert np.array_equal(got, want)
    assert np.array_equal(r["kept"], np.minimum(load, C))
    # the stated property: where a protected token was dropped, no unprotected token was kept
    for e in range(E):
        dropped_protected = (tk[:, e] & ~got[:, e] & (cls == 1)).any()
        kept_unprotected = (got[:, e] & (cls == 0)).any()
        assert not (dropped_protected and kept_unprotected)
    # one modality only: the class is a constant and the result is the uniform Token Drop
    keys1 = oracle.priority_keys(oracle.drop_keys("score", 0, s, None, E), None, E, True,
                                 token_class=np.ones(N, np.uint8))
    assert np.array_equal(oracle.drop_keyed(keys1, idx, C)["keep_mask"], oracle.token_drop(s, idx, C)["keep_mask"])


def test_topk_first_expansion_never_displaces_a_topk_assignment():
    N, E, k, D = 360, 12, 3, 4
    s, idx, load = _routing(N, E, k, 21, q=0.5)
    C = oracle.capacity(N, E, k, 1.0)
    m = E // D
    tk = _dense_topk(idx, E)
    home = (np.arange(N) * D) // N
    cand = tk.copy()
    for t in range(N):
        cand[t, home[t] * m:(home[t] + 1) * m] = True
    keys = oracle.priority_keys(oracle.drop_keys("score", 0, s, None, E), None, E, True, topk_idx=idx)
    r = oracle.drop_keyed(keys, idx, C, D, True)
    got = mask_to_dense(r["keep_mask"], E).astype(bool)
    want = _brute_select(cand, lambda t, e: (int(tk[t, e]), float(s[t, e])), C)
    assert np.array_equal(got, want)
    # the top-k part of the result is exactly Token Drop's result ...
    td = mask_to_dense(oracle.token_drop(s, idx, C)["keep_mask"], E).astype(bool)
    assert np.array_equal(got & tk, td)
    # ... experts overflowed by their top-k candidates take nobody else ...
    for e in range(E):
        if load[e] >= C:
            assert not (got[:, e] & ~tk[:, e]).any()
    # ... and every expert is still filled to min(candidates, C), as under equal competition
    eq = oracle.expanded_drop(s, idx, C, D)
    assert np.array_equal(r["kept"], eq["kept"]) and np.array_equal(r["cand"], eq["cand"])
    # equal competition does displace some top-k pairs on this input: the two readings differ
    assert not np.array_equal(r["keep_mask"], eq["keep_mask"])


def test_limit_experts_keeps_each_tokens_best_k():
    N, E, k, D = 300, 16, 2, 2
    s, idx, _ = _routing(N, E, k, 31, q=0.5)
    C = oracle.capacity(N, E, k, 1.5)
    r = oracle.expanded_drop(s, idx, C, D)
    before = mask_to_dense(r["keep_mask"], E).astype(bool)
    assert before.sum(1).max() > k                           # the case the ablation is about
    after = mask_to_dense(oracle.limit_experts(s, r["keep_mask"], k), E).astype(bool)
    assert (after <= before).all() and after.sum(1).max() == k
    for t in range(N):
        es = sorted(np.nonzero(before[t])[0], key=lambda e: (-float(s[t, e]), e))
        assert sorted(np.nonzero(after[t])[0]) == sorted(es[:k])
    # a limit nobody exceeds changes nothing
    assert np.array_equal(oracle.limit_experts(s, r["keep_mask"], E), r["keep_mask"])
    # limit 0 empties the mask
    assert not oracle.limit_experts(s, r["keep_mask"], 0).any()


@pytest.mark.parametrize("expanded", [False, True])
def test_rows_from_mask_rebuilds_what_the_drop_produced(expanded):
    N, E, k, D = 500, 12, 3, 4
    s, idx, _ = _routing(N, E, k, 41, q=0.25)
    C = oracle.capacity(N, E, k, 1.0)
    r = oracle.expanded_drop(s, idx, C, D) if expanded else oracle.token_drop(s, idx, C)
    slots = k + (E // D if expanded else 0)
    b = oracle.rows_from_mask(r["keep_mask"], idx, E, slots, D)
    for key in ("kept", "offsets", "slot_row"):
        assert np.array_equal(b[key], r[key]), key
    # after 'w/ max' the rows are a bijection onto [0, A) and ascend with the token inside a segment
    if expanded:
        lim = oracle.limit_experts(s, r["keep_mask"], k)
        c = oracle.rows_from_mask(lim, idx, E, slots, D)
        A = int(c["offsets"][-1])
        rows = c["slot_row"][c["slot_row"] >= 0]
        assert sorted(rows.tolist()) == list(range(A))
        dense = mask_to_dense(lim, E)
        assert np.array_equal(c["kept"], dense.sum(0))
        p = oracle.permute(None, s, idx, c["slot_row"], A, D, "f32")
        for e in range(E):
            seg = p["perm_token"][c["offsets"][e]:c["offsets"][e + 1]]
            assert np.array_equal(seg, np.nonzero(dense[:, e])[0])
    # a bit outside the token's slots is refused
    bad = r["keep_mask"].copy()
    t = 0
    outside = [e for e in range(E) if e not in idx[t] and not (expanded and e // (E // D) == 0)]
    bad[t, 0] |= np.uint64(1) << np.uint64(outside[0])
    with pytest.raises(ValueError):
        oracle.rows_from_mask(bad, idx, E, slots, D)


def test_global_expansion_is_token_drop_on_k_plus_m_choices():
    """Candidates = each token's k+m best experts anywhere (the ablation's global top-(k+m)): the
    router with k+m choices followed by the plain drop; with D = 1 the home device holds every
    expert and Expanded Drop coincides with it at k + m = E."""
    N, E, k = 200, 8, 2
    s, idx, _ = _routing(N, E, k, 51)
    idx_all, _, _ = oracle.topk(s, E)
    C = oracle.capacity(N, E, k, 1.0)
    a = oracle.token_drop(s, idx_all, C)
    b = oracle.expanded_drop(s, idx, C, 1)
    assert np.array_equal(a["keep_mask"], b["keep_mask"])
    # fewer extra choices: candidates are a subset, so no expert's threshold can be higher
    idx_km, _, _ = oracle.topk(s, k + 3)
    c = oracle.token_drop(s, idx_km, C)
    assert (c["kept"] <= a["kept"]).all() and (c["kept"] >= oracle.token_drop(s, idx, C)["kept"]).all()
