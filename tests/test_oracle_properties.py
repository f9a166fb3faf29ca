"""Property tests of the CPU checker's routing rules over random small problems (hypothesis):
the invariants that Eq. 6-11 and Algorithms 1-2 fix for every input, whatever the shapes."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle
from tests.util import mask_to_dense


@st.composite
def problems(draw):
    D = draw(st.integers(1, 4))
    m = draw(st.integers(1, 4))
    E = D * m
    k = draw(st.integers(1, min(E, 4)))
    N = draw(st.integers(1, 120))
    gamma = draw(st.sampled_from([0.0, 0.3, 0.5, 1.0, 1.5, 4.0]))
    seed = draw(st.integers(0, 2 ** 20))
    levels = draw(st.sampled_from([0, 3, 8]))          # 0: continuous logits, else that many distinct values (ties)
    rng = np.random.default_rng(seed)
    lg = rng.normal(size=(N, E)).astype(np.float32) - np.log(np.arange(E) + 1.0).astype(np.float32)
    if levels:
        lg = np.round(lg * levels / 4.0).astype(np.float32) * np.float32(4.0 / levels)
    return N, E, k, D, gamma, lg


def _check_layout(r, cand_mask, E, slots):
    keep = mask_to_dense(r["keep_mask"], E).astype(bool)
    assert (keep <= cand_mask).all()                                   # only candidates are kept
    assert np.array_equal(r["kept"], keep.sum(0))
    assert r["offsets"][0] == 0 and np.array_equal(np.diff(r["offsets"]), r["kept"])
    rows = r["slot_row"][r["slot_row"] >= 0]
    assert sorted(rows.tolist()) == list(range(int(r["offsets"][-1])))  # a bijection onto [0, A)
    assert r["slot_row"].shape[1] == slots
    return keep


@settings(max_examples=60, deadline=None)
@given(problems())
def test_token_drop_invariants(p):
    N, E, k, D, gamma, lg = p
    s = oracle.softmax(lg)
    idx, _, load = oracle.topk(s, k)
    C = oracle.capacity(N, E, k, gamma)
    r = oracle.token_drop(s, idx, C)
    tk = np.zeros((N, E), bool)
    np.put_along_axis(tk, idx, True, axis=1)
    keep = _check_layout(r, tk, E, k)
    assert np.array_equal(r["kept"], np.minimum(load, C))              # Eq. 11: dropped_e = max(N_e - C, 0)
    for e in range(E):                                                 # Eq. 8-10 with the tie rule
        kept_t, drop_t = np.nonzero(keep[:, e])[0], np.nonzero(tk[:, e] & ~keep[:, e])[0]
        if len(kept_t) and len(drop_t):
            worst_kept = min((s[t, e], -t) for t in kept_t)
            best_dropped = max((s[t, e], -t) for t in drop_t)
            assert worst_kept > best_dropped
    if C >= load.max():
        assert np.array_equal(keep, tk)                                # no overflow: nothing changes


@settings(max_examples=60, deadline=None)
@given(problems())
def test_expanded_drop_invariants(p):
    N, E, k, D, gamma, lg = p
    s = oracle.softmax(lg)
    idx, _, _ = oracle.topk(s, k)
    C = oracle.capacity(N, E, k, gamma)
    m = E // D
    r = oracle.expanded_drop(s, idx, C, D)
    cand = np.zeros((N, E), bool)
    np.put_along_axis(cand, idx, True, axis=1)
    home = (np.arange(N) * D) // N
    for t in range(N):
        cand[t, home[t] * m:(home[t] + 1) * m] = True
    keep = _check_layout(r, cand, E, k + m)
    assert np.array_equal(r["cand"], cand.sum(0))
    assert np.array_equal(r["kept"], np.minimum(cand.sum(0), C))
    td = oracle.token_drop(s, idx, C)
    for e in range(E):                                                 # more candidates never lower the bar
        kept_t = np.nonzero(keep[:, e])[0]
        td_kept = np.nonzero(mask_to_dense(td["keep_mask"], E)[:, e])[0]
        if len(kept_t) == C and len(td_kept) == C and C > 0:
            assert min((s[t, e], -t) for t in kept_t) >= min((s[t, e], -t) for t in td_kept)


@settings(max_examples=40, deadline=None)
@given(problems(), st.booleans())
def test_device_drop_invariants(p, expanded):
    N, E, k, D, gamma, lg = p
    s = oracle.softmax(lg)
    idx, _, _ = oracle.topk(s, k)
    m = E // D
    Cd = oracle.device_capacity(N, E, k, D, gamma)
    r = oracle.device_drop(s, idx, Cd, D, expanded)
    cand = np.zeros((N, E), bool)
    np.put_along_axis(cand, idx, True, axis=1)
    if expanded:
        home = (np.arange(N) * D) // N
        for t in range(N):
            cand[t, home[t] * m:(home[t] + 1) * m] = True
    keep = _check_layout(r, cand, E, k + (m if expanded else 0))
    per_dev_cand = cand.reshape(N, D, m).sum((0, 2))
    per_dev_kept = keep.reshape(N, D, m).sum((0, 2))
    assert np.array_equal(per_dev_kept, np.minimum(per_dev_cand, Cd))  # the bound is on the device's total
