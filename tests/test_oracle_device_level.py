"""Pins for the device-level capacity variant of the CPU checker ("Advanced Variant:
Device-Level Capacity-Aware Inference"): brute force on tiny inputs, the aggregated-load bound
N_1 + ... + N_{n_l} <= n_l * gamma * N_bar, reduction to the expert-level rule when each device
holds one expert, and the comparison with expert-level capacity the paper argues from."""
import numpy as np
import pytest

import oracle
from paper_2503_05066_b200 import synth
from tests.util import mask_to_dense


def _scores(N, E, seed, quantum=0.0):
    bias = -np.log(np.arange(E) + 1.0)
    return oracle.softmax(synth.synthetic_logits(N, E, seed, bias=bias, quantum=quantum))


def test_device_capacity_values():
    # n_l * gamma * N_bar = gamma * N * k / D
    assert oracle.device_capacity(8192, 8, 2, 2, 1.0) == 8192
    assert oracle.device_capacity(4096, 64, 8, 8, 1.5) == 6144
    assert oracle.device_capacity(128, 60, 4, 4, 0.5) == 64
    assert oracle.device_capacity(100, 60, 4, 4, 1.0, "ceil") == 100
    assert oracle.device_capacity(10, 6, 4, 3, 1.0, "ceil") == 14      # 13.33 -> 14
    assert oracle.device_capacity(10, 6, 4, 3, 1.0, "floor") == 13
    assert oracle.device_capacity(10, 8, 2, 2, float("inf")) == 40     # clamp: N * E/D pairs at most
    assert oracle.device_capacity(10, 8, 2, 2, 0.0) == 0
    # with one expert per device it is the expert capacity
    for N, E, k, g in [(512, 8, 2, 1.0), (100, 60, 4, 1.5)]:
        assert oracle.device_capacity(N, E, k, E, g) == oracle.capacity(N, E, k, g)


@pytest.mark.parametrize("N,E,k,D,C,expanded,q", [(30, 4, 2, 2, 20, False, 0.0), (30, 4, 2, 2, 20, True, 0.0),
                                                  (40, 8, 3, 2, 37, False, 0.5), (36, 6, 2, 3, 10, True, 1.0),
                                                  (25, 8, 2, 4, 0, False, 0.0), (25, 8, 2, 1, 1000, True, 0.0)])
def test_device_drop_brute_force(N, E, k, D, C, expanded, q):
    m = E // D
    s = _scores(N, E, 7 + N, quantum=q)
    idx, _, _ = oracle.topk(s, k)
    r = oracle.device_drop(s, idx, C, D, expanded)
    dense = mask_to_dense(r["keep_mask"], E)
    want = set()
    for g in range(D):
        pairs = []
        for t in range(N):
            home = (t * D) // N
            for e in range(g * m, (g + 1) * m):
                if e in idx[t] or (expanded and home == g):
                    pairs.append((float(s[t, e]), t, e))
        for (sc, t, e) in pairs:      # keep iff fewer than C pairs of this device beat it
            better = sum(1 for (s2, t2, e2) in pairs if s2 > sc or (s2 == sc and (t2, e2) < (t, e)))
            if better < C:
                want.add((t, e))
    assert {(t, e) for t in range(N) for e in range(E) if dense[t, e]} == want
    # rows: expert-major, ascending token inside a segment, a bijection onto [0, A)
    A = int(r["offsets"][-1])
    assert A == len(want) == int(r["kept"].sum())
    rows = r["slot_row"][r["slot_row"] >= 0]
    assert np.array_equal(np.sort(rows), np.arange(A))
    p = oracle.permute(None, s, idx, r["slot_row"], A, D if expanded else 0, "f32")
    for e in range(E):
        seg = p["perm_token"][r["offsets"][e]:r["offsets"][e + 1]]
        assert np.all(np.diff(seg) > 0) and np.array_equal(seg, np.nonzero(dense[:, e])[0])


def test_one_expert_per_device_is_the_expert_level_rule():
    N, E, k = 600, 8, 2
    s = _scores(N, E, 3, quantum=0.25)
    idx, _, _ = oracle.topk(s, k)
    C = oracle.capacity(N, E, k, 1.0)
    a = oracle.device_drop(s, idx, C, E, False)
    b = oracle.token_drop(s, idx, C)
    for key in ("keep_mask", "kept", "offsets", "slot_row"):
        assert np.array_equal(a[key], b[key]), key
    a = oracle.device_drop(s, idx, C, E, True)         # each token's home device holds one expert
    b = oracle.expanded_drop(s, idx, C, E)
    for key in ("keep_mask", "cand", "kept", "offsets", "slot_row"):
        assert np.array_equal(a[key], b[key]), key


def test_device_level_bound_and_comparison_with_expert_level():
    for (N, E, k, D, gamma) in [(2048, 64, 8, 8, 1.0), (1500, 60, 4, 4, 1.5), (1024, 8, 2, 2, 1.0)]:
        m = E // D
        s = _scores(N, E, 11)
        idx, _, load = oracle.topk(s, k)
        C = oracle.capacity(N, E, k, gamma)
        C_dev = oracle.device_capacity(N, E, k, D, gamma)
        for expanded in (False, True):
            r = oracle.device_drop(s, idx, C_dev, D, expanded)
            ex = oracle.expanded_drop(s, idx, C, D) if expanded else oracle.token_drop(s, idx, C)
            dev_kept = r["kept"].reshape(D, m).sum(1)
            dev_cand = r["cand"].reshape(D, m).sum(1)
            # the aggregated load of every device respects n_l * gamma * N_bar, and is exactly
            # min(candidates, C_dev)
            assert np.array_equal(dev_kept, np.minimum(dev_cand, C_dev))
            # a device is never allowed fewer pairs than its experts together (m * C >= C_dev rounding aside)
            ex_dev = ex["kept"].reshape(D, m).sum(1)
            assert np.all(dev_kept >= np.minimum(ex_dev, C_dev))
            # an expert may now exceed its own budget as long as the device has room
            if not expanded and load.max() > C:
                assert r["kept"].max() >= ex["kept"].max()
            # threshold property per device in the order (score, -token, -expert)
            dense = mask_to_dense(r["keep_mask"], E).astype(bool)
            cand_mask = np.zeros((N, E), bool)
            np.put_along_axis(cand_mask, idx, True, axis=1)
            if expanded:
                home = (np.arange(N) * D) // N
                cand_mask |= (np.arange(E)[None, :] // m) == home[:, None]
            assert (~dense | cand_mask).all()
            for g in range(D):
                cols = slice(g * m, (g + 1) * m)
                kp = np.argwhere(dense[:, cols])
                dr = np.argwhere(cand_mask[:, cols] & ~dense[:, cols])
                if len(kp) and len(dr):
                    worst = min((float(s[t, g * m + j]), -t, -j) for t, j in kp)
                    best = max((float(s[t, g * m + j]), -t, -j) for t, j in dr)
                    assert worst > best


def test_gamma_inf_keeps_everything():
    N, E, k, D = 300, 8, 2, 2
    s = _scores(N, E, 5)
    idx, _, load = oracle.topk(s, k)
    r = oracle.device_drop(s, idx, oracle.device_capacity(N, E, k, D, float("inf")), D, False)
    assert np.array_equal(r["kept"], load) and (r["slot_row"] >= 0).all()
