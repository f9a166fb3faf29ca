"""Pins for the CPU checker: every function of oracle/ is checked against something other
than itself - hand-computed values, closed forms, invariants the paper states, brute force
on tiny inputs, and numpy fp64 routines for the dense algebra."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.util import bf16_bits_to_f64, mask_to_dense, to_np

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _scores(N, E, seed, quantum=0.0, bias=None):
    return oracle.softmax(synth.synthetic_logits(N, E, seed, bias=bias, quantum=quantum))


# ----------------------------------------------------------------------------- capacity
def test_capacity_hand_values():
    rows = [l.split() for l in open(os.path.join(GOLD, "capacity.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) >= 16
    for N, E, k, g, cc, cf in rows:
        assert oracle.capacity(int(N), int(E), int(k), float(g), "ceil") == int(cc), (N, E, k, g)
        assert oracle.capacity(int(N), int(E), int(k), float(g), "floor") == int(cf), (N, E, k, g)


def test_capacity_limits():
    assert oracle.capacity(100, 8, 2, float("inf")) == 100          # baseline gamma = +inf
    assert oracle.capacity(100, 8, 2, 1e9) == 100                   # clamped to N
    assert oracle.capacity(0, 8, 2, 1.0) == 0
    for N, E, k, g in [(96, 8, 2, 1.0), (640, 64, 8, 1.5), (64, 4, 1, 2.0)]:
        # ceil and floor agree whenever E divides gamma*N*k
        assert oracle.capacity(N, E, k, g, "ceil") == oracle.capacity(N, E, k, g, "floor") == int(g * N * k / E)
    with pytest.raises(ValueError):
        oracle.capacity(10, 4, 5, 1.0)


def test_stats_hand_values():
    for line in open(os.path.join(GOLD, "dropped_fraction.txt")):
        if not line.strip() or line[0] == "#":
            continue
        a, loads, dt, mom = [s.strip() for s in line.split("|")]
        N, k, C = map(int, a.split())
        st = oracle.stats(np.array(loads.split(), np.int32), N, k, C)
        assert st["dropped_fraction"] == pytest.approx(float(dt), abs=1e-15)
        assert st["max_over_mean"] == pytest.approx(float(mom), abs=1e-15)


# ----------------------------------------------------------------------------- softmax
def test_softmax_close_to_fp64_and_normalised():
    for E, seed in [(8, 1), (60, 2), (64, 3), (130, 4)]:
        lg = synth.synthetic_logits(700, E, seed) * np.float32(3.0)
        s = oracle.softmax(lg)
        l64 = lg.astype(np.float64)
        ref = np.exp(l64 - l64.max(1, keepdims=True))
        ref /= ref.sum(1, keepdims=True)
        # binary32 error budget: the subtraction l - max rounds (|x| * 2^-24, which exp turns into a
        # relative error), exp itself (< 1 ulp), E sequential additions (E * 2^-24) and the division
        xabs = np.abs(l64 - l64.max(1, keepdims=True))
        bound = (xabs + E + 4.0) * 2.0 ** -24 * ref + 1e-45
        live = ref > 1e-30
        assert np.all(np.abs(s.astype(np.float64) - ref)[live] <= bound[live])
        assert np.max(np.abs(s.astype(np.float64).sum(1) - 1.0)) <= E * 2.0 ** -23
        # exp(0) is exactly 1, so the arg-max logit scores 1/S with S >= 1
        am = lg.argmax(1)
        top = s[np.arange(len(s)), am]
        assert np.all(top == s.max(1)) and np.all(top <= 1.0) and np.all(top >= np.float32(1.0 / E) * 0.999)


def test_softmax_special_rows():
    E = 8
    lg = np.zeros((3, E), np.float32)
    lg[1, 3] = 100.0            # gaps beyond 80 underflow to an exact zero
    lg[2] = np.arange(E) * 0.0 + 5.0
    s = oracle.softmax(lg)
    assert np.all(s[0] == np.float32(1.0) / np.float32(8.0))
    assert s[1, 3] == 1.0 and np.all(np.delete(s[1], 3) == 0.0)
    assert np.all(s[2] == np.float32(0.125))
    # shift invariance is exact when the shift itself is: on a 1/64 grid a + 8 is representable,
    # l - max is then the same number for both inputs, and the scores must agree bit for bit
    a = synth.synthetic_logits(50, E, 9, quantum=1.0 / 64.0)
    assert np.array_equal((a + np.float32(8.0)) - np.float32(8.0), a)
    assert np.array_equal(oracle.softmax(a + np.float32(8.0)), oracle.softmax(a))
    assert np.array_equal(oracle.softmax(a - np.float32(16.0)), oracle.softmax(a))
    lg2 = np.array([[0.0, -1.0, -2.0, -90.0]], np.float32)
    s2 = oracle.softmax(lg2)
    ref = np.exp(np.array([0.0, -1.0, -2.0])); ref /= ref.sum()
    assert s2[0, 3] == 0.0 and np.allclose(s2[0, :3], ref, rtol=3e-7)


# ----------------------------------------------------------------------------- router GEMM
def test_router_logits_vs_numpy_fp64():
    cfg = synth.CONFIGS["tiny_f32"].with_(N=37, d=96)
    for dtype in ("f32", "bf16"):
        c = cfg.with_(dtype=dtype)
        x, w, b = synth.hidden_states(c), synth.router_weights(c), synth.router_bias(c)
        got = oracle.router_logits(to_np(x), to_np(w), b.numpy(), dtype)
        ref = x.double().numpy() @ w.double().numpy().T + b.double().numpy()[None]
        assert np.max(np.abs(got - ref)) <= 2e-6 * np.max(np.abs(ref))
        got0 = oracle.router_logits(to_np(x), to_np(w), None, dtype)
        assert np.max(np.abs(got0 - (ref - b.double().numpy()[None]))) <= 2e-6 * np.max(np.abs(ref))


def test_bf16_bits_are_read_exactly():
    t = torch.randn(1000, generator=torch.Generator().manual_seed(0)).to(torch.bfloat16)
    assert np.array_equal(bf16_bits_to_f64(to_np(t)), t.double().numpy())
    # one-hot weights make the router GEMM return x itself
    x = t[:64].reshape(4, 16).contiguous()
    w = torch.eye(16).to(torch.bfloat16)
    got = oracle.router_logits(to_np(x), to_np(w), None, "bf16")
    assert np.array_equal(got.astype(np.float64), x.double().numpy())


# ----------------------------------------------------------------------------- top-k
def test_topk_brute_force_and_load_identities():
    for (N, E, k, q) in [(300, 8, 2, 0.0), (257, 60, 4, 0.0), (128, 64, 8, 0.5), (50, 5, 5, 1.0)]:
        s = _scores(N, E, 11 + E, quantum=q)
        idx, val, load = oracle.topk(s, k)
        for t in range(N):
            order = sorted(range(E), key=lambda e: (-float(s[t, e]), e))[:k]   # ties -> lower expert id
            assert list(idx[t]) == order
            assert np.array_equal(val[t], s[t, order])
        assert load.sum() == N * k                                   # sum_i N_i = t k
        assert np.array_equal(load, np.bincount(idx.ravel(), minlength=E))
        nbar = N * k / E
        assert nbar <= load.max() <= E * nbar / k + 1e-9             # Eq. 5 (upper bound = N)


# ----------------------------------------------------------------------------- token drop
def _brute_keep(cands_by_expert, C):
    """keep (t,e) iff fewer than C candidates of e beat it; a beats b if score higher, or equal
    score and lower token index."""
    keep = set()
    for e, lst in cands_by_expert.items():
        for (t, s) in lst:
            better = sum(1 for (t2, s2) in lst if s2 > s or (s2 == s and t2 < t))
            if better < C:
                keep.add((t, e))
    return keep


@pytest.mark.parametrize("N,E,k,C,q", [(40, 4, 2, 7, 0.0), (64, 8, 2, 16, 0.0), (50, 8, 3, 5, 0.5),
                                       (33, 6, 2, 11, 1.0), (20, 4, 4, 3, 2.0), (16, 8, 1, 0, 0.0),
                                       (16, 8, 2, 16, 0.0)])
def test_token_drop_brute_force(N, E, k, C, q):
    bias = -np.log(np.arange(E) + 1.0)
    s = _scores(N, E, 5 + N, quantum=q, bias=bias)
    idx, _, load = oracle.topk(s, k)
    r = oracle.token_drop(s, idx, C)
    cands = {e: [(t, float(s[t, e])) for t in range(N) if e in idx[t]] for e in range(E)}
    keep = _brute_keep(cands, C)
    dense = mask_to_dense(r["keep_mask"], E)
    assert {(t, e) for t in range(N) for e in range(E) if dense[t, e]} == keep
    assert np.array_equal(r["kept"], np.minimum(load, C))


def _largest_per_expert(scores, eligible, C):
    """Independent statement of Eq. 7-10 / Algorithm 1 on tie-free scores: for every expert the
    kept set is the C largest scores among the tokens eligible for it (all of them if fewer)."""
    N, E = scores.shape
    want = np.zeros((N, E), bool)
    for e in range(E):
        toks = np.nonzero(eligible[:, e])[0]
        best = toks[np.argsort(-scores[toks, e], kind="stable")[:C]]
        want[best, e] = True
    return want


def test_token_drop_keeps_the_C_largest_of_each_expert():
    # tie-free inputs: there the C largest of a column are unique
    for (N, E, k, gamma) in [(512, 8, 2, 1.0), (384, 64, 8, 1.5), (600, 60, 4, 0.5)]:
        bias = -np.log(np.arange(E) + 1.0)
        s = _scores(N, E, 21, bias=bias)
        idx, val, load = oracle.topk(s, k)
        C = min(int(gamma * (N * k) / E), N)
        if len(np.unique(val)) != val.size or val.min() <= 0:
            pytest.skip("inputs not tie-free")
        chose = np.zeros((N, E), bool)
        np.put_along_axis(chose, idx, True, axis=1)
        want = _largest_per_expert(s, chose, C)
        r = oracle.token_drop(s, idx, C)
        assert np.array_equal(mask_to_dense(r["keep_mask"], E).astype(bool), want)
        # the gate weight carried by a kept row is the score of that (token, expert) pair (Eq. 2
        # with the kept set in place of the top-k set)
        A = int(r["offsets"][-1])
        p = oracle.permute(None, s, idx, r["slot_row"], A, 0, "f32")
        assert np.array_equal(p["perm_weight"], s[p["perm_token"], p["perm_expert"]])
        assert want[p["perm_token"], p["perm_expert"]].all() and want.sum() == A


def test_token_drop_invariants():
    for (N, E, k, gamma, q) in [(1000, 8, 2, 1.0, 0.0), (777, 64, 8, 0.5, 0.0), (512, 60, 4, 2.0, 0.25),
                                (300, 16, 4, 1.0, 1.0)]:
        bias = -1.2 * np.log(np.arange(E) + 1.0)
        s = _scores(N, E, 31, quantum=q, bias=bias)
        idx, _, load = oracle.topk(s, k)
        C = oracle.capacity(N, E, k, gamma)
        r = oracle.token_drop(s, idx, C)
        dense = mask_to_dense(r["keep_mask"], E).astype(bool)
        topk_mask = np.zeros((N, E), bool)
        np.put_along_axis(topk_mask, idx, True, axis=1)
        # kept_e = min(N_e, C)  <=>  dropped_e = ReLU(N_e - C)  (Eq. 11)
        assert np.array_equal(r["kept"], np.minimum(load, C))
        assert np.array_equal(dense.sum(0), r["kept"])
        st = oracle.stats(load, N, k, C)
        assert st["dropped_fraction"] * N * k == pytest.approx(np.maximum(load - C, 0).sum())
        assert (~dense | topk_mask).all()                         # final_map is a subset of topk_mask
        # Eq. 6: no expert above C; if the capacities cannot hold all assignments some expert is full
        assert dense.sum(0).max() <= C
        if E * C < N * k:
            assert dense.sum(0).max() == C
        # experts at or below capacity are untouched
        for e in np.nonzero(load <= C)[0]:
            assert np.array_equal(dense[:, e], topk_mask[:, e])
        # threshold property (Eq. 8-10): nothing kept ranks below something dropped, order (score, -t)
        for e in range(E):
            kp = np.nonzero(dense[:, e])[0]
            dr = np.nonzero(topk_mask[:, e] & ~dense[:, e])[0]
            if len(kp) and len(dr):
                worst_kept = min((float(s[t, e]), -t) for t in kp)
                best_drop = max((float(s[t, e]), -t) for t in dr)
                assert worst_kept > best_drop
        # offsets are the exclusive prefix of kept
        assert np.array_equal(r["offsets"], np.concatenate([[0], np.cumsum(r["kept"])]))


def test_no_drop_limit_and_gamma_inf():
    N, E, k = 400, 8, 2
    s = _scores(N, E, 41, bias=-np.log(np.arange(E) + 1.0))
    idx, _, load = oracle.topk(s, k)
    topk_mask = np.zeros((N, E), np.uint8)
    np.put_along_axis(topk_mask, idx, 1, axis=1)
    for C in (oracle.capacity(N, E, k, float("inf")), int(load.max())):
        r = oracle.token_drop(s, idx, C)
        assert np.array_equal(mask_to_dense(r["keep_mask"], E), topk_mask)
        assert (r["slot_row"] >= 0).all()
    r0 = oracle.token_drop(s, idx, 0)                             # gamma = 0
    assert r0["keep_mask"].sum() == 0 and (r0["slot_row"] == -1).all() and r0["offsets"][-1] == 0


def test_token_drop_commutes_with_token_permutation():
    # "Score" is stable under reordering the batch when scores are tie-free
    N, E, k = 500, 16, 4
    s = _scores(N, E, 51, bias=-np.log(np.arange(E) + 1.0))
    idx, val, _ = oracle.topk(s, k)
    assert len(np.unique(val)) == val.size
    C = oracle.capacity(N, E, k, 1.0)
    base = mask_to_dense(oracle.token_drop(s, idx, C)["keep_mask"], E)
    perm = synth.token_permutation(N, 3)
    s2 = np.ascontiguousarray(s[perm])
    idx2, _, _ = oracle.topk(s2, k)
    got = mask_to_dense(oracle.token_drop(s2, idx2, C)["keep_mask"], E)
    assert np.array_equal(got, base[perm])


def test_ties_go_to_lower_token_index():
    # all tokens identical: every score ties, so each expert keeps exactly tokens 0..C-1
    N, E, k, C = 30, 4, 2, 7
    lg = np.tile(np.array([[2.0, 1.0, 0.0, -1.0]], np.float32), (N, 1))
    s = oracle.softmax(lg)
    idx, _, load = oracle.topk(s, k)
    assert list(load) == [N, N, 0, 0]
    r = oracle.token_drop(s, idx, C)
    dense = mask_to_dense(r["keep_mask"], E)
    assert np.array_equal(np.nonzero(dense[:, 0])[0], np.arange(C))
    assert np.array_equal(np.nonzero(dense[:, 1])[0], np.arange(C))
    assert list(r["kept"]) == [C, C, 0, 0]


# ----------------------------------------------------------------------------- expanded drop
@pytest.mark.parametrize("N,E,k,D,C,q", [(40, 4, 2, 2, 9, 0.0), (48, 8, 2, 4, 5, 0.0), (36, 6, 2, 3, 4, 0.5),
                                         (30, 8, 3, 1, 6, 1.0), (24, 8, 2, 8, 3, 0.0), (25, 6, 1, 2, 30, 0.0)])
def test_expanded_drop_brute_force(N, E, k, D, C, q):
    m = E // D
    s = _scores(N, E, 61 + N, quantum=q, bias=-np.log(np.arange(E) + 1.0))
    idx, _, _ = oracle.topk(s, k)
    r = oracle.expanded_drop(s, idx, min(C, N), D)
    cands = {e: [] for e in range(E)}
    for t in range(N):
        g = (t * D) // N
        for e in range(E):
            if e in idx[t] or e // m == g:
                cands[e].append((t, float(s[t, e])))
    keep = _brute_keep(cands, min(C, N))
    dense = mask_to_dense(r["keep_mask"], E)
    assert {(t, e) for t in range(N) for e in range(E) if dense[t, e]} == keep
    assert list(r["cand"]) == [len(cands[e]) for e in range(E)]
    # explicit home groups equal the default contiguous split
    tg = ((np.arange(N) * D) // N).astype(np.int32)
    r2 = oracle.expanded_drop(s, idx, min(C, N), D, token_group=tg)
    for key in r:
        assert np.array_equal(r[key], r2[key])


def test_expanded_drop_invariants_and_closed_form():
    for (N, E, k, D, gamma) in [(512, 8, 2, 2, 1.0), (1024, 64, 8, 8, 1.0), (960, 60, 4, 4, 1.5),
                                (512, 64, 8, 8, 1.5)]:
        m = E // D
        s = _scores(N, E, 71, bias=-np.log(np.arange(E) + 1.0))
        idx, _, load = oracle.topk(s, k)
        C = oracle.capacity(N, E, k, gamma)
        r = oracle.expanded_drop(s, idx, C, D)
        td = oracle.token_drop(s, idx, C)
        dense = mask_to_dense(r["keep_mask"], E).astype(bool)
        topk_mask = np.zeros((N, E), bool)
        np.put_along_axis(topk_mask, idx, True, axis=1)
        home = (np.arange(N) * D) // N
        local = (np.arange(E)[None, :] // m) == home[:, None]
        exp_mask = topk_mask | local
        assert (~dense | exp_mask).all()                          # final_map subset of exp_mask
        assert (~(dense & ~topk_mask) | local).all()              # additions only inside the home group
        assert np.array_equal(r["cand"], exp_mask.sum(0))
        assert np.array_equal(r["kept"], np.minimum(r["cand"], C))
        assert np.array_equal(dense.sum(0), r["kept"])
        if N // D >= C:                                           # every expert has >= C candidates
            assert (r["kept"] == C).all() and r["offsets"][-1] == E * C
        # more candidates can only raise an expert's threshold
        dense_td = mask_to_dense(td["keep_mask"], E).astype(bool)
        for e in range(E):
            if r["kept"][e] == C and td["kept"][e] == C and C > 0:
                assert s[dense[:, e], e].min() >= s[dense_td[:, e], e].min()
        # threshold property among the expanded candidates
        for e in range(E):
            kp = np.nonzero(dense[:, e])[0]
            dr = np.nonzero(exp_mask[:, e] & ~dense[:, e])[0]
            if len(kp) and len(dr):
                assert min((float(s[t, e]), -t) for t in kp) > max((float(s[t, e]), -t) for t in dr)
        # slot layout: slots < k are the top-k order, slot k+i is local expert home*m+i
        sr = r["slot_row"]
        assert sr.shape == (N, k + m)
        for t in range(0, N, 37):
            for j in range(k):
                assert (sr[t, j] >= 0) == dense[t, idx[t, j]]
            for i in range(m):
                e = home[t] * m + i
                assert (sr[t, k + i] >= 0) == (dense[t, e] and not topk_mask[t, e])


def test_expanded_drop_single_group_is_expert_choice():
    # D = 1: every token is a candidate of every expert -> each expert keeps its top-C of all N tokens
    N, E, k, C = 200, 8, 2, 30
    s = _scores(N, E, 81, quantum=0.25)
    idx, _, _ = oracle.topk(s, k)
    r = oracle.expanded_drop(s, idx, C, 1)
    dense = mask_to_dense(r["keep_mask"], E)
    for e in range(E):
        order = np.lexsort((np.arange(N), -s[:, e].astype(np.float64)))[:C]
        assert np.array_equal(np.sort(order), np.nonzero(dense[:, e])[0])


def test_expanded_drop_keeps_the_C_largest_among_topk_and_home_device_tokens():
    # Algorithm 2 on tie-free scores: eligible = chose the expert, or lives on the expert's device
    N, E, k, D = 512, 8, 2, 2
    m = E // D
    s = _scores(N, E, 91, bias=-np.log(np.arange(E) + 1.0))
    idx, _, _ = oracle.topk(s, k)
    if len(np.unique(s)) != s.size or s.min() <= 0:
        pytest.skip("inputs not tie-free")
    C = int(1.0 * (N * k) / E)
    home = (np.arange(N) * D) // N
    eligible = np.zeros((N, E), bool)
    np.put_along_axis(eligible, idx, True, axis=1)
    eligible |= (np.arange(E)[None, :] // m) == home[:, None]
    r = oracle.expanded_drop(s, idx, C, D)
    assert np.array_equal(mask_to_dense(r["keep_mask"], E).astype(bool), _largest_per_expert(s, eligible, C))


# ----------------------------------------------------------------------------- permutation
def test_permutation_is_a_bijection_in_token_order():
    N, E, k, D = 700, 16, 4, 4
    s = _scores(N, E, 101, bias=-np.log(np.arange(E) + 1.0))
    idx, _, _ = oracle.topk(s, k)
    C = oracle.capacity(N, E, k, 1.0)
    for r, Dp in [(oracle.token_drop(s, idx, C), 0), (oracle.expanded_drop(s, idx, C, D), D)]:
        A = int(r["offsets"][-1])
        assert A == r["kept"].sum()
        rows = r["slot_row"][r["slot_row"] >= 0]
        assert np.array_equal(np.sort(rows), np.arange(A))
        x = synth.hidden_states(synth.CONFIGS["tiny_f32"].with_(N=N, d=24)).numpy()
        p = oracle.permute(x, s, idx, r["slot_row"], A, Dp, "f32")
        assert np.array_equal(p["x_perm"], x[p["perm_token"]])
        dense = mask_to_dense(r["keep_mask"], E)
        for e in range(E):
            seg = p["perm_token"][r["offsets"][e]:r["offsets"][e + 1]]
            assert np.all(np.diff(seg) > 0)
            assert np.array_equal(seg, np.nonzero(dense[:, e])[0])
            assert np.all(p["perm_expert"][r["offsets"][e]:r["offsets"][e + 1]] == e)
        assert np.array_equal(p["perm_weight"], s[p["perm_token"], p["perm_expert"]])


# ----------------------------------------------------------------------------- FFN + combine
def _swiglu_np(x, wg, wu, wd):
    g = x @ wg.T
    u = x @ wu.T
    return (g / (1.0 + np.exp(-g)) * u) @ wd.T


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_expert_ffn_vs_numpy_fp64(dtype):
    cfg = synth.CONFIGS["tiny_f32"].with_(N=23, d=48, F=40, E=3, k=1, D=1, dtype=dtype)
    x = synth.hidden_states(cfg)
    wg, wu, wd = synth.expert_weights(cfg, std=0.3)
    row_e = (np.arange(cfg.N) % 3).astype(np.int32)
    y = oracle.expert_ffn(to_np(x), row_e, to_np(wg), to_np(wu), to_np(wd), dtype)
    for e in range(3):
        ref = _swiglu_np(x.double().numpy()[row_e == e], wg[e].double().numpy(), wu[e].double().numpy(),
                         wd[e].double().numpy())
        assert np.allclose(y[row_e == e], ref, rtol=1e-12, atol=1e-13)


def test_layer_reduces_to_dense_ffn_when_all_experts_equal():
    # k = E, C = N, identical experts: y = (sum_e score_e) FFN(x) = FFN(x)
    cfg = synth.CONFIGS["tiny_f32"].with_(N=40, d=32, F=24, E=4, k=4, D=2)
    inp = synth.make_layer_inputs(cfg)
    wg = inp.w_gate[:1].repeat(4, 1, 1).contiguous() * 10
    wu = inp.w_up[:1].repeat(4, 1, 1).contiguous() * 10
    wd = inp.w_down[:1].repeat(4, 1, 1).contiguous() * 10
    out = oracle.layer_forward(to_np(inp.x), to_np(inp.w_router), inp.bias.numpy(), to_np(wg), to_np(wu),
                               to_np(wd), cfg.k, float("inf"), cfg.D, "token_drop", "f32")
    ref = _swiglu_np(inp.x.double().numpy(), wg[0].double().numpy(), wu[0].double().numpy(), wd[0].double().numpy())
    ssum = out["scores"].astype(np.float64).sum(1, keepdims=True)
    assert np.allclose(out["y"], ssum * ref, rtol=1e-12, atol=1e-14)
    assert np.allclose(out["y"], ref, rtol=1e-6, atol=1e-9)


def test_layer_algebraic_properties():
    cfg = synth.CONFIGS["tiny_f32"].with_(N=96, d=32, F=24)
    inp = synth.make_layer_inputs(cfg)
    a = [to_np(inp.x), to_np(inp.w_router), inp.bias.numpy()]
    wg, wu, wd = to_np(inp.w_gate * 10), to_np(inp.w_up * 10), to_np(inp.w_down * 10)
    for mode in ("nodrop", "token_drop", "expanded_drop"):
        base = oracle.layer_forward(*a, wg, wu, wd, cfg.k, 1.0, cfg.D, mode, "f32")
        # zero gate projection -> silu(0) = 0 -> zero output
        z = oracle.layer_forward(*a, np.zeros_like(wg), wu, wd, cfg.k, 1.0, cfg.D, mode, "f32")
        assert np.all(z["y"] == 0.0)
        # linear in W_d
        two = oracle.layer_forward(*a, wg, wu, (wd * np.float32(2.0)), cfg.k, 1.0, cfg.D, mode, "f32")
        assert np.allclose(two["y"], 2.0 * base["y"], rtol=1e-13, atol=0)
        # identity experts: combine(permute(x)) = (sum of kept scores) * x
        ident = oracle.combine(base["x_perm"].astype(np.float64), base["slot_row"], base["scores"],
                               base["topk_idx"], cfg.D if mode == "expanded_drop" else 0)
        dense = mask_to_dense(base["keep_mask"], cfg.E)
        wsum = (base["scores"].astype(np.float64) * dense).sum(1, keepdims=True)
        assert np.allclose(ident, wsum * inp.x.double().numpy(), rtol=1e-12, atol=1e-15)
        none_kept = dense.sum(1) == 0
        assert np.all(base["y"][none_kept] == 0.0)
        # the token-sampled evaluation agrees with the full layer
        toks = np.array([0, 5, 17, 95], np.int32)
        part = oracle.layer_tokens(a[0], toks, base["scores"], base["topk_idx"], base["slot_row"],
                                   cfg.D if mode == "expanded_drop" else 0, wg, wu, wd, "f32")
        assert np.allclose(part, base["y"][toks], rtol=1e-12, atol=1e-15)
    # gamma = inf reproduces the no-drop layer exactly
    nd = oracle.layer_forward(*a, wg, wu, wd, cfg.k, 1.0, cfg.D, "nodrop", "f32")
    inf = oracle.layer_forward(*a, wg, wu, wd, cfg.k, float("inf"), cfg.D, "token_drop", "f32")
    assert np.array_equal(nd["y"], inf["y"])
    # shared expert is added with weight one
    sh_cfg = cfg.with_(F_shared=16)
    sh = synth.shared_expert_weights(sh_cfg, std=0.2)
    shn = tuple(to_np(w) for w in sh)
    with_sh = oracle.layer_forward(*a, wg, wu, wd, cfg.k, 1.0, cfg.D, "token_drop", "f32", shared=shn)
    td = oracle.layer_forward(*a, wg, wu, wd, cfg.k, 1.0, cfg.D, "token_drop", "f32")
    ref_sh = _swiglu_np(inp.x.double().numpy(), sh[0][0].double().numpy(), sh[1][0].double().numpy(),
                        sh[2][0].double().numpy())
    assert np.allclose(with_sh["y"] - td["y"], ref_sh, rtol=1e-9, atol=1e-12)
