"""ctypes front end of the CPU checker (oracle/capmoe_oracle.cpp).  Test infrastructure only.

All arrays are numpy, C-contiguous.  bf16 tensors are passed as uint16 bit patterns
(dtype="bf16"); fp32 as float32 (dtype="f32").
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
import sys
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "capmoe_oracle.cpp")
_LIB = os.path.join(_HERE, "libcapmoe_oracle.so")
_lib = None

__all__ = ["build", "capacity", "device_capacity", "device_drop", "drop_keys", "drop_keyed", "METRICS",
           "priority_keys", "limit_experts", "rows_from_mask", "router_logits", "softmax", "topk", "token_drop",
           "expanded_drop",
           "permute", "expert_ffn", "combine", "layer_tokens", "stats", "layer_forward", "ep_layer", "num_threads"]


def build(force: bool = False) -> str:
    """Compile the checker.  No -march flags beyond AVX2/FMA: the binary travels between machines."""
    if (not force) and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["g++", "-O3", "-std=c++17", "-mavx2", "-mfma", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-shared", "-fPIC", _SRC, "-o", _LIB]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    try:
        _lib = ctypes.CDLL(_LIB)
    except OSError:
        build(force=True)
        _lib = ctypes.CDLL(_LIB)
    return _lib


def num_threads() -> int:
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else (os.cpu_count() or 1)


def _p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return ctypes.c_void_p(a.ctypes.data)


def _dt(dtype: str) -> int:
    return {"f32": 0, "bf16": 1}[dtype]


def _i64(v):
    return ctypes.c_int64(int(v))


def capacity(N: int, E: int, k: int, gamma: float, round_mode: str = "ceil") -> int:
    out = ctypes.c_int64(0)
    rc = _load().oracle_capacity(_i64(N), int(E), int(k), ctypes.c_double(gamma),
                                 0 if round_mode == "ceil" else 1, ctypes.byref(out))
    if rc != 0:
        raise ValueError("bad capacity arguments")
    return out.value


def router_logits(x: np.ndarray, w: np.ndarray, bias: Optional[np.ndarray], dtype: str) -> np.ndarray:
    N, d = x.shape
    E = w.shape[0]
    out = np.empty((N, E), np.float32)
    b = None if bias is None else np.ascontiguousarray(bias, np.float32)
    _load().oracle_router_logits(_p(x), _p(w), _p(b), _i64(N), int(d), int(E), _dt(dtype), _p(out))
    return out


def softmax(logits: np.ndarray) -> np.ndarray:
    logits = np.ascontiguousarray(logits, np.float32)
    N, E = logits.shape
    out = np.empty((N, E), np.float32)
    _load().oracle_softmax(_p(logits), _i64(N), int(E), _p(out))
    return out


def topk(scores: np.ndarray, k: int):
    scores = np.ascontiguousarray(scores, np.float32)
    N, E = scores.shape
    idx = np.empty((N, k), np.int32)
    val = np.empty((N, k), np.float32)
    load = np.empty((E,), np.int32)
    _load().oracle_topk(_p(scores), _i64(N), int(E), int(k), _p(idx), _p(val), _p(load))
    return idx, val, load


def token_drop(scores: np.ndarray, topk_idx: np.ndarray, C: int):
    scores = np.ascontiguousarray(scores, np.float32)
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    N, E = scores.shape
    k = topk_idx.shape[1]
    W = (E + 63) // 64
    keep = np.empty((N, W), np.uint64)
    kept = np.empty((E,), np.int32)
    off = np.empty((E + 1,), np.int32)
    slot_row = np.empty((N, k), np.int32)
    _load().oracle_token_drop(_p(scores), _p(topk_idx), _i64(N), int(E), int(k), _i64(C),
                              _p(keep), _p(kept), _p(off), _p(slot_row))
    return dict(keep_mask=keep, kept=kept, offsets=off, slot_row=slot_row)


def expanded_drop(scores: np.ndarray, topk_idx: np.ndarray, C: int, D: int,
                  token_group: Optional[np.ndarray] = None):
    scores = np.ascontiguousarray(scores, np.float32)
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    N, E = scores.shape
    k = topk_idx.shape[1]
    assert E % D == 0
    m = E // D
    W = (E + 63) // 64
    keep = np.empty((N, W), np.uint64)
    cand = np.empty((E,), np.int32)
    kept = np.empty((E,), np.int32)
    off = np.empty((E + 1,), np.int32)
    slot_row = np.empty((N, k + m), np.int32)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    _load().oracle_expanded_drop(_p(scores), _p(topk_idx), _i64(N), int(E), int(k), _i64(C), int(D),
                                 _p(tg), _p(keep), _p(cand), _p(kept), _p(off), _p(slot_row))
    return dict(keep_mask=keep, cand=cand, kept=kept, offsets=off, slot_row=slot_row)


METRICS = {"score": 0, "order": 1, "reverse_order": 2, "random": 3}


def drop_keys(metric: str, seed: int, scores: np.ndarray, idx: Optional[np.ndarray], E: int) -> np.ndarray:
    """32-bit drop keys for every entry of scores [N,cols] (idx [N,cols] expert ids, or None for a
    dense [N,E] matrix)."""
    scores = np.ascontiguousarray(scores, np.float32)
    N, cols = scores.shape
    ix = None if idx is None else np.ascontiguousarray(idx, np.int32)
    out = np.empty((N, cols), np.uint32)
    _load().oracle_drop_keys(METRICS[metric], ctypes.c_uint64(seed), _p(scores), _p(ix), _i64(N), int(cols), int(E),
                             _p(out))
    return out


def drop_keyed(keys: np.ndarray, topk_idx: np.ndarray, C: int, D: int = 1, expanded: bool = False,
               token_group: Optional[np.ndarray] = None):
    """Token Drop (expanded=False) or Expanded Drop on a dense [N,E] matrix of 32-bit keys."""
    keys = np.ascontiguousarray(keys, np.uint32)
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    N, E = keys.shape
    k = topk_idx.shape[1]
    m = E // D if expanded else 0
    W = (E + 63) // 64
    keep = np.empty((N, W), np.uint64)
    cand = np.empty((E,), np.int32)
    kept = np.empty((E,), np.int32)
    off = np.empty((E + 1,), np.int32)
    slot_row = np.empty((N, k + m), np.int32)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    _load().oracle_drop_keyed(_p(keys), _p(topk_idx), _i64(N), int(E), int(k), _i64(C), int(D), int(bool(expanded)),
                              _p(tg), _p(keep), _p(cand), _p(kept), _p(off), _p(slot_row))
    return dict(keep_mask=keep, cand=cand, kept=kept, offsets=off, slot_row=slot_row)


def priority_keys(base: np.ndarray, idx: Optional[np.ndarray], E: int, exact: bool,
                  token_class: Optional[np.ndarray] = None, topk_idx: Optional[np.ndarray] = None) -> np.ndarray:
    """Keys with a priority class in the two high bits: 2 * [pair is a top-k pair] + token_class[t]
    (modality-first dropping; Expanded Drop as substitution only)."""
    base = np.ascontiguousarray(base, np.uint32)
    N, cols = base.shape
    ix = None if idx is None else np.ascontiguousarray(idx, np.int32)
    tc = None if token_class is None else np.ascontiguousarray(token_class, np.uint8)
    tk = None if topk_idx is None else np.ascontiguousarray(topk_idx, np.int32)
    k = 0 if tk is None else tk.shape[1]
    out = np.empty((N, cols), np.uint32)
    rc = _load().oracle_priority_keys(_p(base), _p(ix), _i64(N), int(cols), int(E), int(bool(exact)), _p(tc), _p(tk),
                                      int(k), _p(out))
    if rc != 0:
        raise ValueError("exact keys must be below 2^30")
    return out


def limit_experts(scores: np.ndarray, keep_mask: np.ndarray, k_max: int) -> np.ndarray:
    """'w/ max': every token retains at most k_max of the experts that kept it, the best by score."""
    scores = np.ascontiguousarray(scores, np.float32)
    N, E = scores.shape
    out = np.ascontiguousarray(keep_mask, np.uint64).copy()
    _load().oracle_limit_experts(_p(scores), _i64(N), int(E), int(k_max), _p(out))
    return out


def rows_from_mask(keep_mask: np.ndarray, topk_idx: np.ndarray, E: int, slots: int, D: int = 1,
                   token_group: Optional[np.ndarray] = None):
    """Counts, offsets and slot rows of a keep mask (segments in ascending token order)."""
    keep_mask = np.ascontiguousarray(keep_mask, np.uint64)
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    N, k = topk_idx.shape
    kept = np.empty((E,), np.int32)
    off = np.empty((E + 1,), np.int32)
    slot_row = np.empty((N, slots), np.int32)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    rc = _load().oracle_rows_from_mask(_p(keep_mask), _p(topk_idx), _i64(N), int(E), int(k), int(slots), int(D),
                                       _p(tg), _p(kept), _p(off), _p(slot_row))
    if rc != 0:
        raise ValueError("mask has a bit outside the token's slots")
    return dict(kept=kept, offsets=off, slot_row=slot_row)


def device_capacity(N: int, E: int, k: int, D: int, gamma: float, round_mode: str = "ceil") -> int:
    out = ctypes.c_int64(0)
    rc = _load().oracle_device_capacity(_i64(N), int(E), int(k), int(D), ctypes.c_double(gamma),
                                        0 if round_mode == "ceil" else 1, ctypes.byref(out))
    if rc != 0:
        raise ValueError("bad device capacity arguments")
    return out.value


def device_drop(scores: np.ndarray, topk_idx: np.ndarray, C_dev: int, D: int, expanded: bool,
                token_group: Optional[np.ndarray] = None):
    """Capacity enforced per device (sum over its E/D experts) instead of per expert."""
    scores = np.ascontiguousarray(scores, np.float32)
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    N, E = scores.shape
    k = topk_idx.shape[1]
    assert E % D == 0
    m = E // D
    W = (E + 63) // 64
    slots = k + m if expanded else k
    keep = np.empty((N, W), np.uint64)
    cand = np.empty((E,), np.int32)
    kept = np.empty((E,), np.int32)
    off = np.empty((E + 1,), np.int32)
    slot_row = np.empty((N, slots), np.int32)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    _load().oracle_device_drop(_p(scores), _p(topk_idx), _i64(N), int(E), int(k), _i64(C_dev), int(D),
                               int(bool(expanded)), _p(tg), _p(keep), _p(cand), _p(kept), _p(off), _p(slot_row))
    return dict(keep_mask=keep, cand=cand, kept=kept, offsets=off, slot_row=slot_row)


def permute(x: Optional[np.ndarray], scores, topk_idx, slot_row, A: int, D: int, dtype: str,
            token_group: Optional[np.ndarray] = None):
    scores = np.ascontiguousarray(scores, np.float32)
    N, E = scores.shape
    k = topk_idx.shape[1]
    slots = slot_row.shape[1]
    d = 0 if x is None else x.shape[1]
    x_perm = None if x is None else np.zeros((A, d), x.dtype)
    perm_token = np.full((A,), -1, np.int32)
    perm_weight = np.zeros((A,), np.float32)
    perm_expert = np.full((A,), -1, np.int32)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    _load().oracle_permute(_p(x), _i64(N), int(d), int(E), int(k), int(slots), int(D), _dt(dtype),
                           _p(scores), _p(np.ascontiguousarray(topk_idx, np.int32)), _p(tg),
                           _p(np.ascontiguousarray(slot_row, np.int32)), _p(x_perm), _p(perm_token),
                           _p(perm_weight), _p(perm_expert))
    return dict(x_perm=x_perm, perm_token=perm_token, perm_weight=perm_weight, perm_expert=perm_expert)


def expert_ffn(x_rows: np.ndarray, row_expert: Optional[np.ndarray], w_gate, w_up, w_down, dtype: str):
    R, d = x_rows.shape
    F = w_gate.shape[-2]
    y = np.empty((R, d), np.float64)
    re_ = None if row_expert is None else np.ascontiguousarray(row_expert, np.int32)
    _load().oracle_expert_ffn(_p(x_rows), _p(re_), _i64(R), int(d), int(F), _dt(dtype),
                              _p(w_gate), _p(w_up), _p(w_down), _p(y))
    return y


def combine(y_perm: np.ndarray, slot_row, scores, topk_idx, D: int, y_shared: Optional[np.ndarray] = None,
            token_group: Optional[np.ndarray] = None):
    scores = np.ascontiguousarray(scores, np.float32)
    N, E = scores.shape
    k = topk_idx.shape[1]
    slots = slot_row.shape[1]
    d = y_perm.shape[1]
    y = np.empty((N, d), np.float64)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    ys = None if y_shared is None else np.ascontiguousarray(y_shared, np.float64)
    _load().oracle_combine(_p(np.ascontiguousarray(y_perm, np.float64)),
                           _p(np.ascontiguousarray(slot_row, np.int32)), _p(scores),
                           _p(np.ascontiguousarray(topk_idx, np.int32)), _p(tg), _i64(N), int(d), int(E),
                           int(k), int(slots), int(D), _p(ys), _p(y))
    return y


def layer_tokens(x, tokens, scores, topk_idx, slot_row, D: int, w_gate, w_up, w_down, dtype: str,
                 token_group: Optional[np.ndarray] = None):
    """Layer output (routed experts only) for the listed tokens, [len(tokens), d] float64."""
    scores = np.ascontiguousarray(scores, np.float32)
    N, E = scores.shape
    k = topk_idx.shape[1]
    slots = slot_row.shape[1]
    d = x.shape[1]
    F = w_gate.shape[-2]
    tokens = np.ascontiguousarray(tokens, np.int32)
    out = np.empty((len(tokens), d), np.float64)
    tg = None if token_group is None else np.ascontiguousarray(token_group, np.int32)
    _load().oracle_layer_tokens(_p(x), _p(tokens), _i64(len(tokens)), _i64(N), int(d), int(E), int(k),
                                int(slots), int(D), int(F), _dt(dtype), _p(scores),
                                _p(np.ascontiguousarray(topk_idx, np.int32)), _p(tg),
                                _p(np.ascontiguousarray(slot_row, np.int32)), _p(w_gate), _p(w_up),
                                _p(w_down), _p(out))
    return out


def stats(load: np.ndarray, N: int, k: int, C: int):
    load = np.ascontiguousarray(load, np.int32)
    out = np.empty((4,), np.float64)
    _load().oracle_stats(_p(load), int(load.shape[0]), _i64(N), int(k), _i64(C), _p(out))
    return dict(max_over_mean=out[0], dropped_fraction=out[1], max_load=out[2], total=out[3])


def layer_forward(x, w_router, bias, w_gate, w_up, w_down, k: int, gamma: float, D: int, mode: str,
                  dtype: str, logits: Optional[np.ndarray] = None, shared=None, round_mode: str = "ceil",
                  token_group: Optional[np.ndarray] = None):
    """Whole layer on the CPU.  mode in {"nodrop", "token_drop", "expanded_drop"}.
    If `logits` is given it replaces the router GEMM (parity checks downstream of the router
    start from identical fp32 logits).  token_group: explicit home device per token for Expanded
    Drop (default: contiguous blocks)."""
    N, d = x.shape
    E = w_router.shape[0]
    if logits is None:
        logits = router_logits(x, w_router, bias, dtype)
    scores = softmax(logits)
    idx, val, load = topk(scores, k)
    C = N if mode == "nodrop" else capacity(N, E, k, gamma, round_mode)
    if mode == "expanded_drop":
        r = expanded_drop(scores, idx, C, D, token_group=token_group)
        Dp = D
    else:
        r = token_drop(scores, idx, C)
        Dp = 0
    A = int(r["offsets"][-1])
    p = permute(x, scores, idx, r["slot_row"], A, Dp, dtype, token_group)
    y_perm = expert_ffn(p["x_perm"], p["perm_expert"], w_gate, w_up, w_down, dtype)
    y_sh = None
    if shared is not None:
        y_sh = expert_ffn(x, None, shared[0], shared[1], shared[2], dtype)
    y = combine(y_perm, r["slot_row"], scores, idx, Dp, y_sh, token_group)
    return dict(logits=logits, scores=scores, topk_idx=idx, topk_score=val, load=load, C=C, A=A, y=y,
                y_perm=y_perm, **r, **p)


def ep_layer(x_ranks, w_router, bias, w_gate, w_up, w_down, k: int, gamma: float, mode: str, dtype: str,
             logits_ranks=None, round_mode: str = "ceil"):
    """The layer under expert parallelism with per-rank capacity, rank by rank and message by message.

    The paper's deployment is data parallel over the tokens and expert parallel over the experts
    (experimental set-up), and the capacity is applied "within each local device" so that no rank
    needs another rank's load and tokens are dropped before the all-to-all (Capacity-Aware Token
    Drop paragraph, Figure 3).  With R = len(x_ranks) ranks and m = E/R experts per rank:
      1. rank r routes its own N_r tokens (Eq. 1) and applies C_r = capacity(N_r, E, k, gamma) to
         them alone: Token Drop, or Expanded Drop with D = R devices and every one of its tokens at
         home on device r (its candidates are its top-k experts plus the m experts rank r owns);
      2. its kept rows, expert-major and token-ascending, are cut by owner: the rows of experts
         r'*m .. r'*m+m-1 form the message r -> r' (at most m * C_r rows);
      3. owner r' runs E_i(x) (Eq. 2) on what it received, with its own m experts only;
      4. the results travel back in the same order and rank r combines them (Eq. 2).
    x_ranks / logits_ranks: one array per rank.  Returns per-rank outputs and the message sizes."""
    R = len(x_ranks)
    E = w_router.shape[0]
    assert E % R == 0
    m = E // R
    ranks = []
    for r in range(R):
        x = x_ranks[r]
        N = x.shape[0]
        logits = router_logits(x, w_router, bias, dtype) if logits_ranks is None else logits_ranks[r]
        scores = softmax(logits)
        idx, val, load = topk(scores, k)
        C = N if mode == "nodrop" else capacity(N, E, k, gamma, round_mode)
        tg = None
        if mode == "expanded_drop":
            tg = np.full((N,), r, np.int32)
            dr = expanded_drop(scores, idx, C, R, token_group=tg)
            Dp = R
        else:
            dr = token_drop(scores, idx, C)
            Dp = 0
        A = int(dr["offsets"][-1])
        p = permute(x, scores, idx, dr["slot_row"], A, Dp, dtype, tg)
        ranks.append(dict(N=N, C=C, scores=scores, topk_idx=idx, load=load, Dp=Dp, tg=tg, A=A, **dr, **p))
    # messages r -> r': rows of the experts r' owns, and how many of each
    off = [rk["offsets"] for rk in ranks]
    send = [[ranks[r]["x_perm"][off[r][o * m]:off[r][(o + 1) * m]] for o in range(R)] for r in range(R)]
    send_counts = np.array([[ranks[r]["kept"][o * m:(o + 1) * m] for o in range(R)] for r in range(R)], np.int64)
    # owners: E_i(x) on the received rows with the owner's m experts (weights [o*m, (o+1)*m) only)
    back = [[None] * R for _ in range(R)]
    for o in range(R):
        wg, wu, wd = (np.ascontiguousarray(w[o * m:(o + 1) * m]) for w in (w_gate, w_up, w_down))
        for r in range(R):
            rows = np.ascontiguousarray(send[r][o])
            local = np.repeat(np.arange(m, dtype=np.int32), send_counts[r, o])
            back[r][o] = (expert_ffn(rows, local, wg, wu, wd, dtype) if len(rows)
                          else np.zeros((0, rows.shape[1]), np.float64))
    ys = []
    for r in range(R):
        rk = ranks[r]
        y_perm = np.concatenate([back[r][o] for o in range(R)], axis=0) if rk["A"] else np.zeros((0, x_ranks[r].shape[1]))
        ys.append(combine(y_perm, rk["slot_row"], rk["scores"], rk["topk_idx"], rk["Dp"], None, rk["tg"]))
    return dict(y=ys, ranks=ranks, send_counts=send_counts, m=m)
