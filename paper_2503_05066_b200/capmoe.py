"""ctypes binding of libcapmoe.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the layer runs inside the CUDA
library.  If the shared library is missing or cannot be loaded, every call raises: there is
no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import math
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libcapmoe.so")
_lib = None

OK, EINVAL, EUNSUPPORTED, EWORKSPACE, ECUDA, ETIMEOUT, EINDEX = range(7)
F32, BF16 = 0, 1
MODE_NODROP, MODE_TOKEN_DROP, MODE_EXPANDED_DROP = 0, 1, 2
MODES = {"nodrop": 0, "token_drop": 1, "expanded_drop": 2, "device_token_drop": 3, "device_expanded_drop": 4}

EXPORTS = ["capmoe_capacity", "capmoe_max_rows", "capmoe_device_max_rows", "capmoe_drop_workspace_bytes", "capmoe_status_str",
           "capmoe_last_cuda_error", "capmoe_launch_count", "capmoe_ffn_uses_tensor_cores", "capmoe_route",
           "capmoe_token_drop", "capmoe_token_drop_static", "capmoe_expanded_drop", "capmoe_device_capacity",
           "capmoe_device_drop", "capmoe_drop_keys", "capmoe_priority_keys", "capmoe_limit_experts",
           "capmoe_rows_from_mask", "capmoe_permute", "capmoe_grouped_ffn",
           "capmoe_combine", "capmoe_layer_forward", "capmoe_layer_forward_host", "capmoe_debug_wait_probe",
           "capmoe_grouped_ffn_segments", "capmoe_debug_ffn_variant", "capmoe_ep_plan", "capmoe_ep_forward_dispatch", "capmoe_ep_forward_experts", "capmoe_ep_forward_combine", "capmoe_ep_segments", "capmoe_ep_dispatch",
           "capmoe_ep_combine", "capmoe_debug_read_probe", "capmoe_debug_check_indices"]


class CapmoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().capmoe_status_str(status).decode()
        if status == ECUDA:
            msg += " (" + lib().capmoe_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {msg} [status {status}]")


class _Layer(ctypes.Structure):
    _fields_ = [
        ("N", ctypes.c_int64), ("d", ctypes.c_int), ("E", ctypes.c_int), ("k", ctypes.c_int),
        ("F", ctypes.c_int), ("D", ctypes.c_int), ("dtype", ctypes.c_int),
        ("mode", ctypes.c_int), ("C", ctypes.c_int64), ("straggler", ctypes.c_int),
        ("x", ctypes.c_void_p), ("w_router", ctypes.c_void_p), ("bias", ctypes.c_void_p),
        ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p), ("w_down", ctypes.c_void_p),
        ("ws_gate", ctypes.c_void_p), ("ws_up", ctypes.c_void_p), ("ws_down", ctypes.c_void_p),
        ("F_shared", ctypes.c_int),
        ("logits", ctypes.c_void_p), ("scores", ctypes.c_void_p), ("topk_idx", ctypes.c_void_p),
        ("topk_score", ctypes.c_void_p), ("load", ctypes.c_void_p),
        ("keep_mask", ctypes.c_void_p), ("cand", ctypes.c_void_p), ("kept", ctypes.c_void_p),
        ("expert_offsets", ctypes.c_void_p), ("slot_row", ctypes.c_void_p),
        ("x_perm", ctypes.c_void_p), ("perm_token", ctypes.c_void_p), ("perm_weight", ctypes.c_void_p),
        ("h_ws", ctypes.c_void_p), ("y_perm", ctypes.c_void_p), ("A_max", ctypes.c_int64),
        ("hs_ws", ctypes.c_void_p), ("y_shared", ctypes.c_void_p), ("one_segment", ctypes.c_void_p),
        ("y", ctypes.c_void_p),
        ("drop_ws", ctypes.c_void_p), ("drop_ws_bytes", ctypes.c_size_t),
        ("dev_status", ctypes.c_void_p),
        ("stage_events", ctypes.POINTER(ctypes.c_void_p)),
        ("metric", ctypes.c_int), ("metric_seed", ctypes.c_uint64), ("token_class", ctypes.c_void_p),
        ("topk_first", ctypes.c_int), ("max_experts", ctypes.c_int), ("drop_keys", ctypes.c_void_p),
        ("bad", ctypes.c_void_p), ("debug_checks", ctypes.c_int),
    ]

class _EPRank(ctypes.Structure):
    _fields_ = [
        ("N", ctypes.c_int64), ("d", ctypes.c_int), ("E", ctypes.c_int), ("k", ctypes.c_int),
        ("F", ctypes.c_int), ("dtype", ctypes.c_int),
        ("R", ctypes.c_int), ("rank", ctypes.c_int), ("mode", ctypes.c_int),
        ("C_local", ctypes.c_int64), ("C", ctypes.c_int64),
        ("x", ctypes.c_void_p), ("w_router", ctypes.c_void_p), ("bias", ctypes.c_void_p),
        ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p), ("w_down", ctypes.c_void_p),
        ("logits", ctypes.c_void_p), ("scores", ctypes.c_void_p), ("topk_idx", ctypes.c_void_p),
        ("topk_score", ctypes.c_void_p), ("load", ctypes.c_void_p),
        ("keep_mask", ctypes.c_void_p), ("cand", ctypes.c_void_p), ("kept", ctypes.c_void_p),
        ("expert_offsets", ctypes.c_void_p), ("slot_row", ctypes.c_void_p),
        ("slot_row_ep", ctypes.c_void_p), ("token_group", ctypes.c_void_p),
        ("perm_token", ctypes.c_void_p), ("perm_weight", ctypes.c_void_p),
        ("x_send", ctypes.c_void_p), ("y_ret", ctypes.c_void_p),
        ("peer_x", ctypes.c_void_p), ("peer_y", ctypes.c_void_p),
        ("x_recv", ctypes.c_void_p), ("h_ws", ctypes.c_void_p), ("y_recv", ctypes.c_void_p),
        ("cnt_recv", ctypes.c_void_p), ("seg_begin", ctypes.c_void_p), ("seg_end", ctypes.c_void_p),
        ("y", ctypes.c_void_p),
        ("drop_ws", ctypes.c_void_p), ("drop_ws_bytes", ctypes.c_size_t),
        ("dev_status", ctypes.c_void_p), ("bad", ctypes.c_void_p),
    ]

N_STAGE_EVENTS = 8
FFN_STATUS_WORDS = 128     # CAPMOE_FFN_STATUS_WORDS: status word + scratch of the FFN's tile schedulers
STAGE_NAMES = ["route", "drop", "permute", "ffn_gate_up", "ffn_down", "shared_ffn", "combine"]


def lib():
    """The loaded CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_05066_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        L.capmoe_status_str.restype = ctypes.c_char_p
        L.capmoe_last_cuda_error.restype = ctypes.c_char_p
        L.capmoe_launch_count.restype = ctypes.c_uint64
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_contiguous(), "capmoe tensors must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dt(t_or_dtype) -> int:
    dt = t_or_dtype.dtype if isinstance(t_or_dtype, torch.Tensor) else t_or_dtype
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise CapmoeError(EUNSUPPORTED, f"dtype {dt}")


def _check(rc: int, where: str):
    if rc != OK:
        raise CapmoeError(rc, where)


def _i64(v):
    return ctypes.c_int64(int(v))


# ----------------------------------------------------------------------------- host helpers
def capacity(N: int, E: int, k: int, gamma: float, round_mode: str = "ceil") -> int:
    out = ctypes.c_int64(0)
    _check(lib().capmoe_capacity(_i64(N), int(E), int(k), ctypes.c_double(gamma),
                                 0 if round_mode == "ceil" else 1, ctypes.byref(out)), "capmoe_capacity")
    return out.value


def max_rows(N: int, E: int, k: int, D: int, C: int, expanded: bool) -> int:
    out = ctypes.c_int64(0)
    _check(lib().capmoe_max_rows(_i64(N), int(E), int(k), int(D), _i64(C), int(bool(expanded)),
                                 ctypes.byref(out)), "capmoe_max_rows")
    return out.value


def device_max_rows(N: int, E: int, k: int, D: int, C_dev: int, expanded: bool) -> int:
    out = ctypes.c_int64(0)
    _check(lib().capmoe_device_max_rows(_i64(N), int(E), int(k), int(D), _i64(C_dev), int(bool(expanded)),
                                        ctypes.byref(out)), "capmoe_device_max_rows")
    return out.value


def drop_workspace_bytes(N: int, E: int, k: int, D: int, expanded: bool) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().capmoe_drop_workspace_bytes(_i64(N), int(E), int(k), int(D), int(bool(expanded)),
                                             ctypes.byref(out)), "capmoe_drop_workspace_bytes")
    return out.value


def launch_count() -> int:
    return int(lib().capmoe_launch_count())


def ffn_uses_tensor_cores(d: int, F: int, dtype) -> bool:
    return bool(lib().capmoe_ffn_uses_tensor_cores(int(d), int(F), _dt(dtype)))


# ----------------------------------------------------------------------------- stages
def route(x, w_router, bias, k: int, logits_in=None, out=None, stream=None):
    """-> dict(logits, scores, topk_idx, topk_score, load); `out` may hand in those buffers to be reused."""
    if logits_in is not None:
        N, E = logits_in.shape
        d, dev, dt = 0, logits_in.device, F32
    else:
        N, d = x.shape
        E = w_router.shape[0]
        dev, dt = x.device, _dt(x)
    f32 = dict(device=dev, dtype=torch.float32)
    i32 = dict(device=dev, dtype=torch.int32)
    if out is None:
        out = dict(logits=torch.empty((N, E), **f32), scores=torch.empty((N, E), **f32),
                   topk_idx=torch.empty((N, k), **i32), topk_score=torch.empty((N, k), **f32),
                   load=torch.empty((E,), **i32))
    _check(lib().capmoe_route(_ptr(x), _ptr(w_router), _ptr(bias), _ptr(logits_in), _i64(N), int(d), int(E),
                              int(k), dt, _ptr(out["logits"]), _ptr(out["scores"]), _ptr(out["topk_idx"]),
                              _ptr(out["topk_score"]), _ptr(out["load"]), _stream(stream)), "capmoe_route")
    return out


def token_drop(topk_score, topk_idx, E: int, C: int, ws=None, stream=None):
    """-> dict(keep_mask, kept, offsets, slot_row)"""
    N, k = topk_idx.shape
    dev = topk_idx.device
    W = (E + 63) // 64
    if ws is None:
        ws = torch.empty((drop_workspace_bytes(N, E, k, 0, False),), device=dev, dtype=torch.uint8)
    out = dict(keep_mask=torch.empty((N, W), device=dev, dtype=torch.int64),
               kept=torch.empty((E,), device=dev, dtype=torch.int32),
               offsets=torch.empty((E + 1,), device=dev, dtype=torch.int32),
               slot_row=torch.empty((N, k), device=dev, dtype=torch.int32))
    _check(lib().capmoe_token_drop(_ptr(topk_score), _ptr(topk_idx), _i64(N), int(E), int(k), _i64(C),
                                   _ptr(out["keep_mask"]), _ptr(out["kept"]), _ptr(out["offsets"]),
                                   _ptr(out["slot_row"]), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                   _stream(stream)), "capmoe_token_drop")
    return out


STATIC_DROP_MAX_PAIRS = 1 << 20


def token_drop_static(topk_score, topk_idx, E: int, C: int, stream=None):
    """Token Drop through the entry point that needs no workspace from the caller (the scratch
    is a fixed array inside the library, shared by all calls on the device: do not overlap calls).
    Limited to N*k <= STATIC_DROP_MAX_PAIRS.  -> dict(keep_mask, kept, offsets, slot_row)"""
    N, k = topk_idx.shape
    dev = topk_idx.device
    W = (E + 63) // 64
    out = dict(keep_mask=torch.empty((N, W), device=dev, dtype=torch.int64),
               kept=torch.empty((E,), device=dev, dtype=torch.int32),
               offsets=torch.empty((E + 1,), device=dev, dtype=torch.int32),
               slot_row=torch.empty((N, k), device=dev, dtype=torch.int32))
    rc = lib().capmoe_token_drop_static(_ptr(topk_score), _ptr(topk_idx), _i64(N), int(E), int(k), _i64(C),
                                        _ptr(out["keep_mask"]), _ptr(out["kept"]), _ptr(out["offsets"]),
                                        _ptr(out["slot_row"]), _stream(stream))
    if rc == EWORKSPACE:
        raise CapmoeError(rc, f"capmoe_token_drop_static: N*k = {N * k} exceeds the built-in scratch "
                              f"({STATIC_DROP_MAX_PAIRS} pairs)")
    _check(rc, "capmoe_token_drop_static")
    return out


def expanded_drop(scores, topk_idx, C: int, D: int, token_group=None, ws=None, stream=None):
    """-> dict(keep_mask, cand, kept, offsets, slot_row)"""
    N, E = scores.shape
    k = topk_idx.shape[1]
    dev = scores.device
    if D < 1 or E % D != 0:
        raise CapmoeError(EINVAL, "capmoe_expanded_drop: E % D != 0")
    m = E // D
    W = (E + 63) // 64
    if ws is None:
        ws = torch.empty((drop_workspace_bytes(N, E, k, D, True),), device=dev, dtype=torch.uint8)
    out = dict(keep_mask=torch.empty((N, W), device=dev, dtype=torch.int64),
               cand=torch.empty((E,), device=dev, dtype=torch.int32),
               kept=torch.empty((E,), device=dev, dtype=torch.int32),
               offsets=torch.empty((E + 1,), device=dev, dtype=torch.int32),
               slot_row=torch.empty((N, k + m), device=dev, dtype=torch.int32))
    _check(lib().capmoe_expanded_drop(_ptr(scores), _ptr(topk_idx), _i64(N), int(E), int(k), _i64(C), int(D),
                                      _ptr(token_group), _ptr(out["keep_mask"]), _ptr(out["cand"]),
                                      _ptr(out["kept"]), _ptr(out["offsets"]), _ptr(out["slot_row"]), _ptr(ws),
                                      ctypes.c_size_t(ws.numel()), _stream(stream)), "capmoe_expanded_drop")
    return out


METRICS = {"score": 0, "order": 1, "reverse_order": 2, "random": 3}


def drop_keys(metric: str, seed: int, scores, idx, E: int, stream=None):
    """32-bit drop keys for every entry of scores [N,cols] (idx [N,cols] expert ids, or None for a
    dense [N,E] matrix).  Returned as a float32-typed tensor holding the key bit patterns, so it
    can be passed straight to token_drop / expanded_drop / device_drop in place of the scores."""
    N, cols = scores.shape
    keys = torch.empty((N, cols), device=scores.device, dtype=torch.float32)
    _check(lib().capmoe_drop_keys(METRICS[metric], ctypes.c_uint64(seed), _ptr(scores), _ptr(idx), _i64(N),
                                  int(cols), int(E), _ptr(keys), _stream(stream)), "capmoe_drop_keys")
    return keys


def priority_keys(base, idx, E: int, exact: bool, token_class=None, topk_idx=None, stream=None):
    """Keys with a priority class above the metric's key: 2 * [pair is one of the token's top-k]
    (when topk_idx is given: Expanded Drop as substitution only) + token_class[t] (uint8, 1 = the
    protected modality).  base: the float32-typed key tensor drop_keys returns; same type back."""
    N, cols = base.shape
    keys = torch.empty_like(base)
    k = 0 if topk_idx is None else topk_idx.shape[1]
    _check(lib().capmoe_priority_keys(_ptr(base), _ptr(idx), _i64(N), int(cols), int(E), int(bool(exact)),
                                      _ptr(token_class), _ptr(topk_idx), int(k), _ptr(keys), _stream(stream)),
           "capmoe_priority_keys")
    return keys


def limit_experts(scores, keep_mask, k_max: int, stream=None):
    """'w/ max': edits keep_mask in place so that no token sits on more than k_max experts."""
    N, E = scores.shape
    _check(lib().capmoe_limit_experts(_ptr(scores), _i64(N), int(E), int(k_max), _ptr(keep_mask), _stream(stream)),
           "capmoe_limit_experts")
    return keep_mask


def rows_from_mask(keep_mask, topk_idx, E: int, slots: int, D: int = 1, token_group=None, ws=None, stream=None):
    """-> dict(kept, offsets, slot_row, bad) for a keep mask whose bits lie on the tokens' slots."""
    N, k = topk_idx.shape
    dev = topk_idx.device
    need = ((N + 255) // 256) * E * 4
    if ws is None:
        ws = torch.empty((max(need, 16),), device=dev, dtype=torch.uint8)
    out = dict(kept=torch.empty((E,), device=dev, dtype=torch.int32),
               offsets=torch.empty((E + 1,), device=dev, dtype=torch.int32),
               slot_row=torch.empty((N, slots), device=dev, dtype=torch.int32),
               bad=torch.zeros((1,), device=dev, dtype=torch.int32))
    _check(lib().capmoe_rows_from_mask(_ptr(keep_mask), _ptr(topk_idx), _i64(N), int(E), int(k), int(slots), int(D),
                                       _ptr(token_group), _ptr(out["kept"]), _ptr(out["offsets"]),
                                       _ptr(out["slot_row"]), _ptr(out["bad"]), _ptr(ws),
                                       ctypes.c_size_t(ws.numel()), _stream(stream)), "capmoe_rows_from_mask")
    return out


def device_capacity(N: int, E: int, k: int, D: int, gamma: float, round_mode: str = "ceil") -> int:
    out = ctypes.c_int64(0)
    _check(lib().capmoe_device_capacity(_i64(N), int(E), int(k), int(D), ctypes.c_double(gamma),
                                        0 if round_mode == "ceil" else 1, ctypes.byref(out)),
           "capmoe_device_capacity")
    return out.value


def device_drop(scores, topk_idx, C_dev: int, D: int, expanded: bool, token_group=None, ws=None, stream=None):
    """Capacity per device instead of per expert.  -> dict(keep_mask, cand, kept, offsets, slot_row)"""
    N, E = scores.shape
    k = topk_idx.shape[1]
    dev = scores.device
    if D < 1 or E % D != 0:
        raise CapmoeError(EINVAL, "capmoe_device_drop: E % D != 0")
    m = E // D
    W = (E + 63) // 64
    slots = k + m if expanded else k
    if ws is None:
        ws = torch.empty((drop_workspace_bytes(N, E, k, D, expanded),), device=dev, dtype=torch.uint8)
    out = dict(keep_mask=torch.empty((N, W), device=dev, dtype=torch.int64),
               cand=torch.empty((E,), device=dev, dtype=torch.int32),
               kept=torch.empty((E,), device=dev, dtype=torch.int32),
               offsets=torch.empty((E + 1,), device=dev, dtype=torch.int32),
               slot_row=torch.empty((N, slots), device=dev, dtype=torch.int32))
    _check(lib().capmoe_device_drop(_ptr(scores), _ptr(topk_idx), _i64(N), int(E), int(k), _i64(C_dev), int(D),
                                    int(bool(expanded)), _ptr(token_group), _ptr(out["keep_mask"]),
                                    _ptr(out["cand"]), _ptr(out["kept"]), _ptr(out["offsets"]),
                                    _ptr(out["slot_row"]), _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(stream)),
           "capmoe_device_drop")
    return out


def permute(x, scores, topk_idx, slot_row, A_max: int, D: int = 0, token_group=None, out=None, stream=None):
    """-> dict(x_perm [A_max,d], perm_token [A_max], perm_weight [A_max]); rows >= A are left unwritten.
    `out` may hand in those three buffers to be reused."""
    N, d = x.shape
    E = scores.shape[1]
    k = topk_idx.shape[1]
    slots = slot_row.shape[1]
    dev = x.device
    if out is None:
        out = dict(x_perm=torch.zeros((A_max, d), device=dev, dtype=x.dtype),
                   perm_token=torch.full((A_max,), -1, device=dev, dtype=torch.int32),
                   perm_weight=torch.zeros((A_max,), device=dev, dtype=torch.float32))
    _check(lib().capmoe_permute(_ptr(x), _i64(N), int(d), int(E), int(k), int(slots), int(D), _dt(x),
                                _ptr(scores), _ptr(topk_idx), _ptr(token_group), _ptr(slot_row),
                                _ptr(out["x_perm"]), _ptr(out["perm_token"]), _ptr(out["perm_weight"]),
                                _stream(stream)), "capmoe_permute")
    return out


def grouped_ffn(x_perm, offsets, w_gate, w_up, w_down, D_straggler: int = 0, h_ws=None, y_perm=None,
                dev_status=None, stream=None):
    """-> y_perm [A_max, d].  dev_status: int32 [FFN_STATUS_WORDS] (word 0 = device status), made here if None."""
    A_max, d = x_perm.shape
    E, F, _ = w_gate.shape
    dev = x_perm.device
    if dev_status is None:
        dev_status = torch.zeros((FFN_STATUS_WORDS,), device=dev, dtype=torch.int32)
    if h_ws is None:
        h_ws = torch.empty((A_max, F), device=dev, dtype=x_perm.dtype)
    if y_perm is None:
        y_perm = torch.zeros((A_max, d), device=dev, dtype=x_perm.dtype)
    _check(lib().capmoe_grouped_ffn(_ptr(x_perm), _ptr(offsets), int(E), int(d), int(F), _dt(x_perm),
                                    _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(h_ws), _ptr(y_perm),
                                    _i64(A_max), int(D_straggler), _ptr(dev_status), _stream(stream)),
           "capmoe_grouped_ffn")
    return y_perm


def grouped_ffn_segments(x_rows, seg_begin, seg_end, w_gate, w_up, w_down, w_mod: int, h_ws=None, y_rows=None,
                         dev_status=None, stream=None):
    """SwiGLU FFN over explicit row segments; segment s uses weight block s % w_mod.  -> y_rows"""
    rows, d = x_rows.shape
    F = w_gate.shape[-2]
    dev = x_rows.device
    if dev_status is None:
        dev_status = torch.zeros((FFN_STATUS_WORDS,), device=dev, dtype=torch.int32)
    if h_ws is None:
        h_ws = torch.empty((rows, F), device=dev, dtype=x_rows.dtype)
    if y_rows is None:
        y_rows = torch.zeros((rows, d), device=dev, dtype=x_rows.dtype)
    _check(lib().capmoe_grouped_ffn_segments(_ptr(x_rows), _ptr(seg_begin), _ptr(seg_end), int(seg_begin.numel()),
                                             int(w_mod), int(d), int(F), _dt(x_rows), _ptr(w_gate), _ptr(w_up),
                                             _ptr(w_down), _ptr(h_ws), _ptr(y_rows), _i64(rows), _ptr(dev_status),
                                             _stream(stream)), "capmoe_grouped_ffn_segments")
    return y_rows


def ep_plan(slot_row, topk_idx, offsets, E: int, C_local: int, D: int = 1, token_group=None, stream=None):
    """-> (slot_row_ep [N,slots], bad [1]): rows of the [E][C_local] space of an expert-parallel rank."""
    N, slots = slot_row.shape
    k = topk_idx.shape[1]
    out = torch.empty_like(slot_row)
    bad = torch.zeros((1,), device=slot_row.device, dtype=torch.int32)
    _check(lib().capmoe_ep_plan(_ptr(slot_row), _ptr(topk_idx), _ptr(offsets), _i64(N), int(E), int(k), int(slots),
                                int(D), _ptr(token_group), _i64(C_local), _ptr(out), _ptr(bad), _stream(stream)),
           "capmoe_ep_plan")
    return out, bad


def ep_segments(counts, C_local: int, stream=None):
    """counts [S] int32 -> (seg_begin, seg_end) of the S fixed-place segments of C_local rows each."""
    S = counts.numel()
    b, e = torch.empty_like(counts), torch.empty_like(counts)
    _check(lib().capmoe_ep_segments(_ptr(counts), int(S), _i64(C_local), _ptr(b), _ptr(e), _stream(stream)),
           "capmoe_ep_segments")
    return b, e


def ep_dispatch(x, scores, topk_idx, slot_row_ep, peer_rows, R: int, rank: int, C_local: int, D: int = 0,
                token_group=None, out=None, stream=None):
    """Permute with every kept row stored into its owner's buffer (peer_rows: int64 tensor of R base
    addresses on the device).  -> dict(perm_token, perm_weight) of the local [E*C_local] row space."""
    N, d = x.shape
    E = scores.shape[1]
    k = topk_idx.shape[1]
    slots = slot_row_ep.shape[1]
    if out is None:
        out = dict(perm_token=torch.full((max(E * C_local, 1),), -1, device=x.device, dtype=torch.int32),
                   perm_weight=torch.zeros((max(E * C_local, 1),), device=x.device, dtype=torch.float32))
    _check(lib().capmoe_ep_dispatch(_ptr(x), _i64(N), int(d), int(E), int(k), int(slots), int(D), _dt(x), _ptr(scores),
                                    _ptr(topk_idx), _ptr(token_group), _ptr(slot_row_ep), _ptr(peer_rows), int(R),
                                    int(rank), _i64(C_local), _ptr(out["perm_token"]), _ptr(out["perm_weight"]),
                                    _stream(stream)), "capmoe_ep_dispatch")
    return out


def ep_combine(peer_rows, R: int, rank: int, E: int, C_local: int, slot_row_ep, perm_weight, d: int, dtype,
               y_shared=None, y=None, stream=None):
    """Combine with every kept row's result read from its owner's buffer (peer_rows as in ep_dispatch)."""
    N, slots = slot_row_ep.shape
    if y is None:
        y = torch.empty((N, d), device=slot_row_ep.device, dtype=dtype)
    _check(lib().capmoe_ep_combine(_ptr(peer_rows), int(R), int(rank), int(E), _i64(C_local), _ptr(slot_row_ep),
                                   _ptr(perm_weight), _i64(N), int(d), int(slots), _dt(dtype), _ptr(y_shared), _ptr(y),
                                   _stream(stream)), "capmoe_ep_combine")
    return y


EP_MODES = {"nodrop": 0, "token_drop": 1, "expanded_drop": 2}


def ep_rank_struct(**fields) -> _EPRank:
    """capmoe_ep_rank from tensors (device pointers taken), ints and None."""
    P = _EPRank()
    for name, v in fields.items():
        if isinstance(v, torch.Tensor):
            assert v.is_contiguous()
            v = v.data_ptr()
        elif v is None:
            v = 0
        setattr(P, name, v)
    return P


def ep_forward_dispatch(P: _EPRank, stream=None):
    _check(lib().capmoe_ep_forward_dispatch(ctypes.byref(P), _stream(stream)), "ep_forward_dispatch")


def ep_forward_experts(P: _EPRank, stream=None):
    _check(lib().capmoe_ep_forward_experts(ctypes.byref(P), _stream(stream)), "ep_forward_experts")


def ep_forward_combine(P: _EPRank, stream=None):
    _check(lib().capmoe_ep_forward_combine(ctypes.byref(P), _stream(stream)), "ep_forward_combine")


def combine(y_perm, slot_row, perm_weight, y_shared=None, y=None, stream=None):
    """-> y [N, d]"""
    N, slots = slot_row.shape
    d = y_perm.shape[1]
    if y is None:
        y = torch.empty((N, d), device=slot_row.device, dtype=y_perm.dtype)
    _check(lib().capmoe_combine(_ptr(y_perm), _ptr(slot_row), _ptr(perm_weight), _i64(N), int(d), int(slots),
                                _dt(y_perm), _ptr(y_shared), _ptr(y), _stream(stream)), "capmoe_combine")
    return y


def debug_check_indices(slot_row, topk_idx, offsets, E: int, A_max: int, D: int = 1, token_group=None, stream=None):
    """Runs the index check; returns the device status it produced (OK or EINDEX)."""
    N, slots = slot_row.shape
    k = topk_idx.shape[1]
    st = torch.zeros((1,), device=slot_row.device, dtype=torch.int32)
    _check(lib().capmoe_debug_check_indices(_ptr(slot_row), _ptr(topk_idx), _ptr(offsets), _i64(N), int(E), int(k),
                                            int(slots), int(D), _ptr(token_group), _i64(A_max), _ptr(st), _stream(stream)),
           "capmoe_debug_check_indices")
    return int(st.item())


FFN_VARIANTS = {"auto": 0, "pair": 1, "single": 2, "short": 3, "short_down": 4}


def debug_ffn_variant(name: str):
    """Forces one tensor-core FFN kernel for the whole process ("auto" restores the choice by shape)."""
    _check(lib().capmoe_debug_ffn_variant(FFN_VARIANTS[name]), "debug_ffn_variant")


def debug_read_probe(t: torch.Tensor, stream=None):
    """One plain pass of loads over the tensor's bytes (the one-shot read floor of that size)."""
    _check(lib().capmoe_debug_read_probe(_ptr(t), ctypes.c_size_t(t.numel() * t.element_size()), ctypes.c_void_p(0),
                                         _stream(stream)), "capmoe_debug_read_probe")


def debug_wait_probe(limit_cycles: int = 50_000_000, stream=None) -> int:
    """Runs the bounded-wait self-test; returns the device status it produced (ETIMEOUT expected)."""
    st = torch.zeros((1,), device="cuda", dtype=torch.int32)
    _check(lib().capmoe_debug_wait_probe(_i64(limit_cycles), _ptr(st), _stream(stream)), "capmoe_debug_wait_probe")
    torch.cuda.synchronize()
    return int(st.item())


# ----------------------------------------------------------------------------- whole layer
class MoELayer:
    """Device buffers for one layer plus the C struct that names them.  `forward()` enqueues
    capmoe_layer_forward; `forward_host()` enqueues the host-buffer variant."""

    def __init__(self, x, w_router, bias, w_gate, w_up, w_down, k: int, D: int, mode: str, gamma: float = 1.0,
                 straggler: bool = False, shared=None, round_mode: str = "ceil", C: Optional[int] = None,
                 metric: str = "score", seed: int = 0, token_class=None, topk_first: bool = False,
                 max_experts: int = 0, debug_checks: bool = False):
        """Variants of the drop (token_drop / expanded_drop modes): `metric` ranks candidates by Score, Order,
        Reverse Order or Random; `token_class` (uint8 [N], 1 = protected modality) drops the other modality
        first; `topk_first` lets the expansion only fill spare capacity; `max_experts` > 0 is 'w/ max'."""
        dev = x.device
        N, d = x.shape
        E, F, _ = w_gate.shape
        self.N, self.d, self.E, self.k, self.F, self.D = N, d, E, k, F, D
        self.mode = mode
        m = E // D
        expanded = mode in ("expanded_drop", "device_expanded_drop")
        device_level = mode.startswith("device_")
        if C is None:
            if mode == "nodrop":
                C = N
            elif device_level:
                C = device_capacity(N, E, k, D, gamma, round_mode)
            else:
                C = capacity(N, E, k, gamma, round_mode)
        self.C = C
        self.slots = k + m if expanded else k
        A_max = device_max_rows(N, E, k, D, C, expanded) if device_level else max_rows(N, E, k, D, C, expanded)
        self.A_max = A_max
        W = (E + 63) // 64
        f32 = dict(device=dev, dtype=torch.float32)
        i32 = dict(device=dev, dtype=torch.int32)
        act = dict(device=dev, dtype=x.dtype)
        t = self.t = {}
        t["x"], t["w_router"], t["bias"] = x, w_router, bias
        t["w_gate"], t["w_up"], t["w_down"] = w_gate, w_up, w_down
        t["logits"] = torch.empty((N, E), **f32)
        t["scores"] = torch.empty((N, E), **f32)
        t["topk_idx"] = torch.empty((N, k), **i32)
        t["topk_score"] = torch.empty((N, k), **f32)
        t["load"] = torch.empty((E,), **i32)
        t["keep_mask"] = torch.empty((N, W), device=dev, dtype=torch.int64)
        t["cand"] = torch.zeros((E,), **i32)
        t["kept"] = torch.empty((E,), **i32)
        t["expert_offsets"] = torch.empty((E + 1,), **i32)
        t["slot_row"] = torch.empty((N, self.slots), **i32)
        t["x_perm"] = torch.zeros((max(A_max, 1), d), **act)
        t["perm_token"] = torch.full((max(A_max, 1),), -1, **i32)
        t["perm_weight"] = torch.zeros((max(A_max, 1),), **f32)
        t["h_ws"] = torch.empty((max(A_max, 1), F), **act)
        t["y_perm"] = torch.zeros((max(A_max, 1), d), **act)
        t["y"] = torch.empty((N, d), **act)
        t["drop_ws"] = torch.empty((drop_workspace_bytes(N, E, k, D, expanded),), device=dev, dtype=torch.uint8)
        t["dev_status"] = torch.zeros((FFN_STATUS_WORDS,), **i32)
        F_shared = 0
        if shared is not None:
            t["ws_gate"], t["ws_up"], t["ws_down"] = shared
            F_shared = shared[0].shape[-2]
            t["hs_ws"] = torch.empty((N, F_shared), **act)
            t["y_shared"] = torch.empty((N, d), **act)
            t["one_segment"] = torch.tensor([0, N], **i32)
        keyed = metric != "score" or token_class is not None or (topk_first and mode == "expanded_drop")
        if keyed or max_experts > 0:
            if mode not in ("token_drop", "expanded_drop"):
                raise ValueError("drop variants apply to the token_drop and expanded_drop modes")
        if keyed:
            t["drop_keys"] = torch.empty((N, E if expanded else k), **f32)
        if token_class is not None:
            assert token_class.dtype == torch.uint8 and token_class.shape == (N,)
            t["token_class"] = token_class
        if max_experts > 0:
            t["bad"] = torch.zeros((1,), **i32)
        L = self.c = _Layer()
        L.metric, L.metric_seed, L.topk_first, L.max_experts = METRICS[metric], seed, int(bool(topk_first)), max_experts
        L.debug_checks = int(bool(debug_checks))
        L.N, L.d, L.E, L.k, L.F, L.D, L.dtype = N, d, E, k, F, D, _dt(x)
        L.mode, L.C, L.straggler = MODES[mode], C, int(bool(straggler))
        L.F_shared, L.A_max = F_shared, A_max
        L.drop_ws_bytes = t["drop_ws"].numel()
        for name, _typ in _Layer._fields_:
            if name in t:
                assert t[name].is_contiguous()
                setattr(L, name, t[name].data_ptr())

    def set_stage_events(self, events):
        """events: None, or N_STAGE_EVENTS recorded torch.cuda.Event(enable_timing=True) objects."""
        if events is None:
            self.c.stage_events = ctypes.POINTER(ctypes.c_void_p)()
            self._ev = None
            return
        assert len(events) == N_STAGE_EVENTS
        arr = (ctypes.c_void_p * N_STAGE_EVENTS)(*[ctypes.c_void_p(e.cuda_event) for e in events])
        self._ev = (arr, events)
        self.c.stage_events = ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p))

    def forward(self, stream=None):
        _check(lib().capmoe_layer_forward(ctypes.byref(self.c), _stream(stream)), "capmoe_layer_forward")
        return self.t["y"]

    def capture_graph(self):
        """Records one forward into a CUDA graph (stage events off), so that `replay()` re-issues the
        whole layer with one launch call.  Run `forward()` at least once before: kernels are loaded on
        their first launch, which a capture does not allow.  Buffers and shapes are frozen."""
        self.set_stage_events(None)
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream(device=self.t["x"].device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(graph, stream=side):
            self.forward()
        self._graph = graph
        return graph

    def replay(self):
        self._graph.replay()
        return self.t["y"]

    def forward_host(self, x_host: torch.Tensor, y_host: torch.Tensor, stream=None):
        assert x_host.is_pinned() and y_host.is_pinned() and x_host.is_contiguous() and y_host.is_contiguous()
        _check(lib().capmoe_layer_forward_host(ctypes.byref(self.c), ctypes.c_void_p(x_host.data_ptr()),
                                               ctypes.c_void_p(y_host.data_ptr()), _stream(stream)),
               "capmoe_layer_forward_host")
        return y_host

    def check_device_status(self):
        s = int(self.t["dev_status"][0].item())
        if s != OK:
            raise CapmoeError(s, "device status")
