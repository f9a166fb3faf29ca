"""CPU-side checks of the C ABI: the library loads, exports every symbol the header declares,
host-only helpers agree with hand values, and argument validation rejects bad calls before
anything touches a GPU."""
import ctypes
import os
import re

import pytest

from paper_2503_05066_b200 import build as capmoe_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="module")
def cm():
    capmoe_build.build()
    from paper_2503_05066_b200 import capmoe
    capmoe.lib()
    return capmoe


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "capmoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(capmoe_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(cm):
    names = _declared_symbols()
    assert len(names) >= 15
    L = ctypes.CDLL(cm.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert set(cm.EXPORTS) == set(names)


def test_capacity_matches_hand_values(cm):
    rows = [l.split() for l in open(os.path.join(GOLD, "capacity.txt")) if l.strip() and l[0] != "#"]
    for N, E, k, g, cc, cf in rows:
        assert cm.capacity(int(N), int(E), int(k), float(g), "ceil") == int(cc)
        assert cm.capacity(int(N), int(E), int(k), float(g), "floor") == int(cf)
    assert cm.capacity(1000, 8, 2, float("inf")) == 1000


def test_max_rows_and_workspace(cm):
    assert cm.max_rows(4096, 64, 8, 8, 512, False) == 32768
    assert cm.max_rows(4096, 64, 8, 8, 768, True) == 49152
    assert cm.max_rows(4096, 64, 8, 8, 4096, False) == 32768
    assert cm.max_rows(4096, 64, 8, 8, 4096, True) == 65536
    assert cm.max_rows(100, 8, 2, 2, 0, False) == 0
    assert cm.drop_workspace_bytes(1024, 8, 2, 2, False) >= 3 * 4 * 2048
    assert cm.drop_workspace_bytes(1024, 8, 2, 2, True) >= 3 * 4 * 1024 * 6
    with pytest.raises(cm.CapmoeError):
        cm.drop_workspace_bytes(1024, 8, 2, 3, True)


def test_status_strings(cm):
    L = cm.lib()
    seen = {L.capmoe_status_str(i).decode() for i in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert L.capmoe_status_str(99).decode() == "unknown status"


def test_validation_happens_before_any_launch(cm):
    """Bad arguments are refused on the host; none of these calls needs (or touches) a GPU."""
    L = cm.lib()
    z = ctypes.c_void_p(0)
    one = ctypes.c_void_p(16)       # non-null, aligned, never dereferenced
    i64 = ctypes.c_int64
    # k > E
    assert L.capmoe_route(one, one, z, z, i64(4), 8, 4, 5, 0, one, one, one, one, one, z) == cm.EINVAL
    # unknown dtype
    assert L.capmoe_route(one, one, z, z, i64(4), 8, 4, 2, 7, one, one, one, one, one, z) == cm.EUNSUPPORTED
    # null outputs
    assert L.capmoe_route(one, one, z, z, i64(4), 8, 4, 2, 0, one, z, one, one, one, z) == cm.EINVAL
    # C out of range, negative N
    assert L.capmoe_token_drop(one, one, i64(4), 4, 2, i64(5), one, one, one, one, one, ctypes.c_size_t(1 << 20), z) == cm.EINVAL
    assert L.capmoe_token_drop(one, one, i64(-1), 4, 2, i64(0), one, one, one, one, one, ctypes.c_size_t(1 << 20), z) == cm.EINVAL
    # E % D != 0
    assert L.capmoe_expanded_drop(one, one, i64(4), 6, 2, i64(2), 4, z, one, one, one, one, one, one,
                                  ctypes.c_size_t(1 << 20), z) == cm.EINVAL
    # E beyond the supported range
    assert L.capmoe_token_drop(one, one, i64(4), 512, 2, i64(2), one, one, one, one, one, ctypes.c_size_t(1 << 20), z) == cm.EUNSUPPORTED
    # permute: row size not a multiple of 16 bytes; slots inconsistent with D
    assert L.capmoe_permute(one, i64(4), 6, 4, 2, 2, 0, 1, one, one, z, one, one, one, one, z) == cm.EUNSUPPORTED
    assert L.capmoe_permute(one, i64(4), 8, 4, 2, 3, 0, 1, one, one, z, one, one, one, one, z) == cm.EINVAL
    # misaligned pointer
    odd = ctypes.c_void_p(24 + 4)
    assert L.capmoe_permute(odd, i64(4), 8, 4, 2, 2, 0, 1, one, one, z, one, one, one, one, z) == cm.EINVAL
    assert L.capmoe_grouped_ffn(odd, one, 4, 64, 64, 1, one, one, one, one, one, i64(8), 0, z, z) == cm.EINVAL
    # straggler groups must divide E
    assert L.capmoe_grouped_ffn(one, one, 6, 64, 64, 1, one, one, one, one, one, i64(8), 4, z, z) == cm.EINVAL
    assert L.capmoe_combine(one, one, one, i64(4), 6, 2, 1, z, one, z) == cm.EUNSUPPORTED
    assert L.capmoe_layer_forward(z, z) == cm.EINVAL


def test_missing_library_fails_loudly(cm, monkeypatch):
    monkeypatch.setattr(cm, "_lib", None)
    monkeypatch.setattr(cm, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        cm.capacity(8, 4, 2, 1.0)


def _fake_layer(cm, **over):
    """A capmoe_layer whose every field passes validation (pointers are aligned dummies that are
    never dereferenced on the host); `over` then breaks one field."""
    L = cm._Layer()
    L.N, L.d, L.E, L.k, L.F, L.D, L.dtype = 64, 64, 8, 2, 64, 2, cm.BF16
    L.mode, L.C, L.straggler = 2, 16, 0
    L.A_max = cm.max_rows(64, 8, 2, 2, 16, True)
    L.drop_ws_bytes = cm.drop_workspace_bytes(64, 8, 2, 2, True)
    for name, typ in cm._Layer._fields_:
        if typ is ctypes.c_void_p and name not in ("ws_gate", "ws_up", "ws_down", "hs_ws", "y_shared", "one_segment",
                                                   "token_class", "drop_keys", "bad"):
            setattr(L, name, 4096)
    for key, v in over.items():
        setattr(L, key, v)
    return L


def test_layer_forward_checks_every_field_before_it_enqueues_anything(cm):
    """Each broken field is reported by the host-side checks: the call returns its status without
    an event record, memset or launch (the launch counter does not move, and on a machine without
    a GPU no CUDA call is reached, which would show as CAPMOE_ECUDA)."""
    lib = cm.lib()
    cases = [
        (dict(mode=5), cm.EINVAL), (dict(k=9), cm.EINVAL), (dict(N=-1), cm.EINVAL), (dict(dtype=3), cm.EUNSUPPORTED),
        (dict(E=512, k=2), cm.EUNSUPPORTED),
        (dict(D=3), cm.EINVAL),                                   # E % D != 0 (Expanded Drop needs D)
        (dict(mode=3, D=3), cm.EINVAL), (dict(mode=1, straggler=1, D=3), cm.EINVAL),
        (dict(C=65), cm.EINVAL), (dict(C=-1), cm.EINVAL),
        (dict(mode=4, C=64 * 4 + 1), cm.EINVAL),                  # device capacity beyond N * E/D
        (dict(metric=7), cm.EINVAL),
        (dict(metric=3), cm.EINVAL),                              # keyed drop without key scratch
        (dict(topk_first=1), cm.EINVAL), (dict(token_class=4096), cm.EINVAL),
        (dict(max_experts=2), cm.EINVAL),                         # "w/ max" without the bad flag
        (dict(mode=3, metric=1, drop_keys=4096), cm.EUNSUPPORTED),
        (dict(mode=4, max_experts=1, bad=4096), cm.EUNSUPPORTED),
        (dict(load=0), cm.EINVAL), (dict(logits=0), cm.EINVAL), (dict(cand=0), cm.EINVAL),
        (dict(kept=0), cm.EINVAL), (dict(expert_offsets=0), cm.EINVAL),
        (dict(x=0), cm.EINVAL), (dict(keep_mask=0), cm.EINVAL), (dict(slot_row=0), cm.EINVAL),
        (dict(y=0), cm.EINVAL), (dict(drop_ws=0), cm.EINVAL), (dict(x=4100), cm.EINVAL),
        (dict(x_perm=0), cm.EINVAL), (dict(h_ws=0), cm.EINVAL), (dict(w_down=0), cm.EINVAL),
        (dict(y_perm=4104), cm.EINVAL),
        (dict(F_shared=64), cm.EINVAL),                           # shared expert without its buffers
        (dict(F_shared=-1), cm.EINVAL),
        (dict(d=60), cm.EUNSUPPORTED),                            # rows not a multiple of 16 bytes
        (dict(dtype=cm.F32, straggler=1), cm.EUNSUPPORTED),       # SM partition exists only on the tensor-core path
        (dict(A_max=16 * 8 - 1), cm.EWORKSPACE),                  # below min(E*C, N*(k+m))
        (dict(mode=0, A_max=64 * 2 - 1), cm.EWORKSPACE),
        (dict(mode=3, C=40, A_max=2 * 40 - 1), cm.EWORKSPACE),
        (dict(drop_ws_bytes=64), cm.EWORKSPACE),
    ]
    before = cm.launch_count()
    for over, want in cases:
        L = _fake_layer(cm, **over)
        got = lib.capmoe_layer_forward(ctypes.byref(L), ctypes.c_void_p(0))
        assert got == want, (over, got, want)
    assert cm.launch_count() == before


def test_device_max_rows(cm):
    assert cm.device_max_rows(4096, 64, 8, 8, 4096, False) == 32768
    assert cm.device_max_rows(4096, 64, 8, 8, 100, False) == 800
    assert cm.device_max_rows(4096, 64, 8, 8, 10 ** 9, True) == 4096 * 16
    with pytest.raises(cm.CapmoeError):
        cm.device_max_rows(4096, 64, 8, 7, 10, False)


def _fake_ep_rank(cm, **over):
    """A capmoe_ep_rank whose every field passes validation (dummy pointers, never dereferenced)."""
    P = cm._EPRank()
    P.N, P.d, P.E, P.k, P.F, P.dtype = 64, 64, 8, 2, 64, cm.BF16
    P.R, P.rank, P.mode, P.C_local, P.C = 4, 1, 2, 16, 20
    P.drop_ws_bytes = cm.drop_workspace_bytes(64, 8, 2, 4, True)
    for name, typ in cm._EPRank._fields_:
        if typ is ctypes.c_void_p:
            setattr(P, name, 4096)
    for key, v in over.items():
        setattr(P, key, v)
    return P


def test_ep_rank_phases_check_every_field_before_they_enqueue_anything(cm):
    lib = cm.lib()
    cases = [
        (dict(mode=3), cm.EINVAL), (dict(R=3), cm.EINVAL), (dict(rank=4), cm.EINVAL), (dict(rank=-1), cm.EINVAL),
        (dict(C=15), cm.EINVAL),                                  # row stride below the rank's own capacity
        (dict(C_local=65, C=65), cm.EINVAL), (dict(mode=0), cm.EINVAL),          # no drop needs C_local = N
        (dict(k=9), cm.EINVAL), (dict(dtype=3), cm.EUNSUPPORTED), (dict(E=512, R=4), cm.EUNSUPPORTED),
        (dict(d=4, dtype=cm.BF16), cm.EUNSUPPORTED),              # rows of 8 bytes: not a multiple of 16
        (dict(token_group=0), cm.EINVAL), (dict(cand=0), cm.EINVAL), (dict(bad=0), cm.EINVAL),
        (dict(cnt_recv=0), cm.EINVAL), (dict(seg_end=0), cm.EINVAL), (dict(slot_row_ep=0), cm.EINVAL),
        (dict(x_recv=0), cm.EINVAL), (dict(w_up=0), cm.EINVAL), (dict(perm_weight=0), cm.EINVAL),
        (dict(peer_x=0, x_send=0), cm.EINVAL), (dict(peer_y=0, y_ret=0), cm.EINVAL),
        (dict(drop_ws_bytes=8), cm.EWORKSPACE),
    ]
    before = cm.launch_count()
    for over, want in cases:
        P = _fake_ep_rank(cm, **over)
        for fn in (lib.capmoe_ep_forward_dispatch, lib.capmoe_ep_forward_experts, lib.capmoe_ep_forward_combine):
            got = fn(ctypes.byref(P), ctypes.c_void_p(0))
            assert got == want, (over, fn.__name__, got, want)
    assert lib.capmoe_ep_forward_dispatch(None, ctypes.c_void_p(0)) == cm.EINVAL
    assert cm.launch_count() == before
