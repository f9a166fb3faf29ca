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
