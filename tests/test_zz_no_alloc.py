"""capmoe_token_drop_static: Token Drop for callers that cannot hand the library any scratch
memory (no cudaMalloc available to them, e.g. a runtime with a memory pool fixed at start-up).
The entry point keeps its scratch in an array inside the library, so consecutive calls reuse
the same memory; this test makes two calls in a row through the C ABI and compares each with
the ordinary capmoe_token_drop, bit for bit.  It lives in a file that pytest collects last."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2503_05066_b200 import synth

pytestmark = pytest.mark.gpu


def _routing(cm, N, E, k, seed, quantum):
    bias = (-np.log(np.arange(E) + 1.0)).astype(np.float32)
    lg = synth.synthetic_logits(N, E, seed, bias=bias, quantum=quantum)
    return cm.route(None, None, None, k, logits_in=torch.from_numpy(lg).cuda())


def _call_static(cm, r, E, C):
    """Straight through the C ABI: plain pointers and sizes."""
    L = cm.lib()
    idx, val = r["topk_idx"], r["topk_score"]
    N, k = idx.shape
    W = (E + 63) // 64
    out = dict(keep_mask=torch.full((N, W), -1, device="cuda", dtype=torch.int64),
               kept=torch.full((E,), -7, device="cuda", dtype=torch.int32),
               offsets=torch.full((E + 1,), -7, device="cuda", dtype=torch.int32),
               slot_row=torch.full((N, k), -7, device="cuda", dtype=torch.int32))
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = L.capmoe_token_drop_static(p(val), p(idx), ctypes.c_int64(N), E, k, ctypes.c_int64(C),
                                    p(out["keep_mask"]), p(out["kept"]), p(out["offsets"]), p(out["slot_row"]),
                                    ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == cm.OK, cm.lib().capmoe_status_str(rc)
    return out


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    from paper_2503_05066_b200 import capmoe as cm
    # first a large, tie-heavy call, then a smaller one that would see stale scratch if anything
    # that must start from zero were not cleared
    cases = [(6000, 64, 8, 1.0, 0.5, 11), (1500, 8, 2, 1.0, 0.0, 12)]
    for N, E, k, gamma, q, seed in cases:
        r = _routing(cm, N, E, k, seed, q)
        C = cm.capacity(N, E, k, gamma)
        got = _call_static(cm, r, E, C)
        ref = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
        torch.cuda.synchronize()
        for key in ("keep_mask", "kept", "offsets", "slot_row"):
            assert torch.equal(got[key], ref[key]), (N, E, key)
        assert int(ref["offsets"][-1]) < N * k          # something was dropped: the select really ran


def test_static_scratch_rejects_oversized_calls_before_launching():
    from paper_2503_05066_b200 import capmoe as cm
    L = cm.lib()
    fake = ctypes.c_void_p(256)                          # never dereferenced: the call is refused on the host
    N = cm.STATIC_DROP_MAX_PAIRS // 2 + 1
    rc = L.capmoe_token_drop_static(fake, fake, ctypes.c_int64(N), 8, 2, ctypes.c_int64(1), fake, fake, fake,
                                    fake, ctypes.c_void_p(0))
    assert rc == cm.EWORKSPACE
    with pytest.raises(cm.CapmoeError, match="built-in scratch"):
        z = torch.zeros((N, 2), device="cuda")
        cm.token_drop_static(z, z.int(), 8, 1)
