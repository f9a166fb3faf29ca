"""capmoe_token_drop_static: Token Drop for callers that cannot hand the library any scratch
memory (no cudaMalloc available to them, e.g. a runtime with a memory pool fixed at start-up).
The entry point keeps its scratch in an array inside the library, so consecutive calls reuse
the same memory; this test makes two calls in a row through the C ABI and compares each with
the ordinary capmoe_token_drop and with the CPU checker, bit for bit, and checks that the call
left the amount of allocated device memory unchanged.  It lives in a file that pytest collects last."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth

pytestmark = pytest.mark.gpu


def _routing(cm, N, E, k, seed, quantum):
    bias = (-np.log(np.arange(E) + 1.0)).astype(np.float32)
    lg = synth.synthetic_logits(N, E, seed, bias=bias, quantum=quantum)
    return cm.route(None, None, None, k, logits_in=torch.from_numpy(lg).cuda())


def _outputs(N, E, k):
    W = (E + 63) // 64
    return dict(keep_mask=torch.full((N, W), -1, device="cuda", dtype=torch.int64),
                kept=torch.full((E,), -7, device="cuda", dtype=torch.int32),
                offsets=torch.full((E + 1,), -7, device="cuda", dtype=torch.int32),
                slot_row=torch.full((N, k), -7, device="cuda", dtype=torch.int32))


def _raw_call(cm, r, E, C, out):
    """Straight through the C ABI: plain pointers and sizes."""
    idx, val = r["topk_idx"], r["topk_score"]
    N, k = idx.shape
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = cm.lib().capmoe_token_drop_static(p(val), p(idx), ctypes.c_int64(N), E, k, ctypes.c_int64(C),
                                           p(out["keep_mask"]), p(out["kept"]), p(out["offsets"]),
                                           p(out["slot_row"]),
                                           ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == cm.OK, cm.lib().capmoe_status_str(rc)


_warm = False


def _call_static(cm, r, E, C):
    global _warm
    if not _warm:
        # The first call on a device looks up the array's address, and the driver loads each kernel
        # on its first launch (which takes device memory of its own); the memory check below is
        # about the calls after that.
        _warm = True
        w = _routing(cm, 64, 8, 2, 1, 0.0)
        _raw_call(cm, w, 8, 4, _outputs(64, 8, 2))
        torch.cuda.synchronize()
    N, k = r["topk_idx"].shape
    out = _outputs(N, E, k)
    torch.cuda.synchronize()
    held = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0])
    _raw_call(cm, r, E, C, out)
    torch.cuda.synchronize()
    # nothing was allocated, by torch or behind its back (free device memory as the driver reports it)
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), torch.cuda.mem_get_info()[0]) == held
    return out


def _check_against_both(cm, r, E, C, got):
    ref = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
    torch.cuda.synchronize()
    for key in ("keep_mask", "kept", "offsets", "slot_row"):
        assert torch.equal(got[key], ref[key]), key
    o = oracle.token_drop(r["scores"].cpu().numpy(), r["topk_idx"].cpu().numpy(), C)
    assert np.array_equal(got["keep_mask"].cpu().numpy().view(np.uint64), o["keep_mask"])
    assert np.array_equal(got["kept"].cpu().numpy(), o["kept"])
    assert np.array_equal(got["offsets"].cpu().numpy(), o["offsets"])
    assert np.array_equal(got["slot_row"].cpu().numpy(), o["slot_row"])
    return ref


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    from paper_2503_05066_b200 import capmoe as cm
    # first a large, tie-heavy call, then a smaller one that would see stale scratch if anything
    # that must start from zero were not cleared
    cases = [(6000, 64, 8, 1.0, 0.5, 11), (1500, 8, 2, 1.0, 0.0, 12)]
    for N, E, k, gamma, q, seed in cases:
        r = _routing(cm, N, E, k, seed, q)
        C = cm.capacity(N, E, k, gamma)
        got = _call_static(cm, r, E, C)
        ref = _check_against_both(cm, r, E, C, got)
        assert int(ref["offsets"][-1]) < N * k          # something was dropped: the select really ran


def test_static_scratch_filled_to_its_last_word_then_reused():
    """N*k equal to the limit: the three candidate lists end exactly at the end of the built-in
    array, and at this batch size the entry point runs the one-CTA-per-expert select that the
    workspace entry point no longer uses for large batches.  A small call follows on the same array."""
    from paper_2503_05066_b200 import capmoe as cm
    E, k = 64, 8
    N = cm.STATIC_DROP_MAX_PAIRS // k                    # 131072 tokens
    for n, e, kk, q, seed in [(N, E, k, 0.5, 21), (700, 16, 4, 0.0, 22)]:
        r = _routing(cm, n, e, kk, seed, q)
        C = cm.capacity(n, e, kk, 1.0)
        got = _call_static(cm, r, e, C)
        ref = _check_against_both(cm, r, e, C, got)
        assert int(ref["offsets"][-1]) < n * kk


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
