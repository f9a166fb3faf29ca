"""Drop metrics on the GPU: keys and the resulting drops against the CPU checker, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.test_gpu_parity import bias_for, cm, dev, host_mask  # noqa: F401

pytestmark = pytest.mark.gpu


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("metric", ["score", "order", "reverse_order", "random"])
@pytest.mark.parametrize("N,E,k,D,q", [(700, 8, 2, 2, 0.0), (3000, 60, 4, 4, 0.5), (20000, 16, 4, 4, 0.0)])
def test_metric_keys_and_drops_match_oracle(cm, metric, N, E, k, D, q):
    lg = synth.synthetic_logits(N, E, 21, bias=bias_for(E), quantum=q)
    r = cm.route(None, None, None, k, logits_in=dev(lg))
    scores, idx = r["scores"].cpu().numpy(), r["topk_idx"].cpu().numpy()
    seed = 0xC0FFEE
    # dense [N,E] keys and sparse [N,k] keys
    kd = cm.drop_keys(metric, seed, r["scores"], None, E)
    ks = cm.drop_keys(metric, seed, r["topk_score"], r["topk_idx"], E)
    ref_d = oracle.drop_keys(metric, seed, scores, None, E)
    assert np.array_equal(_bits(kd), ref_d)
    assert np.array_equal(_bits(ks), np.take_along_axis(ref_d, idx, 1))
    C = cm.capacity(N, E, k, 1.0)
    got = cm.token_drop(ks, r["topk_idx"], E, C)
    ref = oracle.drop_keyed(ref_d, idx, C)
    for key, rk in (("kept", "kept"), ("offsets", "offsets"), ("slot_row", "slot_row")):
        assert np.array_equal(got[key].cpu().numpy(), ref[rk]), (metric, key)
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    got = cm.expanded_drop(kd, r["topk_idx"], C, D)
    ref = oracle.drop_keyed(ref_d, idx, C, D, True)
    for key in ("cand", "kept", "offsets", "slot_row"):
        assert np.array_equal(got[key].cpu().numpy(), ref[key]), (metric, key)
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    # the gate weights of the kept rows are still the real scores
    A = int(ref["offsets"][-1])
    x = torch.zeros((N, 8), device="cuda")
    p = cm.permute(x, r["scores"], r["topk_idx"], got["slot_row"], max(A, 1), D)
    pref = oracle.permute(None, scores, idx, ref["slot_row"], A, D, "f32")
    assert np.array_equal(p["perm_weight"].cpu().numpy()[:A].view(np.uint32), pref["perm_weight"].view(np.uint32))
