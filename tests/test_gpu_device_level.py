"""Device-level capacity on the GPU against the CPU checker: keep masks, counts, offsets and
rows bit for bit; layer output within the bf16 / fp32 bars."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.test_gpu_parity import TOL, bias_for, cached_inputs, cm, dev, host_mask  # noqa: F401
from tests.util import rel_err, to_np

pytestmark = pytest.mark.gpu

CASES = [
    # N, E, k, D, gamma, quantum
    (512, 8, 2, 2, 1.0, 0.0),
    (4096, 64, 8, 8, 1.0, 0.0),
    (4096, 64, 8, 8, 1.5, 0.0),
    (3000, 60, 4, 4, 0.5, 0.0),       # 15 experts per device: three packed rank words
    (3000, 60, 4, 4, 2.0, 0.0),
    (2049, 8, 2, 2, 1.25, 0.0),
    (1023, 16, 4, 1, 1.0, 0.0),       # one device holds everything (m = 16)
    (640, 16, 2, 16, 1.0, 0.0),       # one expert per device: the expert-level rule
    (700, 8, 8, 2, 1.0, 0.0),         # k = E
    (5000, 8, 2, 2, 1.0, 0.5),        # many exact ties
    (2500, 64, 8, 2, 1.0, 1.0),       # 32 experts per device, heavy ties
    (100, 8, 2, 2, 0.0, 0.0),
    (100, 8, 2, 2, float("inf"), 0.0),
    (1, 8, 2, 2, 1.0, 0.0),
    (9000, 8, 2, 4, 1.0, 0.0),
]


def _routing(cm, N, E, k, q, seed=13):
    lg = synth.synthetic_logits(N, E, seed, bias=bias_for(E), quantum=q)
    r = cm.route(None, None, None, k, logits_in=dev(lg))
    return r, r["scores"].cpu().numpy(), r["topk_idx"].cpu().numpy()


@pytest.mark.parametrize("expanded", [False, True])
@pytest.mark.parametrize("N,E,k,D,gamma,q", CASES)
def test_device_drop_bit_exact(cm, N, E, k, D, gamma, q, expanded):
    r, scores, idx = _routing(cm, N, E, k, q)
    C_dev = cm.device_capacity(N, E, k, D, gamma)
    assert C_dev == oracle.device_capacity(N, E, k, D, gamma)
    got = cm.device_drop(r["scores"], r["topk_idx"], C_dev, D, expanded)
    ref = oracle.device_drop(scores, idx, C_dev, D, expanded)
    assert np.array_equal(got["cand"].cpu().numpy(), ref["cand"])
    assert np.array_equal(got["kept"].cpu().numpy(), ref["kept"])
    assert np.array_equal(got["offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    assert np.array_equal(got["slot_row"].cpu().numpy(), ref["slot_row"])


def test_device_drop_explicit_groups_and_determinism(cm):
    N, E, k, D = 3000, 16, 2, 4
    r, scores, idx = _routing(cm, N, E, k, 0.5)
    tg = (synth.token_permutation(N, 5) % D).astype(np.int32)
    C_dev = cm.device_capacity(N, E, k, D, 1.0)
    ref = oracle.device_drop(scores, idx, C_dev, D, True, token_group=tg)
    first = None
    for _ in range(4):
        got = cm.device_drop(r["scores"], r["topk_idx"], C_dev, D, True, token_group=dev(tg))
        for key in ("cand", "kept", "offsets", "slot_row"):
            assert np.array_equal(got[key].cpu().numpy(), ref[key]), key
        if first is None:
            first = got
        else:
            assert all(torch.equal(first[key], got[key]) for key in first)


def _device_layer(cm, cfg, expanded, gamma, straggler=False, sample=None):
    inp = cached_inputs(cfg)
    mode = "device_expanded_drop" if expanded else "device_token_drop"
    layer = cm.MoELayer(dev(inp.x), dev(inp.w_router), dev(inp.bias), dev(inp.w_gate), dev(inp.w_up), dev(inp.w_down),
                        cfg.k, cfg.D, mode, gamma=gamma, straggler=straggler)
    y = layer.forward()
    torch.cuda.synchronize()
    layer.check_device_status()
    t = layer.t
    scores = oracle.softmax(t["logits"].cpu().numpy())
    idx, _, _ = oracle.topk(scores, cfg.k)
    C_dev = oracle.device_capacity(cfg.N, cfg.E, cfg.k, cfg.D, gamma)
    ref = oracle.device_drop(scores, idx, C_dev, cfg.D, expanded)
    assert np.array_equal(host_mask(t["keep_mask"]), ref["keep_mask"])
    assert np.array_equal(t["expert_offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(t["slot_row"].cpu().numpy(), ref["slot_row"])
    toks = (np.arange(cfg.N, dtype=np.int32) if sample is None else
            np.unique(np.concatenate([[0, cfg.N - 1], np.random.default_rng(1).integers(0, cfg.N, sample)])).astype(np.int32))
    yref = oracle.layer_tokens(to_np(inp.x), toks, scores, idx, ref["slot_row"], cfg.D if expanded else 0,
                               to_np(inp.w_gate), to_np(inp.w_up), to_np(inp.w_down), cfg.dtype)
    err = rel_err(y.double().cpu().numpy()[toks], yref)
    assert err <= TOL[cfg.dtype], err
    return layer


@pytest.mark.parametrize("expanded", [False, True])
def test_device_level_layer_tiny_fp32(cm, expanded):
    _device_layer(cm, synth.CONFIGS["tiny_f32"], expanded, 1.0)


@pytest.mark.parametrize("expanded", [False, True])
def test_device_level_layer_bf16_small(cm, expanded):
    _device_layer(cm, synth.CONFIGS["olmoe"].with_(N=600, d=256, F=384, E=16, k=4, D=4), expanded, 1.0)


def test_device_level_layer_mixtral_shape_with_straggler_partition(cm):
    _device_layer(cm, synth.CONFIGS["mixtral"], True, 1.0, straggler=True, sample=12)


def test_device_level_layer_olmoe_shape(cm):
    _device_layer(cm, synth.CONFIGS["olmoe"], True, 1.0, sample=32)
