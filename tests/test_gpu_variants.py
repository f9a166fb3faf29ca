"""Variants of the drop on the GPU against the CPU checker, bit for bit: priority classes
(modality-first dropping, Expanded Drop as substitution only), the 'w/ max' limit with the rebuilt
permutation, global top-(k+m) expansion, and a layer assembled from the stage calls."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.test_gpu_parity import TOL, bias_for, cm, dev, host_mask  # noqa: F401
from tests.util import as_f64, rel_err, to_np

pytestmark = pytest.mark.gpu

CASES = [(700, 8, 2, 2, 0.0, 1.0), (3000, 60, 4, 4, 0.5, 1.0), (2500, 64, 8, 8, 0.0, 1.5),
         (20000, 16, 4, 4, 0.25, 1.0),        # token-parallel select
         (900, 130, 6, 10, 0.0, 1.0),         # three mask words
         (257, 12, 3, 12, 1.0, 0.5)]


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def _route(cm, N, E, k, q, seed=33):
    lg = synth.synthetic_logits(N, E, seed, bias=bias_for(E), quantum=q)
    r = cm.route(None, None, None, k, logits_in=dev(lg))
    return r, r["scores"].cpu().numpy(), r["topk_idx"].cpu().numpy()


def _same_drop(got, ref, keys=("cand", "kept", "offsets", "slot_row")):
    for key in keys:
        assert np.array_equal(got[key].cpu().numpy(), ref[key]), key
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])


@pytest.mark.parametrize("N,E,k,D,q,gamma", CASES)
def test_modality_first_token_drop(cm, N, E, k, D, q, gamma):
    r, scores, idx = _route(cm, N, E, k, q)
    is_image = (np.arange(N) * 7 % 10) < 6
    cls = (~is_image).astype(np.uint8)                       # Image First: text tokens are protected
    C = cm.capacity(N, E, k, gamma)
    for metric, exact in (("score", True), ("random", False)):
        base_d = cm.drop_keys(metric, 5, r["scores"], None, E)
        base_s = cm.drop_keys(metric, 5, r["topk_score"], r["topk_idx"], E)
        kd = cm.priority_keys(base_d, None, E, exact, token_class=dev(cls))
        ks = cm.priority_keys(base_s, r["topk_idx"], E, exact, token_class=dev(cls))
        ref_k = oracle.priority_keys(oracle.drop_keys(metric, 5, scores, None, E), None, E, exact, token_class=cls)
        assert np.array_equal(_bits(kd), ref_k)
        assert np.array_equal(_bits(ks), np.take_along_axis(ref_k, idx, 1))
        _same_drop(cm.token_drop(ks, r["topk_idx"], E, C), oracle.drop_keyed(ref_k, idx, C),
                   ("kept", "offsets", "slot_row"))
        _same_drop(cm.expanded_drop(kd, r["topk_idx"], C, D), oracle.drop_keyed(ref_k, idx, C, D, True))


@pytest.mark.parametrize("N,E,k,D,q,gamma", CASES)
def test_expanded_drop_topk_first(cm, N, E, k, D, q, gamma):
    r, scores, idx = _route(cm, N, E, k, q)
    C = cm.capacity(N, E, k, gamma)
    keys = cm.priority_keys(cm.drop_keys("score", 0, r["scores"], None, E), None, E, True, topk_idx=r["topk_idx"])
    ref_k = oracle.priority_keys(oracle.drop_keys("score", 0, scores, None, E), None, E, True, topk_idx=idx)
    assert np.array_equal(_bits(keys), ref_k)
    got = cm.expanded_drop(keys, r["topk_idx"], C, D)
    _same_drop(got, oracle.drop_keyed(ref_k, idx, C, D, True))
    # its top-k part is Token Drop's result
    td = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
    W = (E + 63) // 64
    tk = np.zeros((N, W), np.uint64)
    for j in range(k):
        np.bitwise_or.at(tk, (np.arange(N), idx[:, j] >> 6), np.uint64(1) << (idx[:, j] & 63).astype(np.uint64))
    assert np.array_equal(host_mask(got["keep_mask"]) & tk, host_mask(td["keep_mask"]))


@pytest.mark.parametrize("N,E,k,D,q,gamma", CASES)
def test_limit_experts_and_rows_from_mask(cm, N, E, k, D, q, gamma):
    r, scores, idx = _route(cm, N, E, k, q)
    C = cm.capacity(N, E, k, gamma)
    m = E // D
    ed = cm.expanded_drop(r["scores"], r["topk_idx"], C, D)
    ref = oracle.expanded_drop(scores, idx, C, D)
    # rebuilding the rows of the untouched mask gives the drop's own outputs back
    rb = cm.rows_from_mask(ed["keep_mask"], r["topk_idx"], E, k + m, D)
    for key in ("kept", "offsets", "slot_row"):
        assert np.array_equal(rb[key].cpu().numpy(), ref[key]), key
    assert int(rb["bad"].item()) == 0
    for k_max in (k, 1, 0):
        mask = ed["keep_mask"].clone()
        cm.limit_experts(r["scores"], mask, k_max)
        ref_mask = oracle.limit_experts(scores, ref["keep_mask"], k_max)
        assert np.array_equal(host_mask(mask), ref_mask)
        rb = cm.rows_from_mask(mask, r["topk_idx"], E, k + m, D)
        rr = oracle.rows_from_mask(ref_mask, idx, E, k + m, D)
        for key in ("kept", "offsets", "slot_row"):
            assert np.array_equal(rb[key].cpu().numpy(), rr[key]), (k_max, key)
    # Token Drop layout (slots = k) as well
    td = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
    rb = cm.rows_from_mask(td["keep_mask"], r["topk_idx"], E, k)
    for key in ("kept", "offsets", "slot_row"):
        assert np.array_equal(rb[key].cpu().numpy(), td[key].cpu().numpy()), key
    # a bit that is on none of the token's slots raises the flag
    bad = td["keep_mask"].clone()
    e_out = next(e for e in range(E) if e not in idx[0])
    bad[0, e_out >> 6] |= (1 << (e_out & 63)) if (e_out & 63) < 63 else -(1 << 63)
    assert int(cm.rows_from_mask(bad, r["topk_idx"], E, k)["bad"].item()) == 1


def test_rows_from_mask_empty_batch_and_workspace(cm):
    E, k = 8, 2
    idx = torch.zeros((0, k), device="cuda", dtype=torch.int32)
    mask = torch.zeros((0, 1), device="cuda", dtype=torch.int64)
    rb = cm.rows_from_mask(mask, idx, E, k)
    assert not rb["kept"].any() and not rb["offsets"].any()
    r, _, _ = _route(cm, 1000, E, k, 0.0)
    td = cm.token_drop(r["topk_score"], r["topk_idx"], E, 100)
    with pytest.raises(cm.CapmoeError) as e:
        cm.rows_from_mask(td["keep_mask"], r["topk_idx"], E, k, ws=torch.empty((64,), device="cuda", dtype=torch.uint8))
    assert e.value.status == cm.EWORKSPACE


def test_global_expansion_is_route_with_more_choices(cm):
    N, E, k, m = 3000, 60, 4, 15
    lg = synth.synthetic_logits(N, E, 9, bias=bias_for(E))
    r = cm.route(None, None, None, k + m, logits_in=dev(lg))
    C = cm.capacity(N, E, k, 1.0)
    got = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
    s = oracle.softmax(lg)
    idx, _, _ = oracle.topk(s, k + m)
    _same_drop(got, oracle.token_drop(s, idx, C), ("kept", "offsets", "slot_row"))


@pytest.mark.parametrize("variant", ["topk_first", "with_max", "image_first"])
def test_layer_from_stage_calls(cm, variant):
    """route -> keys -> Expanded Drop -> (limit, rows) -> permute -> FFN -> combine against the
    CPU checker run on the same decisions."""
    cfg = synth.CONFIGS["olmoe"].with_(N=1200, d=256, F=192, E=16, k=4, D=4)
    inp = synth.make_layer_inputs(cfg)
    g = {n: getattr(inp, n).cuda() for n in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}
    N, E, k, D, m = cfg.N, cfg.E, cfg.k, cfg.D, cfg.E // cfg.D
    r = cm.route(g["x"], g["w_router"], g["bias"], k)
    scores, idx = r["scores"].cpu().numpy(), r["topk_idx"].cpu().numpy()
    C = cm.capacity(N, E, k, 1.0)
    base = cm.drop_keys("score", 0, r["scores"], None, E)
    ref_base = oracle.drop_keys("score", 0, scores, None, E)
    if variant == "topk_first":
        keys = cm.priority_keys(base, None, E, True, topk_idx=r["topk_idx"])
        ref_k = oracle.priority_keys(ref_base, None, E, True, topk_idx=idx)
    elif variant == "image_first":
        cls = ((np.arange(N) % 5) < 2).astype(np.uint8)
        keys = cm.priority_keys(base, None, E, True, token_class=dev(cls))
        ref_k = oracle.priority_keys(ref_base, None, E, True, token_class=cls)
    else:
        keys, ref_k = base, ref_base
    ed = cm.expanded_drop(keys, r["topk_idx"], C, D)
    ref = oracle.drop_keyed(ref_k, idx, C, D, True)
    slot_row, offsets, ref_rows = ed["slot_row"], ed["offsets"], ref["slot_row"]
    if variant == "with_max":
        cm.limit_experts(r["scores"], ed["keep_mask"], k)
        rb = cm.rows_from_mask(ed["keep_mask"], r["topk_idx"], E, k + m, D)
        slot_row, offsets = rb["slot_row"], rb["offsets"]
        ref_rows = oracle.rows_from_mask(oracle.limit_experts(scores, ref["keep_mask"], k), idx, E, k + m, D)["slot_row"]
        assert int((slot_row >= 0).sum(1).max()) <= k
    assert np.array_equal(slot_row.cpu().numpy(), ref_rows)
    A = int(offsets[-1].item())
    pm = cm.permute(g["x"], r["scores"], r["topk_idx"], slot_row, max(A, 1), D)
    y_perm = cm.grouped_ffn(pm["x_perm"], offsets, g["w_gate"], g["w_up"], g["w_down"])
    y = cm.combine(y_perm, slot_row, pm["perm_weight"])
    torch.cuda.synchronize()
    tokens = np.arange(0, N, 7, dtype=np.int32)
    y_ref = oracle.layer_tokens(to_np(inp.x), tokens, scores, idx, ref_rows, D, to_np(inp.w_gate), to_np(inp.w_up),
                                to_np(inp.w_down), cfg.dtype)
    assert rel_err(as_f64(y)[tokens], y_ref) <= TOL[cfg.dtype]


@pytest.mark.parametrize("mode,kw", [
    ("token_drop", dict(metric="order")),
    ("token_drop", dict(metric="random", seed=11)),
    ("token_drop", dict(image_first=True)),
    ("expanded_drop", dict(topk_first=True)),
    ("expanded_drop", dict(image_first=True, topk_first=True)),
    ("expanded_drop", dict(max_experts=4)),
    ("expanded_drop", dict(metric="reverse_order", max_experts=2)),
])
def test_layer_forward_with_variants(cm, mode, kw):
    """The same variants selected through the layer struct: one capmoe_layer_forward call."""
    cfg = synth.CONFIGS["olmoe"].with_(N=1500, d=256, F=192, E=16, k=4, D=4)
    inp = synth.make_layer_inputs(cfg)
    g = {n: getattr(inp, n).cuda() for n in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}
    N, E, k, D, m = cfg.N, cfg.E, cfg.k, cfg.D, cfg.E // cfg.D
    kw = dict(kw)
    cls = None
    if kw.pop("image_first", False):
        cls = ((np.arange(N) % 5) < 2).astype(np.uint8)
        kw["token_class"] = dev(cls)
    layer = cm.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], k, D, mode, gamma=1.0,
                        **kw)
    y = layer.forward()
    torch.cuda.synchronize()
    layer.check_device_status()
    scores, idx = layer.t["scores"].cpu().numpy(), layer.t["topk_idx"].cpu().numpy()
    expanded = mode == "expanded_drop"
    metric, seed = kw.get("metric", "score"), kw.get("seed", 0)
    keys = oracle.drop_keys(metric, seed, scores, None, E)
    if cls is not None or kw.get("topk_first"):
        keys = oracle.priority_keys(keys, None, E, metric == "score", token_class=cls,
                                    topk_idx=idx if (expanded and kw.get("topk_first")) else None)
    ref = oracle.drop_keyed(keys, idx, layer.C, D, expanded)
    rows, mask = ref["slot_row"], ref["keep_mask"]
    if kw.get("max_experts", 0) > 0:
        mask = oracle.limit_experts(scores, mask, kw["max_experts"])
        rows = oracle.rows_from_mask(mask, idx, E, k + (m if expanded else 0), D)["slot_row"]
        assert int(layer.t["bad"].item()) == 0
    assert np.array_equal(host_mask(layer.t["keep_mask"]), mask)
    assert np.array_equal(layer.t["slot_row"].cpu().numpy(), rows)
    tokens = np.arange(0, N, 5, dtype=np.int32)
    y_ref = oracle.layer_tokens(to_np(inp.x), tokens, scores, idx, rows, D if expanded else 0, to_np(inp.w_gate),
                                to_np(inp.w_up), to_np(inp.w_down), cfg.dtype)
    assert rel_err(as_f64(y)[tokens], y_ref) <= TOL[cfg.dtype]


def test_layer_variants_are_refused_for_device_level_capacity(cm):
    cfg = synth.CONFIGS["tiny_f32"]
    inp = synth.make_layer_inputs(cfg)
    g = {n: getattr(inp, n).cuda() for n in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}
    with pytest.raises(ValueError):
        cm.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k, cfg.D,
                    "device_token_drop", metric="order")
    layer = cm.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k, cfg.D,
                        "device_token_drop")
    layer.c.metric = cm.METRICS["order"]                   # bypass the binding's own check
    with pytest.raises(cm.CapmoeError) as e:
        layer.forward()
    assert e.value.status == cm.EUNSUPPORTED
