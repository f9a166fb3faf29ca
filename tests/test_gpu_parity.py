"""Parity of the CUDA path against the CPU checker, stage by stage and end to end, through the
C ABI.  Integer outputs (keep masks, counts, offsets, permutation) must match bit for bit given
identical fp32 router logits; layer outputs within max|diff|/max|ref| <= 1e-5 (fp32 storage)
and <= 2e-2 (bf16 storage, fp32 accumulation)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.util import mask_to_dense, rel_err, to_np

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 2e-2}
ROUTER_TOL = {"f32": 1e-5, "bf16": 1e-4}


@pytest.fixture(scope="module")
def cm():
    from paper_2503_05066_b200 import capmoe
    capmoe.lib()
    return capmoe


_INPUT_CACHE = {}


def cached_inputs(cfg):
    """One set of inputs at a time (the Mixtral-shape weights are 2.8 GB on the host)."""
    if cfg not in _INPUT_CACHE:
        _INPUT_CACHE.clear()
        _INPUT_CACHE[cfg] = synth.make_layer_inputs(cfg)
    return _INPUT_CACHE[cfg]


def dev(a):
    if isinstance(a, np.ndarray):
        a = torch.from_numpy(a)
    return a.cuda().contiguous()


def host_mask(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint64)


def bias_for(E, s=1.0):
    return (-s * np.log(np.arange(E) + 1.0)).astype(np.float32)


# ----------------------------------------------------------------------------- stage 1
@pytest.mark.parametrize("name,N,d", [("tiny_f32", 512, 256), ("tiny_f32", 77, 100), ("olmoe", 300, 2048),
                                      ("mixtral", 129, 4096), ("qwen", 200, 2048), ("dsv2lite", 64, 2048)])
def test_route_matches_oracle(cm, name, N, d):
    cfg = synth.CONFIGS[name].with_(N=N, d=d)
    x, w, b = synth.hidden_states(cfg), synth.router_weights(cfg), synth.router_bias(cfg)
    out = cm.route(dev(x), dev(w), dev(b), cfg.k)
    torch.cuda.synchronize()
    ref_logits = oracle.router_logits(to_np(x), to_np(w), b.numpy(), cfg.dtype)
    got_logits = out["logits"].cpu().numpy()
    assert rel_err(got_logits.astype(np.float64), ref_logits.astype(np.float64)) <= ROUTER_TOL[cfg.dtype]
    # everything downstream of the GEMM is a pure function of the fp32 logits: bit-exact
    s_ref = oracle.softmax(got_logits)
    assert np.array_equal(out["scores"].cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    idx, val, load = oracle.topk(s_ref, cfg.k)
    assert np.array_equal(out["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["topk_score"].cpu().numpy().view(np.uint32), val.view(np.uint32))
    assert np.array_equal(out["load"].cpu().numpy(), load)


@pytest.mark.parametrize("N,E,k,q", [(1000, 8, 2, 0.0), (333, 60, 4, 0.0), (4096, 64, 8, 0.0), (500, 256, 8, 0.0),
                                     (257, 16, 16, 0.5), (64, 5, 1, 1.0), (1, 8, 2, 0.0)])
def test_route_from_given_logits(cm, N, E, k, q):
    lg = synth.synthetic_logits(N, E, 7, bias=bias_for(E), quantum=q) * np.float32(2.5)
    out = cm.route(None, None, None, k, logits_in=dev(lg))
    s_ref = oracle.softmax(lg)
    idx, val, load = oracle.topk(s_ref, k)
    assert np.array_equal(out["scores"].cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(out["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["topk_score"].cpu().numpy().view(np.uint32), val.view(np.uint32))
    assert np.array_equal(out["load"].cpu().numpy(), load)
    assert np.array_equal(out["logits"].cpu().numpy(), lg)


def test_softmax_extreme_logits(cm):
    E = 8
    lg = np.zeros((4, E), np.float32)
    lg[1, 3] = 100.0
    lg[2] = np.linspace(-85, 0, E)
    lg[3] = np.linspace(0, -79.9, E)
    out = cm.route(None, None, None, 2, logits_in=dev(lg))
    assert np.array_equal(out["scores"].cpu().numpy().view(np.uint32), oracle.softmax(lg).view(np.uint32))


@pytest.mark.parametrize("N,d,E,k,scale", [
    (333, 128, 17, 3, 1.0),        # 32 padded experts, scalar stores (E % 4 != 0)
    (1000, 256, 32, 32, 1.0),      # k = E: every expert selected, in score order
    (2500, 192, 33, 5, 1.0),       # 64 padded experts, E % 4 != 0
    (20000, 64, 60, 4, 1.0),       # several row tiles per SM, ragged last tile
    (19001, 128, 64, 8, 1.0),
    (700, 128, 63, 6, 40.0),       # logit gaps far beyond 80: exp -> 0 and quotients down to 1e-35
    (4100, 64, 24, 2, 12.0),
])
def test_route_one_launch_router(cm, N, d, E, k, scale):
    """bf16 inputs with 16 < E <= 64: GEMM, softmax, top-k and histogram in one tensor-core launch.
    Pairs of identical router rows give exact score ties, which must go to the lower expert id."""
    g = torch.Generator().manual_seed(1000 + N + E)
    x = torch.randn((N, d), generator=g).to(torch.bfloat16)
    w = (torch.randn((E, d), generator=g) * (scale / d ** 0.5)).to(torch.bfloat16)
    w[E // 2] = w[1]
    w[E - 1] = w[0]
    b = torch.zeros(E)
    b[3] = 0.25
    out = cm.route(dev(x), dev(w), dev(b), k)
    torch.cuda.synchronize()
    got_logits = out["logits"].cpu().numpy()
    ref_logits = oracle.router_logits(to_np(x), to_np(w), b.numpy(), "bf16")
    assert rel_err(got_logits.astype(np.float64), ref_logits.astype(np.float64)) <= ROUTER_TOL["bf16"]
    assert np.array_equal(got_logits[:, E // 2], got_logits[:, 1])
    s_ref = oracle.softmax(got_logits)
    assert np.array_equal(out["scores"].cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    idx, val, load = oracle.topk(s_ref, k)
    assert np.array_equal(out["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["topk_score"].cpu().numpy().view(np.uint32), val.view(np.uint32))
    assert np.array_equal(out["load"].cpu().numpy(), load)
    if scale > 1.0:
        assert (s_ref == 0).any() or s_ref[s_ref > 0].min() < 1e-20


# ----------------------------------------------------------------------------- stages 2, 3
DROP_CASES = [
    # N, E, k, D, gamma, quantum
    (512, 8, 2, 2, 1.0, 0.0),        # tiny config
    (4096, 64, 8, 8, 1.0, 0.0),      # OLMoE-like
    (4096, 64, 8, 8, 1.5, 0.0),
    (3000, 60, 4, 4, 0.5, 0.0),      # E not a power of two, ragged N
    (3000, 60, 4, 4, 2.0, 0.0),
    (2049, 8, 2, 2, 1.25, 0.0),      # just over two 1024-token chunks
    (1023, 16, 4, 1, 1.0, 0.0),      # D = 1
    (640, 16, 2, 16, 1.0, 0.0),      # D = E (one expert per device)
    (700, 8, 8, 2, 1.0, 0.0),        # k = E
    (5000, 8, 2, 2, 1.0, 0.5),       # quantised logits: many exact ties
    (2500, 64, 8, 8, 1.0, 1.0),      # heavy ties
    (900, 130, 6, 10, 1.0, 0.0),     # two mask words... E = 130
    (100, 8, 2, 2, 0.0, 0.0),        # gamma = 0: everything dropped
    (100, 8, 2, 2, float("inf"), 0.0),
    (1, 8, 2, 2, 1.0, 0.0),
    (7, 4, 1, 2, 1.0, 0.0),
    # cluster select with several tokens per thread (2, 4, 8) and clusters of 8, 4, 2 and 1 CTAs
    (20000, 8, 2, 2, 1.0, 0.5),      # ties at the threshold
    (16384, 64, 8, 8, 1.0, 0.0),
    (40000, 8, 2, 2, 1.0, 0.25),
    (16384, 8, 2, 2, 0.0, 0.0),
    (16384, 8, 2, 2, float("inf"), 0.0),
    (3500, 130, 6, 10, 1.0, 0.0),
    (4000, 200, 4, 8, 1.0, 1.0),
    (16000, 60, 4, 4, 1.0, 1.0),     # Expanded Drop: 8 tokens per thread with many experts, heavy ties
    (15000, 64, 8, 8, 0.5, 0.5),
    # the limits of the interface: 256 experts, 32 experts per token
    (600, 256, 32, 8, 1.0, 0.0),
    (300, 256, 32, 256, 1.0, 0.5),
    (9000, 256, 32, 4, 1.5, 0.0),
    # larger batches take the token-parallel select
    (17001, 60, 4, 4, 0.5, 1.0),     # ties at the threshold resolved by position
    (16400, 130, 6, 10, 1.0, 0.0),
    (40000, 64, 8, 8, 1.0, 0.0),
    (70000, 8, 2, 2, 1.0, 0.5),
    (70000, 8, 2, 2, 0.0, 0.0),
    (70000, 8, 2, 2, float("inf"), 0.0),
]


def _routing(cm, N, E, k, q, seed=3, s=1.0):
    lg = synth.synthetic_logits(N, E, seed, bias=bias_for(E, s), quantum=q)
    r = cm.route(None, None, None, k, logits_in=dev(lg))
    scores = r["scores"].cpu().numpy()
    idx = r["topk_idx"].cpu().numpy()
    return r, scores, idx


@pytest.mark.parametrize("N,E,k,D,gamma,q", DROP_CASES)
def test_token_drop_bit_exact(cm, N, E, k, D, gamma, q):
    r, scores, idx = _routing(cm, N, E, k, q)
    C = cm.capacity(N, E, k, gamma)
    assert C == oracle.capacity(N, E, k, gamma)
    got = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
    ref = oracle.token_drop(scores, idx, C)
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    assert np.array_equal(got["kept"].cpu().numpy(), ref["kept"])
    assert np.array_equal(got["offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(got["slot_row"].cpu().numpy(), ref["slot_row"])


@pytest.mark.parametrize("N,E,k,D,gamma,q", DROP_CASES)
def test_expanded_drop_bit_exact(cm, N, E, k, D, gamma, q):
    r, scores, idx = _routing(cm, N, E, k, q)
    C = cm.capacity(N, E, k, gamma)
    got = cm.expanded_drop(r["scores"], r["topk_idx"], C, D)
    ref = oracle.expanded_drop(scores, idx, C, D)
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    assert np.array_equal(got["cand"].cpu().numpy(), ref["cand"])
    assert np.array_equal(got["kept"].cpu().numpy(), ref["kept"])
    assert np.array_equal(got["offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(got["slot_row"].cpu().numpy(), ref["slot_row"])


def test_expanded_drop_explicit_groups(cm):
    N, E, k, D = 1500, 16, 2, 4
    r, scores, idx = _routing(cm, N, E, k, 0.0)
    tg = (synth.token_permutation(N, 5) % D).astype(np.int32)      # scattered home devices
    C = cm.capacity(N, E, k, 1.0)
    got = cm.expanded_drop(r["scores"], r["topk_idx"], C, D, token_group=dev(tg))
    ref = oracle.expanded_drop(scores, idx, C, D, token_group=tg)
    for key in ("cand", "kept", "offsets", "slot_row"):
        assert np.array_equal(got[key].cpu().numpy(), ref[key]), key
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])


def test_drop_is_deterministic_across_runs(cm):
    N, E, k, D = 6000, 64, 8, 8
    r, _, _ = _routing(cm, N, E, k, 0.5)
    C = cm.capacity(N, E, k, 1.0)
    first = cm.expanded_drop(r["scores"], r["topk_idx"], C, D)
    for _ in range(5):
        again = cm.expanded_drop(r["scores"], r["topk_idx"], C, D)
        for key in first:
            assert torch.equal(first[key], again[key]), key


def test_drop_empty_batch(cm):
    E, k = 8, 2
    z = torch.empty((0, k), device="cuda")
    got = cm.token_drop(z.float(), z.int(), E, 0)
    assert got["offsets"].cpu().tolist() == [0] * (E + 1) and got["kept"].cpu().tolist() == [0] * E


# ----------------------------------------------------------------------------- stages 4, 6
@pytest.mark.parametrize("dtype,d", [("f32", 256), ("bf16", 2048), ("bf16", 72), ("f32", 36)])
@pytest.mark.parametrize("mode", ["token_drop", "expanded_drop"])
def test_permute_and_combine(cm, dtype, d, mode):
    N, E, k, D = 777, 16, 4, 4
    cfg = synth.CONFIGS["tiny_f32"].with_(N=N, d=d, E=E, k=k, D=D, dtype=dtype)
    x = synth.hidden_states(cfg)
    r, scores, idx = _routing(cm, N, E, k, 0.0)
    C = cm.capacity(N, E, k, 1.0)
    if mode == "token_drop":
        got = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
        ref = oracle.token_drop(scores, idx, C)
        Dp = 0
    else:
        got = cm.expanded_drop(r["scores"], r["topk_idx"], C, D)
        ref = oracle.expanded_drop(scores, idx, C, D)
        Dp = D
    A = int(ref["offsets"][-1])
    A_max = cm.max_rows(N, E, k, D, C, mode == "expanded_drop")
    assert A <= A_max
    p = cm.permute(dev(x), r["scores"], r["topk_idx"], got["slot_row"], A_max, Dp)
    pref = oracle.permute(to_np(x), scores, idx, ref["slot_row"], A, Dp, dtype)
    assert np.array_equal(p["perm_token"].cpu().numpy()[:A], pref["perm_token"])
    assert np.array_equal(p["perm_weight"].cpu().numpy()[:A].view(np.uint32), pref["perm_weight"].view(np.uint32))
    assert np.array_equal(to_np(p["x_perm"])[:A], pref["x_perm"])
    # identity experts: combine(permute(x)) against the checker's double-precision combine
    y = cm.combine(p["x_perm"], got["slot_row"], p["perm_weight"])
    yref = oracle.combine(pref["x_perm"].astype(np.float64) if dtype == "f32"
                          else x.double().numpy()[pref["perm_token"]], ref["slot_row"], scores, idx, Dp)
    assert rel_err(y.double().cpu().numpy(), yref) <= (2e-6 if dtype == "f32" else 6e-3)
    # tokens with nothing kept give exact zeros; a shared term is added with weight one
    none_kept = mask_to_dense(ref["keep_mask"], E).sum(1) == 0
    assert torch.all(y[torch.from_numpy(none_kept).cuda()] == 0)
    ysh = cm.combine(p["x_perm"], got["slot_row"], p["perm_weight"], y_shared=dev(x))
    yref2 = yref + x.double().numpy()
    assert rel_err(ysh.double().cpu().numpy(), yref2) <= (2e-6 if dtype == "f32" else 6e-3)


# ----------------------------------------------------------------------------- stage 5 and the layer
def _layer_case(cm, cfg, mode, gamma, straggler=False, sample=None, std=0.02, cover_blocks=False):
    """Run the CUDA layer, then the checker from the GPU's own fp32 logits; compare.
    sample: compare the layer output on that many random tokens (None = all).  cover_blocks: also
    on one token out of every 128-row block of every expert's row segment (and of every 128-token
    block of the batch when there is a shared expert), so that every row tile of both GEMMs is checked."""
    inp = cached_inputs(cfg)
    wg, wu, wd = inp.w_gate, inp.w_up, inp.w_down
    shared = inp.shared
    layer = cm.MoELayer(dev(inp.x), dev(inp.w_router), dev(inp.bias), dev(wg), dev(wu), dev(wd), cfg.k, cfg.D,
                        mode, gamma=gamma, straggler=straggler,
                        shared=None if shared is None else tuple(dev(s) for s in shared))
    y = layer.forward()
    torch.cuda.synchronize()
    layer.check_device_status()
    t = layer.t
    logits = t["logits"].cpu().numpy()
    ref_logits = oracle.router_logits(to_np(inp.x), to_np(inp.w_router), inp.bias.numpy(), cfg.dtype)
    assert rel_err(logits.astype(np.float64), ref_logits.astype(np.float64)) <= ROUTER_TOL[cfg.dtype]
    scores = oracle.softmax(logits)
    idx, val, load = oracle.topk(scores, cfg.k)
    C = cfg.N if mode == "nodrop" else oracle.capacity(cfg.N, cfg.E, cfg.k, gamma)
    if mode == "expanded_drop":
        ref = oracle.expanded_drop(scores, idx, C, cfg.D)
        Dp = cfg.D
    else:
        ref = oracle.token_drop(scores, idx, C)
        Dp = 0
    assert np.array_equal(t["scores"].cpu().numpy().view(np.uint32), scores.view(np.uint32))
    assert np.array_equal(t["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(t["load"].cpu().numpy(), load)
    assert np.array_equal(host_mask(t["keep_mask"]), ref["keep_mask"])
    assert np.array_equal(t["kept"].cpu().numpy(), ref["kept"])
    assert np.array_equal(t["expert_offsets"].cpu().numpy(), ref["offsets"])
    assert np.array_equal(t["slot_row"].cpu().numpy(), ref["slot_row"])
    A = int(ref["offsets"][-1])
    pref = oracle.permute(None, scores, idx, ref["slot_row"], A, Dp, cfg.dtype)
    assert np.array_equal(t["perm_token"].cpu().numpy()[:A], pref["perm_token"])
    xs = to_np(inp.x)
    args = (to_np(wg), to_np(wu), to_np(wd))
    if sample is None:
        toks = np.arange(cfg.N, dtype=np.int32)
    else:
        rng = np.random.default_rng(0)
        picks = [np.array([0, cfg.N - 1]), rng.integers(0, cfg.N, sample)]
        if cover_blocks:
            off = ref["offsets"].astype(np.int64)
            rows = []
            for e in range(cfg.E):
                for r0 in range(int(off[e]), int(off[e + 1]), 128):
                    rows.append(r0 + int(rng.integers(0, min(128, int(off[e + 1]) - r0))))
            picks.append(pref["perm_token"][np.array(rows, dtype=np.int64)] if rows else np.array([], np.int64))
            if shared is not None:
                starts = np.arange(0, cfg.N, 128)
                picks.append(starts + rng.integers(0, np.minimum(128, cfg.N - starts)))
        toks = np.unique(np.concatenate(picks)).astype(np.int32)
    yref = oracle.layer_tokens(xs, toks, scores, idx, ref["slot_row"], Dp, *args, cfg.dtype)
    if shared is not None:
        ysh = oracle.expert_ffn(np.ascontiguousarray(xs[toks]), None, *(to_np(s) for s in shared), cfg.dtype)
        yref = yref + ysh
    got = y.double().cpu().numpy()[toks]
    # normalise by the largest reference magnitude over the compared rows
    err = rel_err(got, yref)
    assert err <= TOL[cfg.dtype], err
    return layer, err


@pytest.mark.parametrize("mode", ["nodrop", "token_drop", "expanded_drop"])
def test_layer_tiny_fp32(cm, mode):
    _layer_case(cm, synth.CONFIGS["tiny_f32"], mode, 1.0)


@pytest.mark.parametrize("mode", ["nodrop", "token_drop", "expanded_drop"])
@pytest.mark.parametrize("dtype,d,F", [("bf16", 64, 128), ("f32", 24, 20)])
def test_layer_at_the_expert_and_k_limits(cm, mode, dtype, d, F):
    """256 experts, 32 per token, 8 devices: 64 slots per token under Expanded Drop."""
    cfg = synth.CONFIGS["tiny_f32"].with_(N=700, d=d, F=F, E=256, k=32, D=8, dtype=dtype, bias_kind="zipf")
    _layer_case(cm, cfg, mode, 1.0)


@pytest.mark.parametrize("mode", ["nodrop", "token_drop", "expanded_drop"])
def test_layer_fp32_ragged_shapes(cm, mode):
    cfg = synth.CONFIGS["tiny_f32"].with_(N=333, d=100, F=72, E=6, k=3, D=3)
    _layer_case(cm, cfg, mode, 1.0)


def test_layer_fp32_gamma_limits(cm):
    cfg = synth.CONFIGS["tiny_f32"].with_(N=200, d=64, F=48)
    nd, _ = _layer_case(cm, cfg, "nodrop", 1.0)
    inf, _ = _layer_case(cm, cfg, "token_drop", float("inf"))
    assert torch.equal(nd.t["y"], inf.t["y"])                   # gamma = inf is the no-drop layer
    zero, _ = _layer_case(cm, cfg, "token_drop", 0.0)
    assert torch.all(zero.t["y"] == 0)


@pytest.mark.parametrize("mode,gamma", [("nodrop", 1.0), ("token_drop", 1.0), ("expanded_drop", 1.5)])
def test_layer_bf16_small(cm, mode, gamma):
    # OLMoE-like proportions, shrunk so the checker finishes in seconds; spans several tiles and ragged tails
    cfg = synth.CONFIGS["olmoe"].with_(N=600, d=256, F=384, E=16, k=4, D=4)
    _layer_case(cm, cfg, mode, gamma)


def test_layer_bf16_shared_expert(cm):
    cfg = synth.CONFIGS["dsv2lite"].with_(N=300, d=256, F=128, E=16, k=3, D=4, F_shared=256)
    _layer_case(cm, cfg, "token_drop", 1.0)


def test_layer_bf16_odd_shape_uses_plain_kernel(cm):
    cfg = synth.CONFIGS["qwen"].with_(N=250, d=72, F=40, E=12, k=4, D=4)
    assert not cm.ffn_uses_tensor_cores(cfg.d, cfg.F, torch.bfloat16)
    _layer_case(cm, cfg, "expanded_drop", 1.0)


def test_layer_host_buffers_round_trip(cm):
    cfg = synth.CONFIGS["tiny_f32"]
    inp = synth.make_layer_inputs(cfg)
    layer = cm.MoELayer(torch.zeros_like(inp.x).cuda(), dev(inp.w_router), dev(inp.bias), dev(inp.w_gate),
                        dev(inp.w_up), dev(inp.w_down), cfg.k, cfg.D, "token_drop", gamma=1.0)
    xh = inp.x.clone().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    layer.forward_host(xh, yh)
    torch.cuda.synchronize()
    ref = cm.MoELayer(dev(inp.x), dev(inp.w_router), dev(inp.bias), dev(inp.w_gate), dev(inp.w_up),
                      dev(inp.w_down), cfg.k, cfg.D, "token_drop", gamma=1.0)
    y = ref.forward()
    torch.cuda.synchronize()
    assert torch.equal(yh, y.cpu())
