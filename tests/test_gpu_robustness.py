"""Run-to-run determinism, out-of-bounds guard bands around every output, the bounded device-side
wait, and status codes of the GPU entry points."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2503_05066_b200 import synth

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes of canary on each side of a guarded buffer
PATTERN = 0xA5


@pytest.fixture(scope="module")
def cm():
    from paper_2503_05066_b200 import capmoe
    capmoe.lib()
    return capmoe


class Guarded:
    """A device buffer with canary bytes before and after the part handed to the library."""

    def __init__(self, nbytes: int):
        self.nbytes = nbytes
        self.raw = torch.full((nbytes + 2 * GUARD,), PATTERN, device="cuda", dtype=torch.uint8)

    @property
    def ptr(self):
        return ctypes.c_void_p(self.raw.data_ptr() + GUARD)

    def view(self, dtype, shape):
        return self.raw[GUARD:GUARD + self.nbytes].view(dtype).view(shape)

    def intact(self) -> bool:
        return bool((self.raw[:GUARD] == PATTERN).all() and (self.raw[GUARD + self.nbytes:] == PATTERN).all())


def _inputs(cfg):
    inp = synth.make_layer_inputs(cfg)
    return {k: getattr(inp, k).cuda() for k in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}


@pytest.mark.parametrize("name,mode", [("tiny_f32", "expanded_drop"), ("olmoe", "token_drop"), ("olmoe", "expanded_drop")])
def test_layer_outputs_are_bit_identical_across_runs(cm, name, mode):
    cfg = synth.CONFIGS[name] if name == "tiny_f32" else synth.CONFIGS[name].with_(N=1500, d=512, F=256, E=16, k=4, D=4)
    g = _inputs(cfg)
    layer = cm.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k, cfg.D, mode,
                        gamma=1.0)
    keys = ["logits", "scores", "topk_idx", "topk_score", "load", "keep_mask", "kept", "expert_offsets", "slot_row",
            "perm_token", "perm_weight", "y"]
    layer.forward()
    torch.cuda.synchronize()
    first = {k: layer.t[k].clone() for k in keys}
    A = int(first["expert_offsets"][-1])
    for _ in range(9):
        layer.forward()
        torch.cuda.synchronize()
        for k in keys:
            a, b = first[k], layer.t[k]
            if k in ("perm_token", "perm_weight"):
                a, b = a[:A], b[:A]
            assert torch.equal(a, b), k


def test_no_stage_writes_outside_its_outputs(cm):
    """Every output buffer sits between canaries; rows of x_perm / y_perm beyond A stay untouched."""
    cfg = synth.CONFIGS["olmoe"].with_(N=777, d=256, F=192, E=12, k=3, D=4)      # ragged everything
    g = _inputs(cfg)
    L = cm.lib()
    N, d, E, k, F, D = cfg.N, cfg.d, cfg.E, cfg.k, cfg.F, cfg.D
    m, W = E // D, 1
    slots = k + m
    C = cm.capacity(N, E, k, 1.0)
    A_max = cm.max_rows(N, E, k, D, C, True)
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    i64 = ctypes.c_int64
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    bufs = dict(logits=Guarded(N * E * 4), scores=Guarded(N * E * 4), topk_idx=Guarded(N * k * 4),
                topk_score=Guarded(N * k * 4), load=Guarded(E * 4), keep_mask=Guarded(N * W * 8),
                cand=Guarded(E * 4), kept=Guarded(E * 4), offsets=Guarded((E + 1) * 4),
                slot_row=Guarded(N * slots * 4), x_perm=Guarded(A_max * d * 2), perm_token=Guarded(A_max * 4),
                perm_weight=Guarded(A_max * 4), h=Guarded(A_max * F * 2), y_perm=Guarded(A_max * d * 2),
                y=Guarded(N * d * 2), ws=Guarded(cm.drop_workspace_bytes(N, E, k, D, True)))
    b = bufs
    assert L.capmoe_route(p(g["x"]), p(g["w_router"]), p(g["bias"]), None, i64(N), d, E, k, cm.BF16, b["logits"].ptr,
                          b["scores"].ptr, b["topk_idx"].ptr, b["topk_score"].ptr, b["load"].ptr, st) == cm.OK
    assert L.capmoe_expanded_drop(b["scores"].ptr, b["topk_idx"].ptr, i64(N), E, k, i64(C), D, None,
                                  b["keep_mask"].ptr, b["cand"].ptr, b["kept"].ptr, b["offsets"].ptr,
                                  b["slot_row"].ptr, b["ws"].ptr, ctypes.c_size_t(b["ws"].nbytes), st) == cm.OK
    assert L.capmoe_permute(p(g["x"]), i64(N), d, E, k, slots, D, cm.BF16, b["scores"].ptr, b["topk_idx"].ptr, None,
                            b["slot_row"].ptr, b["x_perm"].ptr, b["perm_token"].ptr, b["perm_weight"].ptr,
                            st) == cm.OK
    assert L.capmoe_grouped_ffn(b["x_perm"].ptr, b["offsets"].ptr, E, d, F, cm.BF16, p(g["w_gate"]), p(g["w_up"]),
                                p(g["w_down"]), b["h"].ptr, b["y_perm"].ptr, i64(A_max), 0, None, st) == cm.OK
    assert L.capmoe_combine(b["y_perm"].ptr, b["slot_row"].ptr, b["perm_weight"].ptr, i64(N), d, slots, cm.BF16, None,
                            b["y"].ptr, st) == cm.OK
    torch.cuda.synchronize()
    for name, buf in bufs.items():
        assert buf.intact(), name
    A = int(b["offsets"].view(torch.int32, (E + 1,))[-1])
    assert 0 < A <= A_max
    if A < A_max:       # the tail rows were never written: still the fill pattern
        for name, cols in (("x_perm", d), ("y_perm", d)):
            tail = b[name].view(torch.uint8, (A_max, cols * 2))[A:]
            assert bool((tail == PATTERN).all()), name
    assert torch.isfinite(b["y"].view(torch.bfloat16, (N, d)).float()).all()


def test_bounded_wait_runs_out_and_reports(cm):
    """A wait on a barrier nothing signals must end by itself and raise the status word."""
    assert cm.debug_wait_probe(20_000_000) == cm.ETIMEOUT
    # the context is still usable afterwards
    x = torch.ones(8, device="cuda")
    assert float(x.sum()) == 8.0
    assert cm.debug_wait_probe(1_000_000) == cm.ETIMEOUT


def test_status_codes_from_gpu_calls(cm):
    cfg = synth.CONFIGS["tiny_f32"]
    g = _inputs(cfg)
    r = cm.route(g["x"], g["w_router"], g["bias"], cfg.k)
    # workspace too small
    small = torch.empty((64,), device="cuda", dtype=torch.uint8)
    with pytest.raises(cm.CapmoeError) as e:
        cm.token_drop(r["topk_score"], r["topk_idx"], cfg.E, 10, ws=small)
    assert e.value.status == cm.EWORKSPACE
    # capacity beyond N
    with pytest.raises(cm.CapmoeError) as e:
        cm.token_drop(r["topk_score"], r["topk_idx"], cfg.E, cfg.N + 1)
    assert e.value.status == cm.EINVAL
    # straggler groups on a shape the tensor-core kernel does not take
    td = cm.token_drop(r["topk_score"], r["topk_idx"], cfg.E, cfg.N)
    pm = cm.permute(g["x"], r["scores"], r["topk_idx"], td["slot_row"], cfg.N * cfg.k)
    with pytest.raises(cm.CapmoeError) as e:
        cm.grouped_ffn(pm["x_perm"], td["offsets"], g["w_gate"], g["w_up"], g["w_down"], D_straggler=2)
    assert e.value.status == cm.EUNSUPPORTED
    # and nothing above left an error behind
    torch.cuda.synchronize()
    y = cm.grouped_ffn(pm["x_perm"], td["offsets"], g["w_gate"], g["w_up"], g["w_down"])
    assert torch.isfinite(y).all()


@pytest.mark.parametrize("name,mode", [("tiny_f32", "token_drop"), ("olmoe", "expanded_drop"),
                                       ("olmoe", "device_expanded_drop")])
def test_cuda_graph_replay_matches_direct_launches(cm, name, mode):
    cfg = synth.CONFIGS[name] if name == "tiny_f32" else synth.CONFIGS[name].with_(N=2048, d=512, F=256, E=16, k=4, D=4)
    g = _inputs(cfg)
    layer = cm.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k, cfg.D, mode,
                        gamma=1.0)
    y0 = layer.forward().clone()
    torch.cuda.synchronize()
    keep0, rows0 = layer.t["keep_mask"].clone(), layer.t["slot_row"].clone()
    layer.capture_graph()
    for _ in range(3):
        layer.t["y"].zero_()
        layer.t["slot_row"].fill_(12345)
        y = layer.replay()
        torch.cuda.synchronize()
        assert torch.equal(y, y0) and torch.equal(layer.t["keep_mask"], keep0) and torch.equal(layer.t["slot_row"], rows0)
    layer.check_device_status()


def test_ffn_result_does_not_depend_on_how_tiles_are_handed_out(cm):
    """Long expert segments run on CTA pairs that take their tiles from a device counter when the
    caller lends a status block, and walk fixed lists without one: same bits either way, run after run."""
    E, d, F, rows = 4, 2048, 256, 1536
    A = E * rows
    g = torch.Generator().manual_seed(5)
    x_perm = torch.randn((A, d), generator=g).to(torch.bfloat16).cuda()
    wg = (torch.randn((E, F, d), generator=g) * 0.02).to(torch.bfloat16).cuda()
    wu = (torch.randn((E, F, d), generator=g) * 0.02).to(torch.bfloat16).cuda()
    wd = (torch.randn((E, d, F), generator=g) * 0.02).to(torch.bfloat16).cuda()
    offsets = torch.arange(0, A + 1, rows, dtype=torch.int32).cuda()
    L = cm.lib()
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def run(status, D_straggler):
        h = torch.empty((A, F), device="cuda", dtype=torch.bfloat16)
        y = torch.zeros((A, d), device="cuda", dtype=torch.bfloat16)
        rc = L.capmoe_grouped_ffn(p(x_perm), p(offsets), E, d, F, cm.BF16, p(wg), p(wu), p(wd), p(h), p(y),
                                  ctypes.c_int64(A), D_straggler, None if status is None else p(status), st)
        assert rc == cm.OK
        torch.cuda.synchronize()
        return y

    for D_straggler in (0, 2):
        fixed = run(None, D_straggler)
        status = torch.zeros((cm.FFN_STATUS_WORDS,), device="cuda", dtype=torch.int32)
        for _ in range(3):
            assert torch.equal(run(status, D_straggler), fixed)
            assert int(status[0].item()) == cm.OK
        # each GEMM's counters handed out every one of its tiles, then ran past the end once per pair
        groups = max(D_straggler, 1)
        for base, n_tiles in ((1, (A // 256) * (F // 128)), (63, (A // 256) * (d // 256))):
            assert int(status[base:base + groups].sum().item()) >= n_tiles
    assert torch.isfinite(fixed.float()).all() and float(fixed.float().abs().max()) > 0


@pytest.mark.parametrize("name,mode,over", [
    ("olmoe", "expanded_drop", dict(N=4096, d=512, F=256)),          # CTA pairs, tile counters, per-expert select
    ("qwen", "device_expanded_drop", dict(N=6000, d=256, F=128)),    # token-parallel select, ragged segments
])
def test_two_layers_on_two_streams_do_not_disturb_each_other(cm, name, mode, over):
    """Two instances (own buffers and status blocks, shared weights) running at the same time on two
    streams give, step after step, the bits a lone forward gives."""
    cfg = synth.CONFIGS[name].with_(**over)
    g = _inputs(cfg)
    mk = lambda: cm.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k, cfg.D,
                             mode, gamma=1.0)
    a, b = mk(), mk()
    ref = a.forward().clone()
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    for it in range(60):
        with torch.cuda.stream(s1):
            ya = a.forward()
        with torch.cuda.stream(s2):
            yb = b.forward()
        if it % 20 == 19:
            torch.cuda.synchronize()
            assert torch.equal(ya, ref) and torch.equal(yb, ref), it
    torch.cuda.synchronize()
    a.check_device_status()
    b.check_device_status()


def test_debug_index_check_passes_on_real_drops_and_flags_bad_indices(cm):
    """The index check (the stand-in for a memory checker) accepts what the drop stages produce and
    flags, through the status word and without touching anything, a row outside its expert's segment,
    a row count beyond the buffers, and offsets that go backwards."""
    import numpy as np
    from paper_2503_05066_b200 import synth
    N, E, k, D = 3000, 16, 4, 4
    lg = synth.synthetic_logits(N, E, 8, bias=(-np.log(np.arange(E) + 1.0)).astype(np.float32))
    r = cm.route(None, None, None, k, logits_in=torch.from_numpy(lg).cuda())
    C = cm.capacity(N, E, k, 1.0)
    td = cm.token_drop(r["topk_score"], r["topk_idx"], E, C)
    ed = cm.expanded_drop(r["scores"], r["topk_idx"], C, D)
    A_td, A_ed = int(td["offsets"][-1]), int(ed["offsets"][-1])
    assert cm.debug_check_indices(td["slot_row"], r["topk_idx"], td["offsets"], E, A_td) == cm.OK
    assert cm.debug_check_indices(ed["slot_row"], r["topk_idx"], ed["offsets"], E, A_ed, D=D) == cm.OK
    # buffers one row too short
    assert cm.debug_check_indices(td["slot_row"], r["topk_idx"], td["offsets"], E, A_td - 1) == cm.EINDEX
    # one kept pair pointed at another expert's segment
    bad = td["slot_row"].clone()
    t, s = [int(v[0]) for v in torch.nonzero(bad >= 0, as_tuple=True)]
    e = int(r["topk_idx"][t, s])
    bad[t, s] = int(td["offsets"][(e + 1) % E + 1]) - 1 if int(td["kept"][(e + 1) % E]) > 0 else A_td + 5
    assert cm.debug_check_indices(bad, r["topk_idx"], td["offsets"], E, A_td) == cm.EINDEX
    # offsets that go backwards
    off = td["offsets"].clone()
    off[3] = off[4] + 1
    assert cm.debug_check_indices(td["slot_row"], r["topk_idx"], off, E, A_td) == cm.EINDEX


def test_layer_forward_with_debug_checks(cm):
    from paper_2503_05066_b200 import synth
    cfg = synth.CONFIGS["olmoe"].with_(N=1500, d=256, F=256, E=16, k=4, D=4)
    inp = synth.make_layer_inputs(cfg)
    for mode in ("nodrop", "token_drop", "expanded_drop", "device_expanded_drop"):
        lay = cm.MoELayer(inp.x.cuda(), inp.w_router.cuda(), inp.bias.cuda(), inp.w_gate.cuda(), inp.w_up.cuda(),
                          inp.w_down.cuda(), cfg.k, cfg.D, mode, gamma=1.0, debug_checks=True)
        plain = cm.MoELayer(inp.x.cuda(), inp.w_router.cuda(), inp.bias.cuda(), inp.w_gate.cuda(), inp.w_up.cuda(),
                            inp.w_down.cuda(), cfg.k, cfg.D, mode, gamma=1.0)
        y = lay.forward()
        y0 = plain.forward()
        torch.cuda.synchronize()
        lay.check_device_status()                       # raises on CAPMOE_EINDEX / CAPMOE_ETIMEOUT
        assert torch.equal(y, y0)
