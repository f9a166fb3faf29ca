"""Seeded random shapes through the routing stages on the GPU against the CPU checker, bit for bit:
sizes that are not multiples of any tile, chunk or warp size, every number of experts from 2 to
130, both selection paths (one CTA per expert below 16384 tokens, token-parallel above) and both
capacity levels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.test_gpu_parity import ROUTER_TOL, bias_for, cm, dev, host_mask  # noqa: F401
from tests.util import rel_err, to_np

pytestmark = pytest.mark.gpu


def _cases(n, seed, big):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        D = int(rng.choice([1, 2, 3, 4, 5, 8]))
        m = int(rng.integers(1, 17))
        E = D * m
        if E < 2 or E > 130:
            continue
        k = int(rng.integers(1, min(E, 8) + 1))
        N = int(rng.integers(16384, 40000)) if big else int(rng.integers(1, 6000))
        gamma = float(rng.choice([0.25, 0.5, 1.0, 1.0, 1.5, 3.0]))
        q = float(rng.choice([0.0, 0.0, 0.25, 1.0]))
        out.append((N, E, k, D, gamma, q))
    return out


CASES = _cases(28, 2024, False) + _cases(8, 2025, True)


@pytest.mark.parametrize("N,E,k,D,gamma,q", CASES)
def test_drops_on_random_shapes(cm, N, E, k, D, gamma, q):
    lg = synth.synthetic_logits(N, E, 1000 + N, bias=bias_for(E, 0.8), quantum=q)
    r = cm.route(None, None, None, k, logits_in=dev(lg))
    scores, idx = r["scores"].cpu().numpy(), r["topk_idx"].cpu().numpy()
    assert np.array_equal(scores.view(np.uint32), oracle.softmax(lg).view(np.uint32))
    C = cm.capacity(N, E, k, gamma)
    got, ref = cm.token_drop(r["topk_score"], r["topk_idx"], E, C), oracle.token_drop(scores, idx, C)
    for key in ("kept", "offsets", "slot_row"):
        assert np.array_equal(got[key].cpu().numpy(), ref[key]), ("token", key)
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    got, ref = cm.expanded_drop(r["scores"], r["topk_idx"], C, D), oracle.expanded_drop(scores, idx, C, D)
    for key in ("cand", "kept", "offsets", "slot_row"):
        assert np.array_equal(got[key].cpu().numpy(), ref[key]), ("expanded", key)
    assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])
    Cd = cm.device_capacity(N, E, k, D, gamma)
    for expanded in (False, True):
        got = cm.device_drop(r["scores"], r["topk_idx"], Cd, D, expanded)
        ref = oracle.device_drop(scores, idx, Cd, D, expanded)
        for key in ("cand", "kept", "offsets", "slot_row"):
            assert np.array_equal(got[key].cpu().numpy(), ref[key]), ("device", expanded, key)
        assert np.array_equal(host_mask(got["keep_mask"]), ref["keep_mask"])


def _router_cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        E = int(rng.integers(2, 131))
        k = int(rng.integers(1, min(E, 16) + 1))
        d = 64 * int(rng.integers(1, 9))
        N = int(rng.integers(1, 9000))
        out.append((N, d, E, k))
    return out


@pytest.mark.parametrize("N,d,E,k", _router_cases(16, 7))
def test_router_on_random_shapes(cm, N, d, E, k):
    g = torch.Generator().manual_seed(N * 131 + E)
    x = torch.randn((N, d), generator=g).to(torch.bfloat16)
    w = (torch.randn((E, d), generator=g) * (2.0 / d ** 0.5)).to(torch.bfloat16)
    b = torch.randn((E,), generator=g) * 0.5
    out = cm.route(dev(x), dev(w), dev(b), k)
    torch.cuda.synchronize()
    got_logits = out["logits"].cpu().numpy()
    ref_logits = oracle.router_logits(to_np(x), to_np(w), b.numpy(), "bf16")
    assert rel_err(got_logits.astype(np.float64), ref_logits.astype(np.float64)) <= ROUTER_TOL["bf16"]
    s_ref = oracle.softmax(got_logits)
    assert np.array_equal(out["scores"].cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    idx, val, load = oracle.topk(s_ref, k)
    assert np.array_equal(out["topk_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["topk_score"].cpu().numpy().view(np.uint32), val.view(np.uint32))
    assert np.array_equal(out["load"].cpu().numpy(), load)


def _ffn_cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        E = int(rng.integers(1, 9))
        d = 64 * int(rng.integers(1, 7))
        F = 64 * int(rng.integers(1, 7))
        style = i % 4
        if style == 0:      # ragged, some experts empty
            rows = [int(rng.choice([0, 1, 17, 127, 128, 129, 300, 511])) for _ in range(E)]
        elif style == 1:    # long segments: CTA pairs
            rows = [int(rng.integers(1024, 1400)) for _ in range(E)]
        elif style == 2:    # multiples of 256: CTA pairs with exact tiles
            rows = [256 * int(rng.integers(1, 4)) for _ in range(E)]
        else:               # one expert holds nearly everything
            rows = [int(rng.integers(0, 40)) for _ in range(E)]
            rows[int(rng.integers(0, E))] = int(rng.integers(1500, 2500))
        D = int(rng.choice([0, 0, 1, E])) if style != 0 else 0
        out.append((E, d, F, tuple(rows), D))
    return out


# CTA-pair kernel with an expert width that is an odd multiple of 64 (the last 128-column block of
# the gate/up GEMM is half filled), with and without straggler emulation
_FFN_ODD_WIDTH = [(4, 128, 192, (1100, 1200, 1300, 1025), 0), (3, 64, 320, (256, 512, 768), 3),
                  (2, 192, 64, (1500, 30), 0), (2, 128, 448, (1024, 1024), 2)]


@pytest.mark.parametrize("E,d,F,rows,D_straggler", _ffn_cases(16, 99) + _FFN_ODD_WIDTH)
def test_grouped_ffn_on_random_segments(cm, E, d, F, rows, D_straggler):
    """bf16 tensor-core FFN over random expert segments against the double-precision SwiGLU of the
    CPU checker on sampled rows; rows past the last segment stay untouched."""
    A = int(sum(rows))
    A_max = A + 5
    g = torch.Generator().manual_seed(E * 1000 + d + F + A)
    x_perm = torch.randn((A_max, d), generator=g).to(torch.bfloat16)
    wg = (torch.randn((E, F, d), generator=g) * 0.05).to(torch.bfloat16)
    wu = (torch.randn((E, F, d), generator=g) * 0.05).to(torch.bfloat16)
    wd = (torch.randn((E, d, F), generator=g) * 0.05).to(torch.bfloat16)
    offsets = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
    y = torch.full((A_max, d), 7.0, dtype=torch.bfloat16).cuda()
    out = cm.grouped_ffn(dev(x_perm), dev(offsets), dev(wg), dev(wu), dev(wd), D_straggler=D_straggler, y_perm=y)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    assert (got[A:] == 7.0).all()                               # never written
    if A == 0:
        return
    rng = np.random.default_rng(A)
    sample = np.unique(np.concatenate([rng.integers(0, A, size=min(A, 96)), offsets[:-1][np.array(rows) > 0],
                                       offsets[1:][np.array(rows) > 0] - 1]))
    row_expert = (np.searchsorted(offsets, sample, side="right") - 1).astype(np.int32)
    ref = oracle.expert_ffn(np.ascontiguousarray(to_np(x_perm)[sample]), row_expert, to_np(wg), to_np(wu), to_np(wd),
                            "bf16")
    assert rel_err(got[sample], ref) <= 2e-2


# Every tensor-core FFN kernel on the same segments: short and ragged ones (token counts around the
# short-segment kernel's steps of 16 and its 256-token tiles), long ones, empty ones, widths that are
# odd multiples of 64, with and without the straggler partition.
_FFN_VARIANT_CASES = [
    (6, 128, 256, (0, 1, 15, 16, 17, 255), 0),
    (5, 192, 192, (256, 257, 300, 512, 513), 0),
    (4, 64, 320, (31, 33, 700, 1), 2),
    (3, 256, 448, (1030, 129, 270), 3),
    (8, 128, 128, (40, 0, 0, 90, 272, 16, 48, 600), 4),
]


@pytest.mark.parametrize("variant", ["pair", "single", "short", "short_down", "auto"])
@pytest.mark.parametrize("E,d,F,rows,D_straggler", _FFN_VARIANT_CASES)
def test_every_ffn_kernel_on_the_same_segments(cm, variant, E, d, F, rows, D_straggler):
    A = int(sum(rows))
    A_max = A + 40                                               # rows a last tile may read but never write
    g = torch.Generator().manual_seed(E * 77 + d + F + A)
    x_perm = torch.randn((A_max, d), generator=g).to(torch.bfloat16)
    x_perm[A:] = float("nan")                                    # what lies past the last segment must not leak in
    wg = (torch.randn((E, F, d), generator=g) * 0.05).to(torch.bfloat16)
    wu = (torch.randn((E, F, d), generator=g) * 0.05).to(torch.bfloat16)
    wd = (torch.randn((E, d, F), generator=g) * 0.05).to(torch.bfloat16)
    offsets = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
    y = torch.full((A_max, d), 7.0, dtype=torch.bfloat16).cuda()
    st = torch.zeros((cm.FFN_STATUS_WORDS,), dtype=torch.int32).cuda()
    cm.debug_ffn_variant(variant)
    try:
        out = cm.grouped_ffn(dev(x_perm), dev(offsets), dev(wg), dev(wu), dev(wd), D_straggler=D_straggler, y_perm=y,
                             dev_status=st)
        torch.cuda.synchronize()
    finally:
        cm.debug_ffn_variant("auto")
    assert int(st[0].item()) == cm.OK
    got = out.float().cpu().numpy().astype(np.float64)
    assert (got[A:] == 7.0).all()                               # never written
    assert np.isfinite(got[:A]).all()
    rng = np.random.default_rng(A)
    nz = np.array(rows) > 0
    edges = np.concatenate([offsets[:-1][nz], offsets[1:][nz] - 1])
    steps = np.concatenate([np.arange(offsets[e], offsets[e + 1], 16) for e in range(E)] + [np.zeros(0, np.int64)])
    sample = np.unique(np.concatenate([rng.integers(0, A, size=64), edges, steps, np.minimum(steps + 15, A - 1)])).astype(np.int64)
    row_expert = (np.searchsorted(offsets, sample, side="right") - 1).astype(np.int32)
    ref = oracle.expert_ffn(np.ascontiguousarray(to_np(x_perm)[sample]), row_expert, to_np(wg), to_np(wu), to_np(wd),
                            "bf16")
    assert rel_err(got[sample], ref) <= 2e-2
    # all kernels accumulate over K in the same order: the same bits
    if variant != "single":
        cm.debug_ffn_variant("single")
        try:
            y2 = torch.full((A_max, d), 7.0, dtype=torch.bfloat16).cuda()
            ref_k = cm.grouped_ffn(dev(x_perm), dev(offsets), dev(wg), dev(wu), dev(wd), D_straggler=D_straggler, y_perm=y2)
            torch.cuda.synchronize()
        finally:
            cm.debug_ffn_variant("auto")
        assert torch.equal(out[:A].view(torch.int16), ref_k[:A].view(torch.int16))


def _layer_cases(n, seed):
    """Random whole-layer configurations: token counts that leave ragged tiles, expert counts that
    are not powers of two, every drop mode, with and without shared experts and the straggler
    partition; bf16 shapes on the tensor-core kernels and fp32 shapes on the FMA kernel."""
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        bf16 = i % 3 != 2
        D = int(rng.choice([1, 2, 3, 4]))
        m = int(rng.integers(1, 6))
        E = D * m
        k = int(rng.integers(1, min(E, 6) + 1))
        N = int(rng.choice([1, 63, 200, 777, 1500, 2304]))
        if bf16:
            d, F = 64 * int(rng.integers(1, 5)), 64 * int(rng.integers(1, 6))
        else:
            d, F = int(rng.integers(3, 40)) * 4, int(rng.integers(5, 90))
        mode = ["nodrop", "token_drop", "expanded_drop"][int(rng.integers(0, 3))]
        gamma = float(rng.choice([0.5, 1.0, 1.3, 2.0]))
        F_shared = int(rng.choice([0, 0, 64 * int(rng.integers(1, 4)) if bf16 else int(rng.integers(4, 50))]))
        straggler = bool(bf16 and rng.integers(0, 3) == 0)
        out.append((N, d, E, k, F, D, "bf16" if bf16 else "f32", mode, gamma, F_shared, straggler, 100 + i))
    return out


@pytest.mark.parametrize("N,d,E,k,F,D,dtype,mode,gamma,F_shared,straggler,seed", _layer_cases(24, 2024) + _layer_cases(24, 7))
def test_layer_on_random_configurations(cm, N, d, E, k, F, D, dtype, mode, gamma, F_shared, straggler, seed):
    from tests.test_gpu_parity import _layer_case
    cfg = synth.LayerConfig("random", N=N, d=d, E=E, k=k, F=F, D=D, dtype=dtype, gammas=(gamma,), bias_kind="zipf",
                            bias_s=0.7, F_shared=F_shared, seed=seed)
    _layer_case(cm, cfg, mode, gamma, straggler=straggler, std=0.05)
