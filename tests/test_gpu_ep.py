"""Expert parallelism with per-rank capacity on one GPU: all R ranks of a group run on the device,
stage after stage (no kernel waits for another rank), with both ways of moving the rows - block
copies standing for the equal-split all-to-all, and the dispatch / combine kernels that store to
and load from the owners' buffers directly.  Everything integer is compared bit for bit with the
checker's ep_layer (routing per rank, the fixed row places, the counts an owner receives, its
segment bounds), the outputs within the layer tolerances."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import ep, synth
from tests.test_gpu_parity import TOL, cm, dev, host_mask  # noqa: F401  (cm is a fixture)
from tests.util import rel_err, to_np

pytestmark = pytest.mark.gpu


def _group(cm, cfg, R, n_locals, mode, gamma, transport):
    inp = synth.make_layer_inputs(cfg)
    m = cfg.E // R
    bounds = np.concatenate([[0], np.cumsum(n_locals)])
    xs = [inp.x[bounds[r]:bounds[r + 1]].contiguous() for r in range(R)]
    wr, b = dev(inp.w_router), dev(inp.bias)
    wg, wu, wd = dev(inp.w_gate), dev(inp.w_up), dev(inp.w_down)
    caps = [n if mode == "nodrop" else cm.capacity(n, cfg.E, cfg.k, gamma) for n in n_locals]
    ranks = [ep.EPRank(r, R, dev(xs[r]), wr, b, wg[r * m:(r + 1) * m].contiguous(), wu[r * m:(r + 1) * m].contiguous(),
                       wd[r * m:(r + 1) * m].contiguous(), cfg.k, mode, gamma, C_buf=max(caps)) for r in range(R)]
    return inp, xs, ranks, ep.EPGroupOnOneDevice(ranks, transport)


CASES = [
    # config overrides, R, tokens per rank
    (dict(N=384, d=64, E=8, k=2, F=48, dtype="f32"), 2, [192, 192]),
    (dict(N=600, d=96, E=12, k=3, F=40, dtype="f32"), 4, [100, 250, 50, 200]),       # unequal ranks: one stride for all
    (dict(N=2048, d=256, E=16, k=4, F=256, dtype="bf16"), 4, [512, 512, 512, 512]),  # tensor-core segments
    (dict(N=3000, d=128, E=64, k=8, F=192, dtype="bf16"), 8, [375] * 8),
    (dict(N=700, d=128, E=8, k=2, F=128, dtype="bf16"), 1, [700]),                   # one rank: the ordinary layer
]


@pytest.mark.parametrize("transport", ["collective", "peer"])
@pytest.mark.parametrize("mode,gamma", [("token_drop", 1.0), ("expanded_drop", 1.0), ("token_drop", 0.5), ("nodrop", 1.0)])
@pytest.mark.parametrize("over,R,n_locals", CASES)
def test_ep_group_matches_oracle(cm, over, R, n_locals, mode, gamma, transport):
    cfg = synth.CONFIGS["tiny_f32"].with_(D=R, **over)
    inp, xs, ranks, group = _group(cm, cfg, R, n_locals, mode, gamma, transport)
    ys = group.forward()
    torch.cuda.synchronize()
    for rk in ranks:
        rk.check()
    w = [to_np(t) for t in (inp.w_router, inp.w_gate, inp.w_up, inp.w_down)]
    ref = oracle.ep_layer([to_np(x) for x in xs], w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, gamma, mode,
                          cfg.dtype, logits_ranks=[rk.r["logits"].cpu().numpy() for rk in ranks])
    m, C = cfg.E // R, ranks[0].C
    for r, rk in enumerate(ranks):
        o = ref["ranks"][r]
        assert rk.C_local == o["C"]
        assert np.array_equal(host_mask(rk.dr["keep_mask"]), o["keep_mask"])
        assert np.array_equal(rk.dr["kept"].cpu().numpy(), o["kept"])
        assert np.array_equal(rk.dr["slot_row"].cpu().numpy(), o["slot_row"])
        # the fixed place of every kept row: expert * C + rank inside the expert's kept list
        sr, off = o["slot_row"], o["offsets"]
        want = np.full_like(sr, -1)
        for row in range(o["A"]):
            e = int(o["perm_expert"][row])
            t = int(o["perm_token"][row])
            want[t][sr[t] == row] = e * C + (row - off[e])
        assert np.array_equal(rk.slot_row_ep.cpu().numpy(), want)
        # what this rank receives as an owner: counts per (source, local expert), and the segments
        cnt = ref["send_counts"][:, r, :].reshape(-1)
        assert np.array_equal(rk.cnt_recv.cpu().numpy(), cnt)
        assert np.array_equal(rk.seg_begin.cpu().numpy(), np.arange(R * m) * C)
        assert np.array_equal(rk.seg_end.cpu().numpy(), np.arange(R * m) * C + cnt)
        assert rel_err(ys[r].double().cpu().numpy(), ref["y"][r]) <= TOL[cfg.dtype]


def test_ep_transports_agree_bit_for_bit(cm):
    cfg = synth.CONFIGS["tiny_f32"].with_(N=2048, d=256, E=16, k=4, F=256, dtype="bf16", D=4)
    outs = []
    for transport in ("collective", "peer"):
        _, _, ranks, group = _group(cm, cfg, 4, [512] * 4, "expanded_drop", 1.0, transport)
        outs.append([y.clone() for y in group.forward()])
    torch.cuda.synchronize()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_ep_plan_flags_a_capacity_that_is_too_small(cm):
    lg = synth.synthetic_logits(500, 8, 4)
    r = cm.route(None, None, None, 2, logits_in=dev(lg))
    dr = cm.token_drop(r["topk_score"], r["topk_idx"], 8, 200)
    _, bad = cm.ep_plan(dr["slot_row"], r["topk_idx"], dr["offsets"], 8, 200)
    assert int(bad.item()) == 0
    _, bad = cm.ep_plan(dr["slot_row"], r["topk_idx"], dr["offsets"], 8, int(dr["kept"].max().item()) - 1)
    assert int(bad.item()) == 1
