"""Pins of the checker's expert-parallel layer (oracle.ep_layer): the same result as R separate
single-rank layers whose tokens are all at home on that rank, R = 1 is the ordinary layer, every
message respects the bound the per-rank capacity gives, and nothing a rank computes depends on
another rank's tokens."""
import numpy as np
import pytest

import oracle
from paper_2503_05066_b200 import synth
from tests.util import to_np


def _inputs(R, N_local, d=64, E=8, k=2, F=48, dtype="f32", seed=0):
    cfg = synth.CONFIGS["tiny_f32"].with_(N=N_local * R, d=d, E=E, k=k, F=F, D=R, dtype=dtype, seed=seed)
    inp = synth.make_layer_inputs(cfg)
    x = to_np(inp.x)
    xs = [np.ascontiguousarray(x[r * N_local:(r + 1) * N_local]) for r in range(R)]
    return cfg, inp, xs


@pytest.mark.parametrize("mode", ["nodrop", "token_drop", "expanded_drop"])
@pytest.mark.parametrize("R,gamma", [(2, 1.0), (4, 0.5), (4, 1.5)])
def test_ep_layer_equals_one_layer_per_rank(mode, R, gamma):
    cfg, inp, xs = _inputs(R, 96)
    w = [to_np(t) for t in (inp.w_router, inp.w_gate, inp.w_up, inp.w_down)]
    got = oracle.ep_layer(xs, w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, gamma, mode, cfg.dtype)
    for r in range(R):
        tg = np.full((96,), r, np.int32)
        ref = oracle.layer_forward(xs[r], w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, gamma, R, mode, cfg.dtype,
                                   token_group=tg)
        # the single-rank layer holds all E experts: a different program (no messages, no weight
        # slices) that must give the same numbers, since E_i(x) acts on each row by itself
        assert np.array_equal(got["ranks"][r]["keep_mask"], ref["keep_mask"])
        assert np.array_equal(got["ranks"][r]["slot_row"], ref["slot_row"])
        assert np.array_equal(got["y"][r], ref["y"])


@pytest.mark.parametrize("mode", ["token_drop", "expanded_drop"])
def test_one_rank_is_the_ordinary_layer(mode):
    cfg, inp, xs = _inputs(1, 128)
    w = [to_np(t) for t in (inp.w_router, inp.w_gate, inp.w_up, inp.w_down)]
    got = oracle.ep_layer(xs, w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, 1.0, mode, cfg.dtype)
    ref = oracle.layer_forward(xs[0], w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, 1.0, 1, mode, cfg.dtype)
    assert np.array_equal(got["y"][0], ref["y"])
    assert got["send_counts"].shape == (1, 1, cfg.E)


def test_messages_respect_the_capacity_bound_and_ranks_are_independent():
    R, N_local = 4, 80
    cfg, inp, xs = _inputs(R, N_local, E=16, k=4)
    w = [to_np(t) for t in (inp.w_router, inp.w_gate, inp.w_up, inp.w_down)]
    for mode in ("token_drop", "expanded_drop"):
        got = oracle.ep_layer(xs, w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, 1.0, mode, cfg.dtype)
        C = oracle.capacity(N_local, cfg.E, cfg.k, 1.0)
        sc = got["send_counts"]                       # [source, owner, local expert]
        assert sc.max() <= C                          # at most C_local rows per (source, expert)
        assert sc.sum(axis=2).max() <= got["m"] * C   # hence at most m * C_local rows per message
        for r in range(R):
            assert sc[r].sum() == got["ranks"][r]["A"]
            if mode == "expanded_drop":
                # N_local >= C: the experts a rank owns are filled to the brim by its own tokens
                assert np.all(sc[r, r] == C)
        # changing rank 3's tokens leaves what ranks 0..2 compute untouched (no load information
        # crosses ranks: the capacity is local)
        xs2 = list(xs)
        xs2[3] = np.ascontiguousarray(xs[3][::-1])
        got2 = oracle.ep_layer(xs2, w[0], inp.bias.numpy(), w[1], w[2], w[3], cfg.k, 1.0, mode, cfg.dtype)
        for r in range(3):
            assert np.array_equal(got["y"][r], got2["y"][r])
