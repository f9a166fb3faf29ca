"""Parity at the full workload sizes, in the launch configuration bench.py times (whole-layer
entry point, straggler emulation where the workload asks for it).  Routing, drop and
permutation outputs are compared with the CPU checker element by element over all N tokens;
the layer output on a sample of tokens the checker computes one by one, chosen so that every
128-row block of every expert's segment (every row tile of the two GEMMs) holds a checked row."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05066_b200 import synth
from tests.test_gpu_parity import _layer_case, cm, dev, host_mask  # noqa: F401  (cm is a fixture)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode,gamma,straggler", [("expanded_drop", 1.0, True), ("token_drop", 1.25, True),
                                                  ("nodrop", 1.0, False)])
def test_mixtral_shape(cm, mode, gamma, straggler):
    cfg = synth.CONFIGS["mixtral"]
    assert cm.ffn_uses_tensor_cores(cfg.d, cfg.F, torch.bfloat16)
    _layer_case(cm, cfg, mode, gamma, straggler=straggler, sample=12, cover_blocks=True)


@pytest.mark.parametrize("mode,gamma", [("nodrop", 1.0), ("token_drop", 1.0), ("expanded_drop", 1.5)])
def test_olmoe_shape(cm, mode, gamma):
    _layer_case(cm, synth.CONFIGS["olmoe"], mode, gamma, sample=48, cover_blocks=True)


@pytest.mark.parametrize("mode", ["token_drop", "expanded_drop"])
def test_dsv2lite_shape_with_shared_experts(cm, mode):
    _layer_case(cm, synth.CONFIGS["dsv2lite"], mode, 1.0, sample=48, cover_blocks=True)


@pytest.mark.parametrize("N,gamma,mode", [(128, 0.5, "token_drop"), (128, 2.0, "expanded_drop"),
                                          (1024, 1.0, "expanded_drop"), (8192, 1.5, "token_drop"),
                                          (65536, 1.0, "expanded_drop"), (65536, 2.0, "token_drop")])
def test_qwen_sweep_points(cm, N, gamma, mode):
    _layer_case(cm, synth.CONFIGS["qwen"].with_(N=N), mode, gamma, sample=32)


def test_straggler_partition_gives_identical_results(cm):
    """The SM partition only changes which CTA runs which tile: outputs are bit-identical."""
    cfg = synth.CONFIGS["olmoe"].with_(N=2048)
    a, _ = _layer_case(cm, cfg, "token_drop", 1.0, straggler=False, sample=8)
    ya = a.t["y"].clone()
    b, _ = _layer_case(cm, cfg, "token_drop", 1.0, straggler=True, sample=8)
    assert torch.equal(ya, b.t["y"])
