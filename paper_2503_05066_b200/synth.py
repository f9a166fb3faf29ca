"""Seeded synthetic inputs for the capacity-aware MoE layer.

This module only draws random tensors; it contains none of the method's
arithmetic (no softmax, no top-k, no capacity rule).  Both the CUDA path and
the CPU checker consume the bytes produced here, so a given (config, seed)
always denotes the same inputs on both sides.

Recipe (stand-in for trained routers and real activations, which are not
available offline):
  hidden states   X    ~ N(0, 1)
  router weights  W_r  ~ N(0, variance 1/d)   -> logits ~ N(0, 1) before bias
  expert weights       ~ N(0, std 0.02)
  router bias     b_e  : a per-expert popularity skew, by config
       "log"   : b_e = 0.5 * ln(1/(e+1))
       "zipf"  : b_e = -s * ln(e+1)
       "normal": b_e ~ N(0, std 0.5)
Expert id equals popularity rank (no shuffle), so virtual group 0 is the
hottest device.  Every tensor has its own Philox stream keyed by
(seed, tensor id, chunk id); large tensors are drawn chunk-by-chunk in a
thread pool (numpy releases the GIL while sampling).
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np
import torch

# tensor ids (second word of the Philox key)
_TID = {"x": 1, "w_router": 2, "bias": 3, "w_gate": 4, "w_up": 5, "w_down": 6,
        "ws_gate": 7, "ws_up": 8, "ws_down": 9, "perm": 10, "ties": 11}


@dataclass(frozen=True)
class LayerConfig:
    name: str
    N: int            # tokens
    d: int            # hidden size
    E: int            # routed experts
    k: int            # experts per token
    F: int            # expert FFN width
    D: int            # virtual expert-parallel groups (E % D == 0)
    dtype: str        # "f32" | "bf16"
    gammas: Tuple[float, ...] = (1.0,)
    bias_kind: str = "zipf"
    bias_s: float = 1.0
    F_shared: int = 0          # total width of the always-on shared experts (0 = none)
    straggler: bool = False    # config asks for the SM-partitioned mode
    seed: int = 0

    @property
    def m(self) -> int:
        return self.E // self.D

    def with_(self, **kw) -> "LayerConfig":
        return replace(self, **kw)


# The five workload shapes this repository measures and tests.
CONFIGS: Dict[str, LayerConfig] = {
    "tiny_f32": LayerConfig("tiny_f32", N=512, d=256, E=8, k=2, F=512, D=2, dtype="f32",
                            gammas=(1.0,), bias_kind="log"),
    "olmoe": LayerConfig("olmoe", N=4096, d=2048, E=64, k=8, F=1024, D=8, dtype="bf16",
                         gammas=(1.0, 1.5), bias_kind="zipf", bias_s=1.0),
    "mixtral": LayerConfig("mixtral", N=8192, d=4096, E=8, k=2, F=14336, D=2, dtype="bf16",
                           gammas=(1.0, 1.25), bias_kind="normal", straggler=True),
    "dsv2lite": LayerConfig("dsv2lite", N=16384, d=2048, E=64, k=6, F=1408, D=8, dtype="bf16",
                            gammas=(1.0,), bias_kind="zipf", bias_s=1.2, F_shared=2 * 1408),
    "qwen": LayerConfig("qwen", N=8192, d=2048, E=60, k=4, F=1408, D=4, dtype="bf16",
                        gammas=(0.5, 1.0, 1.5, 2.0), bias_kind="zipf", bias_s=1.0),
}
QWEN_SWEEP_N = (128, 1024, 8192, 65536)


def _rng(seed: int, tid: int, chunk: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 16) ^ tid, chunk]))


def _normal_f32(shape, std: float, seed: int, tid: int, chunk: int = 0) -> np.ndarray:
    a = _rng(seed, tid, chunk).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def _to_dtype(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(a)
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _stacked(n_chunks: int, shape, std: float, seed: int, tid: int, dtype: str,
             threads: int = 8) -> torch.Tensor:
    """[n_chunks, *shape] tensor, one Philox stream per leading index."""
    out = torch.empty((n_chunks, *shape), dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)

    def work(i):
        out[i].copy_(_to_dtype(_normal_f32(shape, std, seed, tid, i), dtype))

    if n_chunks == 1 or threads <= 1:
        for i in range(n_chunks):
            work(i)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(n_chunks)))
    return out


def router_bias(cfg: LayerConfig) -> torch.Tensor:
    e = np.arange(cfg.E, dtype=np.float64)
    if cfg.bias_kind == "log":
        b = 0.5 * np.log(1.0 / (e + 1.0))
    elif cfg.bias_kind == "zipf":
        b = -cfg.bias_s * np.log(e + 1.0)
    elif cfg.bias_kind == "normal":
        b = 0.5 * _rng(cfg.seed, _TID["bias"]).standard_normal(size=cfg.E)
    elif cfg.bias_kind == "none":
        b = np.zeros(cfg.E)
    else:
        raise ValueError(cfg.bias_kind)
    return torch.from_numpy(b.astype(np.float32))


def hidden_states(cfg: LayerConfig, N: Optional[int] = None) -> torch.Tensor:
    N = cfg.N if N is None else N
    rows = 4096
    chunks = []
    for c, r0 in enumerate(range(0, N, rows)):
        n = min(rows, N - r0)
        chunks.append(_to_dtype(_normal_f32((n, cfg.d), 1.0, cfg.seed, _TID["x"], c), cfg.dtype))
    if not chunks:
        return torch.empty((0, cfg.d), dtype=torch.bfloat16 if cfg.dtype == "bf16" else torch.float32)
    return torch.cat(chunks, 0)


def router_weights(cfg: LayerConfig) -> torch.Tensor:
    return _to_dtype(_normal_f32((cfg.E, cfg.d), 1.0 / math.sqrt(cfg.d), cfg.seed, _TID["w_router"]),
                     cfg.dtype)


def expert_weights(cfg: LayerConfig, std: float = 0.02):
    """(w_gate [E,F,d], w_up [E,F,d], w_down [E,d,F]) in the config's storage dtype."""
    wg = _stacked(cfg.E, (cfg.F, cfg.d), std, cfg.seed, _TID["w_gate"], cfg.dtype)
    wu = _stacked(cfg.E, (cfg.F, cfg.d), std, cfg.seed, _TID["w_up"], cfg.dtype)
    wd = _stacked(cfg.E, (cfg.d, cfg.F), std, cfg.seed, _TID["w_down"], cfg.dtype)
    return wg, wu, wd


def shared_expert_weights(cfg: LayerConfig, std: float = 0.02):
    """Always-on shared experts folded into one FFN of width F_shared
    (a sum of SwiGLU FFNs equals one SwiGLU FFN over the concatenated hidden units)."""
    if cfg.F_shared == 0:
        return None
    wg = _stacked(1, (cfg.F_shared, cfg.d), std, cfg.seed, _TID["ws_gate"], cfg.dtype)
    wu = _stacked(1, (cfg.F_shared, cfg.d), std, cfg.seed, _TID["ws_up"], cfg.dtype)
    wd = _stacked(1, (cfg.d, cfg.F_shared), std, cfg.seed, _TID["ws_down"], cfg.dtype)
    return wg, wu, wd


@dataclass
class LayerInputs:
    cfg: LayerConfig
    x: torch.Tensor
    w_router: torch.Tensor
    bias: torch.Tensor
    w_gate: torch.Tensor
    w_up: torch.Tensor
    w_down: torch.Tensor
    shared: Optional[tuple] = None
    extra: dict = field(default_factory=dict)


def make_layer_inputs(cfg: LayerConfig, with_experts: bool = True) -> LayerInputs:
    x = hidden_states(cfg)
    wr = router_weights(cfg)
    b = router_bias(cfg)
    if with_experts:
        wg, wu, wd = expert_weights(cfg)
        sh = shared_expert_weights(cfg)
    else:
        wg = wu = wd = None
        sh = None
    return LayerInputs(cfg, x, wr, b, wg, wu, wd, sh)


def synthetic_logits(N: int, E: int, seed: int, bias: Optional[np.ndarray] = None,
                     quantum: float = 0.0) -> np.ndarray:
    """fp32 router logits drawn directly (N(0,1) + bias), for tests of the stages
    downstream of the router.  quantum > 0 rounds them to a coarse grid so that
    equal scores (ties) occur often."""
    a = _rng(seed, _TID["ties"]).standard_normal(size=(N, E)).astype(np.float32)
    if bias is not None:
        a = a + bias.astype(np.float32)[None, :]
    if quantum > 0.0:
        a = (np.round(a / np.float32(quantum)) * np.float32(quantum)).astype(np.float32)
    return np.ascontiguousarray(a, dtype=np.float32)


def token_permutation(N: int, seed: int) -> np.ndarray:
    return _rng(seed, _TID["perm"]).permutation(N)
