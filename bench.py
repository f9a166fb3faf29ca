#!/usr/bin/env python
"""Benchmark of the capacity-aware MoE layer forward (one step = one layer forward over one
batch of synthetic tokens: route -> drop -> permute -> grouped SwiGLU FFN -> combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config mixtral] [--mode expanded_drop]
                    [--gamma 1.0] [--no-straggler] [--no-sweep] [--impl reference]

Prints ONE JSON line.  `value` is tokens/s of the whole job with the inputs resident in HBM;
`e2e` is the same metric through the host-buffer entry point (pinned host activations copied
in and out inside the timed region); `roofline` is for the dominant kernel (the gate/up
tcgen05 GEMM with the SwiGLU epilogue); `cpu_baseline` is the CPU checker timed on a bounded
sample of the same workload; `modes` lists the other routing modes of the same workload
(no-drop, Token Drop, Expanded Drop, with and without straggler emulation); `configs` the other
workload shapes (tiny, OLMoE, DeepSeek-V2-Lite, Qwen at 128 and 8192 tokens) in the three modes.
With --impl reference the CPU checker itself is the timed program.
With N > 1 each rank runs the same per-GPU workload (weak scaling, no collective on the data
path); times are device times, max over ranks.  `python bench.py --gpus N` starts the N ranks
itself; under torchrun it is one of them.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MoE-layer tokens/s at Mixtral shape"
UNIT = "tokens/s"

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the two FFN GEMM
# kernels, from a one-pass ncu capture.  A capture describes one build of the kernel: it is keyed
# by the SHA-256 of the kernel's source files (concatenated) at the time of the capture, and is
# reported only while they still have that hash (else `traffic` is null and says why).
# key = (config, N, F, mode, gamma, straggler) -> {"gate_up": bytes, "down": bytes}
NCU_TRAFFIC = {
    "kernel_sources": ["paper_2503_05066_b200/csrc/ffn_tc.cu", "paper_2503_05066_b200/csrc/tc_common.cuh"],
    "sha256": "50320e18dc87454ff7b6bb78d56bdd910562c4331286dba03e2abdceefe292fe",
    "captures": {
        # ncu --metrics gpu__time_duration.sum,dram__bytes_read.sum,dram__bytes_write.sum (one pass),
        # means of nine launches each of the two GEMM kernels
        ("mixtral", 8192, 14336, "expanded_drop", 1.0, True): {"gate_up": 2591500000 + 460600000,
                                                                "down": 3039100000 + 126300000},
    },
}


def _recorded_traffic(key):
    """(gate_up_bytes, down_bytes, note) for this workload from the recorded ncu capture, or
    (None, None, reason)."""
    import hashlib
    try:
        digest = hashlib.sha256(b"".join(open(os.path.join(ROOT, f), "rb").read()
                                         for f in NCU_TRAFFIC["kernel_sources"])).hexdigest()
    except OSError:
        return None, None, "kernel source not found"
    if NCU_TRAFFIC["sha256"] is None:
        return None, None, "no ncu capture recorded for this build of the kernel"
    if digest != NCU_TRAFFIC["sha256"]:
        return None, None, "the kernel source changed after the recorded ncu capture"
    cap = NCU_TRAFFIC["captures"].get(key)
    if cap is None:
        return None, None, "this workload was not captured"
    return cap.get("gate_up"), cap.get("down"), "recorded one-pass ncu capture of this kernel build (not measured in this run)"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 100 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.rows = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # "under load": the upper half of the power samples
        cut = statistics.median(power)
        loaded = [s for s, p in zip(sm, power) if p >= cut] or sm
        return {"sm_mhz": statistics.median(loaded), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def _to_np(t):
    import numpy as np
    import torch
    t = t.detach().cpu().contiguous()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def cpu_oracle_run(cfg, inp, mode: str, gamma: float, budget_tokens: int):
    """The CPU checker on a bounded sample: routing and the drop over all N tokens, the expert FFN
    and the combine for `budget_tokens` tokens spread over the batch.  Returns (tokens/s, detail)."""
    import numpy as np
    import oracle
    x, wr, b = _to_np(inp.x), _to_np(inp.w_router), inp.bias.numpy()
    t0 = time.perf_counter()
    logits = oracle.router_logits(x, wr, b, cfg.dtype)
    scores = oracle.softmax(logits)
    idx, _, load = oracle.topk(scores, cfg.k)
    C = cfg.N if mode == "nodrop" else oracle.capacity(cfg.N, cfg.E, cfg.k, gamma)
    if mode.startswith("device_"):
        expanded = mode == "device_expanded_drop"
        r = oracle.device_drop(scores, idx, oracle.device_capacity(cfg.N, cfg.E, cfg.k, cfg.D, gamma), cfg.D, expanded)
        Dp = cfg.D if expanded else 0
    elif mode == "expanded_drop":
        r = oracle.expanded_drop(scores, idx, C, cfg.D)
        Dp = cfg.D
    else:
        r = oracle.token_drop(scores, idx, C)
        Dp = 0
    t_route = time.perf_counter() - t0
    toks = np.linspace(0, cfg.N - 1, budget_tokens).astype(np.int32)
    t1 = time.perf_counter()
    oracle.layer_tokens(x, toks, scores, idx, r["slot_row"], Dp, _to_np(inp.w_gate), _to_np(inp.w_up),
                        _to_np(inp.w_down), cfg.dtype)
    t_ffn = time.perf_counter() - t1
    per_token = t_route / cfg.N + t_ffn / budget_tokens
    return 1.0 / per_token, dict(route_drop_s_full_N=t_route, ffn_combine_s_sample=t_ffn,
                                 sample_tokens=int(budget_tokens), cores=oracle.num_threads())


def run_reference(args, rank):
    """--impl reference: the CPU checker as it stands, on the host cores."""
    from paper_2503_05066_b200 import synth
    if rank != 0:
        return
    cfg = _pick_config(args)
    inp = synth.make_layer_inputs(cfg)
    if os.environ.get("TORCHELASTIC_RUN_ID") and os.environ.get("OMP_NUM_THREADS") == "1":
        # torchrun pins every rank to one OpenMP thread; this arm runs on rank 0 alone and is meant
        # to use the machine's host cores, as it does when started without the launcher
        try:
            import ctypes
            ctypes.CDLL("libgomp.so.1").omp_set_num_threads(os.cpu_count() or 1)
        except OSError:
            pass
    sample = args.ref_tokens or 64
    vals, walls = [], []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        v, detail = cpu_oracle_run(cfg, inp, args.mode, args.gamma, sample)
        if i >= args.warmup:
            vals.append(v)
            walls.append(time.perf_counter() - t0)
    v = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        # what one step of this arm really ran: routing and drop on all tokens, the FFN on the sample
        "ms_per_step": 1e3 * statistics.mean(walls),
        # `value` scales the sampled FFN time to all tokens: it is an extrapolation, not a timed full step
        "extrapolated": True, "ms_per_step_full_workload_extrapolated": 1e3 * cfg.N / v,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config_dict(cfg, args),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": detail["cores"], "kind": "oracle",
                         "sample": f"router+drop on all {cfg.N} tokens, expert FFN+combine on {sample} tokens "
                                   "spread over the batch; per-token times added"},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_table(args):
    """Latency, load statistics and drop rate per (N, gamma, mode) point: device time per layer over
    `steps` forwards after `warmup`, one JSON line per point."""
    import torch
    from paper_2503_05066_b200 import capmoe, synth
    base = _pick_config(args)
    Ns = synth.QWEN_SWEEP_N if (base.name == "qwen" and args.N is None) else (base.N,)
    steps, warmup = max(3, min(args.steps, 30)), max(3, min(args.warmup, 5))
    md_head = False
    for N in Ns:
        cfg = base.with_(N=N)
        inp = synth.make_layer_inputs(cfg)
        g = {k: getattr(inp, k).cuda() for k in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}
        shared = None if inp.shared is None else tuple(s.cuda() for s in inp.shared)
        nodrop_ms = {}
        points = [("nodrop", None, "", {})] + [(m, gm, "", {}) for gm in cfg.gammas
                                               for m in ("token_drop", "expanded_drop", "device_token_drop",
                                                         "device_expanded_drop")]
        # variants of the drop at the first capacity factor
        g0 = cfg.gammas[0]
        points += [("token_drop", g0, "+random", dict(metric="random", seed=1)),
                   ("expanded_drop", g0, "+topk_first", dict(topk_first=True)),
                   ("expanded_drop", g0, "+max_k", dict(max_experts=cfg.k))]
        for mode, gamma, tag, variant in points:
            for strag in ([False, True] if cfg.straggler else [False]):
                lay = capmoe.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k,
                                      cfg.D, mode, gamma=1.0 if gamma is None else gamma, straggler=strag,
                                      shared=shared, **variant)
                ms = time_layer(lay, steps, warmup, torch)
                graph_ms = time_graph(lay, steps, torch)
                if mode == "nodrop":
                    nodrop_ms[strag] = ms
                load = lay.t["load"].cpu().numpy()
                kept = lay.t["kept"].cpu().numpy()
                A = int(lay.t["expert_offsets"][-1].item())
                nbar = N * cfg.k / cfg.E
                m = cfg.E // cfg.D
                row = {
                    "config": cfg.name, "N": N, "mode": mode + tag, "gamma": gamma, "straggler_emulation": strag,
                    "C": int(lay.C), "ms_per_layer": ms, "ms_per_layer_graph": graph_ms, "tokens_per_s": N / (ms * 1e-3),
                    "speedup_vs_nodrop": nodrop_ms[strag] / ms,
                    "max_load_over_mean": float(load.max() / nbar), "max_kept_over_mean": float(kept.max() / nbar),
                    "max_device_kept_over_mean": float(kept.reshape(cfg.D, m).sum(1).max() / (nbar * m)),
                    "A": A, "kept_over_Nk": A / (N * cfg.k),
                    "dropped_fraction_of_topk": float(1.0 - min(A, N * cfg.k) / (N * cfg.k)) if "expanded" not in mode
                    else None}
                if args.markdown:
                    if not md_head:
                        md_head = True
                        print("| N | mode | γ | strag | C | A | A/(N·k) | max load | max kept | max dev | ms/layer | as one graph "
                              "| tokens/s | speedup |\n|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
                    print("| %d | %s | %s | %s | %d | %d | %.2f | %.2f | %.2f | %.2f | %.3f | %.3f | %.2e | %.2f |" % (
                        N, mode + tag, "∞" if gamma is None else gamma, "on" if strag else "off", row["C"], A,
                        row["kept_over_Nk"], row["max_load_over_mean"], row["max_kept_over_mean"],
                        row["max_device_kept_over_mean"], ms, graph_ms, row["tokens_per_s"], row["speedup_vs_nodrop"]),
                        flush=True)
                else:
                    print(json.dumps(row), flush=True)
                del lay
        del g, inp


def run_ep(args):
    """--ep R: the layer under expert parallelism with per-rank capacity, R ranks with N/R tokens and
    E/R experts each, every rank's stages timed ALONE on this one GPU (as if it had a B200 to itself).
    What a rank's owner FFN takes depends on the rows the other ranks send it, so the slowest owner is
    the straggler of the paper's latency model (Eq. 4); the layer time under expert parallelism is
    estimated as the sum over the stages of the slowest rank's time.  The exchange itself is not timed
    (one GPU): this is a measurement of the per-rank work, not a multi-GPU number.  One JSON line per mode."""
    import torch
    from paper_2503_05066_b200 import capmoe, ep, synth
    cfg = _pick_config(args)
    R = args.ep
    assert cfg.E % R == 0 and cfg.N % R == 0
    n_local, m = cfg.N // R, cfg.E // R
    inp = synth.make_layer_inputs(cfg)
    wr, b = inp.w_router.cuda(), inp.bias.cuda()
    wg, wu, wd = inp.w_gate.cuda(), inp.w_up.cuda(), inp.w_down.cuda()
    xs = [inp.x[r * n_local:(r + 1) * n_local].cuda().contiguous() for r in range(R)]
    steps = max(3, min(args.steps, 20))

    def med(fn):
        ts = []
        for i in range(steps + 2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if i >= 2:
                ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)

    base = None
    for mode, gam in [("nodrop", None)] + [(mo, g_) for g_ in cfg.gammas for mo in ("token_drop", "expanded_drop")]:
        ranks = [ep.EPRank(r, R, xs[r], wr, b, wg[r * m:(r + 1) * m], wu[r * m:(r + 1) * m], wd[r * m:(r + 1) * m],
                           cfg.k, mode, 1.0 if gam is None else gam) for r in range(R)]
        group = ep.EPGroupOnOneDevice(ranks, "peer")
        group.forward()
        torch.cuda.synchronize()
        for rk in ranks:
            rk.check()
        t_disp = [med(rk.dispatch) for rk in ranks]
        t_ffn = [med(rk.expert_ffn) for rk in ranks]
        t_comb = [med(rk.combine) for rk in ranks]
        rows = [int(rk.cnt_recv.sum().item()) for rk in ranks]
        layer_ms = max(t_disp) + max(t_ffn) + max(t_comb)
        if mode == "nodrop":
            base = layer_ms
        print(json.dumps({
            "workload": f"{cfg.name}: N={cfg.N} d={cfg.d} E={cfg.E} k={cfg.k} F={cfg.F} {cfg.dtype}, {R} ranks x {n_local} tokens, "
                        f"{m} expert(s) per rank", "mode": mode, "gamma": gam, "C_local": ranks[0].C_local,
            "rows_received_per_owner": rows, "max_over_mean_rows": max(rows) / (sum(rows) / R) if sum(rows) else None,
            "owner_ffn_ms": t_ffn, "route_drop_dispatch_ms_max": max(t_disp),
            "combine_ms_max": max(t_comb), "ep_layer_ms_slowest_rank_per_stage": layer_ms,
            "tokens_per_s_all_ranks": cfg.N / (layer_ms * 1e-3), "speedup_vs_nodrop": base / layer_ms,
            "note": "each rank timed alone on one GPU; exchange not timed; not a multi-GPU measurement"}), flush=True)
        del group, ranks
        torch.cuda.empty_cache()


def _pick_config(args):
    from paper_2503_05066_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.N is not None:
        cfg = cfg.with_(N=args.N)
    if args.F is not None:
        cfg = cfg.with_(F=args.F)
    if args.D is not None:
        cfg = cfg.with_(D=args.D)
    return cfg


def _config_dict(cfg, args):
    return {"workload": f"{cfg.name}: N={cfg.N} d={cfg.d} E={cfg.E} k={cfg.k} F={cfg.F} D={cfg.D} {cfg.dtype}",
            "mode": args.mode, "gamma": args.gamma, "straggler_emulation": bool(args.straggler),
            "l2": "expert weights (%.2f GB) are larger than L2, no flush needed" %
                  (3 * cfg.E * cfg.d * cfg.F * (2 if cfg.dtype == "bf16" else 4) / 1e9),
            "inputs": "hidden N(0,1); router N(0,1/d) + per-expert bias (%s); experts N(0,0.02); seed %d"
                      % (cfg.bias_kind, cfg.seed)}


def time_layer(layer, steps, warmup, torch, events=None):
    """ms per step (device time, CUDA events on the launching stream)."""
    for _ in range(warmup):
        layer.forward()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        if events is not None:
            layer.set_stage_events(events[i])
        layer.forward()
    e1.record()
    torch.cuda.synchronize()
    layer.set_stage_events(None)
    layer.check_device_status()
    return e0.elapsed_time(e1) / steps


def time_graph(layer, steps, torch):
    """ms per step when the whole layer is replayed as one CUDA graph (no per-kernel launch cost on the host)."""
    layer.capture_graph()
    for _ in range(3):
        layer.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        layer.replay()
    e1.record()
    torch.cuda.synchronize()
    layer.check_device_status()
    return e0.elapsed_time(e1) / steps


def spawn_ranks(n: int, argv) -> int:
    """Re-runs this script as n ranks on this node (torch.distributed.run, rendezvous on 127.0.0.1),
    the way the N > 1 benchmark is meant to be launched; returns the launcher's exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def per_config_sweep(capmoe, synth, torch, steps: int):
    """Layer latency and tokens/s of the other workload shapes for no-drop, Token Drop and Expanded
    Drop at each capacity factor of the shape (device time, CUDA events, no stage events inside)."""
    shapes = [synth.CONFIGS["tiny_f32"], synth.CONFIGS["olmoe"], synth.CONFIGS["dsv2lite"],
              synth.CONFIGS["qwen"].with_(N=128), synth.CONFIGS["qwen"].with_(N=8192)]
    out = []
    for cfg in shapes:
        inp = synth.make_layer_inputs(cfg)
        g = {k: getattr(inp, k).cuda() for k in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}
        shared = None if inp.shared is None else tuple(t.cuda() for t in inp.shared)
        base_ms = None
        for mode, gam in [("nodrop", None)] + [(m, gm) for gm in cfg.gammas for m in ("token_drop", "expanded_drop")]:
            lay = capmoe.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k, cfg.D,
                                  mode, gamma=1.0 if gam is None else gam, shared=shared)
            ms = time_layer(lay, steps, 3, torch)
            if mode == "nodrop":
                base_ms = ms
            a = int(lay.t["expert_offsets"][-1].item())
            out.append({"workload": f"{cfg.name}: N={cfg.N} d={cfg.d} E={cfg.E} k={cfg.k} F={cfg.F} D={cfg.D} {cfg.dtype}",
                        "mode": mode, "gamma": gam, "ms_per_layer": ms, "tokens_per_s": cfg.N / (ms * 1e-3), "A": a,
                        "speedup_vs_nodrop": base_ms / ms})
            del lay
        del g, shared, inp
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="mixtral")
    ap.add_argument("--N", type=int, default=None, help="override the number of tokens (sweeps, small ncu cases)")
    ap.add_argument("--F", type=int, default=None, help="override the expert FFN width (small ncu cases)")
    ap.add_argument("--D", type=int, default=None,
                    help="override the number of virtual expert-parallel devices (E %% D == 0), e.g. the paper's "
                         "one or two experts per GPU for the Mixtral shape: --D 8, --D 4")
    ap.add_argument("--mode", default="expanded_drop", choices=["nodrop", "token_drop", "expanded_drop", "device_token_drop", "device_expanded_drop"])
    ap.add_argument("--gamma", type=float, default=1.0)
    ap.add_argument("--no-straggler", dest="straggler", action="store_false")
    ap.add_argument("--no-sweep", dest="sweep", action="store_false", help="skip the other modes")
    ap.add_argument("--table", action="store_true",
                    help="instead of the benchmark line, print one JSON line per (N, gamma, mode) point of the "
                         "chosen config (for the Qwen-shape sweep: N in 128..65536, gamma in 0.5..2.0)")
    ap.add_argument("--markdown", action="store_true", help="with --table: print a markdown table instead of JSON lines")
    ap.add_argument("--no-cpu", dest="cpu", action="store_false", help="skip the CPU baseline")
    ap.add_argument("--ep", type=int, default=0,
                    help="R > 0: instead of the benchmark line, time the ranks of an R-way expert-parallel group with "
                         "per-rank capacity one after another on this GPU (one JSON line per mode)")
    ap.add_argument("--impl", default="capmoe", choices=["capmoe", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=None,
                    help="tokens in the CPU checker's FFN sample (default 1024 for cpu_baseline, 64 per step "
                         "for --impl reference)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "capmoe":
        args.warmup = 3

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # called as `python bench.py --gpus N`: start the N ranks here (one process per GPU)
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.table:
        run_table(args)
        return
    if args.ep > 0:
        run_ep(args)
        return

    import torch
    from paper_2503_05066_b200 import capmoe, distrib, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local_rank)
    info = distrib.RankInfo(rank, world, local_rank)
    distrib.init(info, backend="nccl", device=torch.device("cuda", local_rank))
    capmoe.lib()
    peaks = _peaks()

    cfg = _pick_config(args)
    cfg = cfg.with_(seed=distrib.shard_seed(cfg.seed, info))
    if not cfg.straggler:
        args.straggler = args.straggler and False
    inp = synth.make_layer_inputs(cfg)
    dev = torch.device("cuda", local_rank)
    g = {k: getattr(inp, k).to(dev) for k in ("x", "w_router", "bias", "w_gate", "w_up", "w_down")}
    shared = None if inp.shared is None else tuple(s.to(dev) for s in inp.shared)

    def make(mode, gamma, straggler):
        return capmoe.MoELayer(g["x"], g["w_router"], g["bias"], g["w_gate"], g["w_up"], g["w_down"], cfg.k,
                               cfg.D, mode, gamma=gamma, straggler=straggler, shared=shared)

    def barrier():
        torch.cuda.synchronize()
        distrib.barrier(info)
        torch.cuda.synchronize()

    def max_over_ranks(v: float) -> float:
        return distrib.max_over_ranks(v, info, device=dev)

    # ------------------------------------------------------------------ headline: K timed steps
    # Region A: exactly K forwards, nothing else on the stream, bracketed by barrier + synchronize:
    # the headline.  Region B: K more forwards with the layer recording an event after every stage,
    # which gives the per-stage and per-kernel times (the records sit between the kernels and cost
    # about 2 % at this shape, which is why the headline is not taken from them).  The clock sampler
    # runs over both.
    layer = make(args.mode, args.gamma, args.straggler)
    K = args.steps
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(capmoe.N_STAGE_EVENTS)] for _ in range(K)]
    for evs in events:
        for e in evs:
            e.record()                                   # creates the handles
    for _ in range(args.warmup):
        layer.forward()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = capmoe.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(K):
        layer.forward()
    e1.record()
    barrier()
    launches = capmoe.launch_count() - launches0
    ms_step = max_over_ranks(e0.elapsed_time(e1) / K)
    value = distrib.job_throughput(cfg.N, ms_step, info)
    e0.record()
    for i in range(K):
        layer.set_stage_events(events[i])
        layer.forward()
    e1.record()
    barrier()
    clocks = sampler.stop()
    layer.set_stage_events(None)
    layer.check_device_status()
    ms_with_events = max_over_ranks(e0.elapsed_time(e1) / K)

    # per-step device time from each step's first to its last stage event: spread of the K steps
    per_step = sorted(events[i][0].elapsed_time(events[i][capmoe.N_STAGE_EVENTS - 1]) for i in range(K))
    step_spread = {"median_ms": statistics.median(per_step), "min_ms": per_step[0], "max_ms": per_step[-1],
                   "note": "first to last stage event of one step in the pass that records stage events"}
    stage_ms = {}
    for si, name in enumerate(capmoe.STAGE_NAMES):
        stage_ms[name] = statistics.mean(events[i][si].elapsed_time(events[i][si + 1]) for i in range(K))
    A = int(layer.t["expert_offsets"][-1].item())
    kept = layer.t["kept"].cpu().tolist()
    load = layer.t["load"].cpu().tolist()

    # ------------------------------------------------------------------ roofline of the dominant kernel
    elt = 2 if cfg.dtype == "bf16" else 4
    gemm1_flops = 4.0 * A * cfg.d * cfg.F                # 2 * A * d * (2F)
    gemm2_flops = 2.0 * A * cfg.d * cfg.F
    t1 = stage_ms["ffn_gate_up"] * 1e-3
    t2 = stage_ms["ffn_down"] * 1e-3
    use_tc = capmoe.ffn_uses_tensor_cores(cfg.d, cfg.F, g["x"].dtype)
    # Which measured cuBLAS figure bounds the kernel depends on the clock regime of the timed region:
    # a region of a second or more runs under the power cap like the sustained measurement, a short
    # one at burst clocks.  Both fractions are printed; `frac` uses the regime this run was in (the
    # denominator is cuBLAS measured the same way, so a fraction slightly above 1 is possible).
    region_s = (ms_step + ms_with_events) * 1e-3 * K
    ach1 = gemm1_flops / t1 / 1e12 if t1 > 0 else None
    ach2 = gemm2_flops / t2 / 1e12 if t2 > 0 else None
    regime = "sustained" if (region_s >= 0.5 and "sw_power_cap" in (clocks.get("reasons") or [])) else "burst"
    peak_tf = (peaks["bf16_tflops_sustained"] if regime == "sustained" else peaks["bf16_tflops"]) if use_tc else None
    tr1, tr2, tr_note = _recorded_traffic((cfg.name, cfg.N, cfg.F, args.mode, args.gamma, bool(args.straggler)))
    sm_mhz, sm_max = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    roofline = {
        "kernel": "k_ffn_tc / k_ffn_tc2 <gate/up> (grouped GEMM + SwiGLU, tcgen05)" if use_tc else "k_grouped_gemm (fp32 FMA)",
        "bound": "tensor" if use_tc else "alu",
        "achieved": ach1, "peak": peak_tf, "unit": "TFLOP/s",
        "frac": (ach1 / peak_tf) if (ach1 and peak_tf) else None,
        "peak_source": "%s cuBLAS bf16, %s figure (timed region %.2f s, median SM clock %s MHz of %s)"
                       % (peaks["source"], regime, region_s, sm_mhz, sm_max),
        "frac_note": ("above 1: this launch ran faster than the cuBLAS loop behind the %s figure, which was measured in the "
                      "same clock regime; see frac_of_burst_peak for the other denominator" % regime)
        if (ach1 and peak_tf and ach1 > peak_tf) else None,
        "frac_of_burst_peak": (ach1 / peaks["bf16_tflops"]) if (ach1 and use_tc) else None,
        "frac_of_sustained_peak": (ach1 / peaks["bf16_tflops_sustained"]) if (ach1 and use_tc) else None,
        "peak_burst": peaks["bf16_tflops"], "peak_sustained": peaks["bf16_tflops_sustained"],
        # the same throughput scaled to the maximum SM clock (time x median sampled MHz / max MHz)
        "achieved_at_max_clock": (ach1 * sm_max / sm_mhz) if (ach1 and sm_mhz and sm_max) else None,
        "achieved_at_max_clock_note": "extrapolation from the median of 100 ms nvidia-smi clock samples over the whole timed "
                                      "region; under the power cap the clock moves within a step, so this can overshoot",
        "flops_per_launch": gemm1_flops,
        "traffic": tr1, "traffic_note": tr_note,
        "algorithmic_bytes": (2 * cfg.E * cfg.F * cfg.d + A * cfg.d + A * cfg.F) * elt,
        # the same launch against the HBM roofline (it is the binding one when few rows are kept per
        # expert and the weights are streamed for little work): algorithmic bytes / time / measured copy bandwidth
        "hbm_frac": ((2 * cfg.E * cfg.F * cfg.d + A * cfg.d + A * cfg.F) * elt / t1 / 1e9 / peaks["hbm_gbs"])
        if t1 > 0 else None,
        "down_gemm": {"achieved": ach2,
                      "frac": (ach2 / peak_tf) if (ach2 and peak_tf) else None,
                      "traffic": tr2, "algorithmic_bytes": (cfg.E * cfg.F * cfg.d + A * cfg.d + A * cfg.F) * elt,
                      "hbm_frac": ((cfg.E * cfg.F * cfg.d + A * cfg.d + A * cfg.F) * elt / t2 / 1e9 / peaks["hbm_gbs"])
                      if t2 > 0 else None},
    }
    # HBM-bound stages: algorithmic bytes over stage time
    n_kept_tok = int((layer.t["keep_mask"] != 0).any(dim=1).sum().item())
    slots = layer.slots
    hbm = {
        "route": (cfg.N * cfg.d * elt + cfg.E * cfg.d * elt + 2 * 4 * cfg.N * cfg.E + 8 * cfg.N * cfg.k),
        "permute": (n_kept_tok * cfg.d * elt + A * cfg.d * elt + 8 * A + 4 * cfg.N * slots),
        "combine": (A * cfg.d * elt + cfg.N * cfg.d * elt + 4 * A + 4 * cfg.N * slots),
    }
    hbm_stages = {k: {"bytes": v, "GB/s": v / (stage_ms[k] * 1e-3) / 1e9,
                      "frac_of_measured_copy": v / (stage_ms[k] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
                  for k, v in hbm.items() if stage_ms[k] > 0}

    # Kernel-only bandwidth of the three HBM-bound stages: the same launches back to back, rotating
    # over input copies that together exceed L2 (126 MB), so that no launch finds its input cached
    # and no event record sits between launches.
    hbm_kernels = {}
    if rank == 0:
        reps = 24

        def timed(fn):
            """ms per call of fn(i), i = 0..reps-1, replayed from one CUDA graph: device time of the
            stage's launches back to back, without the host's per-call cost (which exceeds the
            duration of the shortest of these kernels)."""
            for i in range(2):
                fn(i)
            torch.cuda.synchronize()
            gr = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(gr, stream=side):
                for i in range(reps):
                    fn(i)
            gr.replay()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(3):
                gr.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / (3 * reps)

        t = layer.t
        ncopy = max(2, int(200e6 // (cfg.N * cfg.d * elt)) + 1)
        xs = [g["x"]] + [g["x"].clone() for _ in range(ncopy - 1)]
        r_out = capmoe.route(g["x"], g["w_router"], g["bias"], cfg.k)
        ms = timed(lambda i: capmoe.route(xs[i % ncopy], g["w_router"], g["bias"], cfg.k, out=r_out))
        hbm_kernels["route"] = ms
        # what a kernel that only reads the same activations once would take (launch included)
        route_floor_ms = timed(lambda i: capmoe.debug_read_probe(xs[i % ncopy]))
        A_rows = t["x_perm"].shape[0]
        pcopy = max(2, int(200e6 // (A_rows * cfg.d * elt)) + 1)
        p_outs = [dict(x_perm=torch.empty_like(t["x_perm"]), perm_token=torch.empty_like(t["perm_token"]),
                       perm_weight=torch.empty_like(t["perm_weight"])) for _ in range(pcopy)]
        Dp = cfg.D if layer.slots > cfg.k else 0
        ms = timed(lambda i: capmoe.permute(xs[i % ncopy], t["scores"], t["topk_idx"], t["slot_row"], A_rows, Dp,
                                            out=p_outs[i % pcopy]))
        hbm_kernels["permute"] = ms
        ys = [t["y_perm"]] + [t["y_perm"].clone() for _ in range(pcopy - 1)]
        y_outs = [torch.empty_like(t["y"]) for _ in range(2)]
        ms = timed(lambda i: capmoe.combine(ys[i % pcopy], t["slot_row"], t["perm_weight"], y=y_outs[i % 2]))
        hbm_kernels["combine"] = ms
        hbm_kernels = {k: {"ms": v, "bytes": hbm[k], "GB/s": hbm[k] / (v * 1e-3) / 1e9,
                           "frac_of_measured_copy": hbm[k] / (v * 1e-3) / 1e9 / peaks["hbm_gbs"]}
                       for k, v in hbm_kernels.items()}
        hbm_kernels["route"]["one_shot_read_floor_ms"] = route_floor_ms
        hbm_kernels["route"]["frac_of_read_floor"] = route_floor_ms / hbm_kernels["route"]["ms"]
        hbm_kernels["route"]["read_floor_frac_of_measured_copy"] = (cfg.N * cfg.d * elt / (route_floor_ms * 1e-3) / 1e9 /
                                                                    peaks["hbm_gbs"])
        del xs, p_outs, ys, y_outs

    # The drop stage moves a few MB: it is bound by launch and dependency latency, not by bandwidth.
    # Reported against the measured device time of a launch that does (almost) nothing: a one-element
    # capmoe_drop_keys call, the smallest kernel the library has (both replayed from CUDA graphs).
    latency_stages = {}
    if rank == 0 and args.mode != "nodrop":
        t = layer.t

        def timed_graph(fn, inner=16, graph_reps=10):
            """ms per call of fn, replayed from a CUDA graph of `inner` calls: device time without the
            host's per-call cost (which exceeds these kernels' duration)."""
            fn(0)
            torch.cuda.synchronize()
            gr = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(gr, stream=side):
                for i in range(inner):
                    fn(i)
            gr.replay()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(graph_reps):
                gr.replay()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / (graph_reps * inner)

        one = torch.zeros((1, cfg.E), device=dev, dtype=torch.float32)
        one_keys = torch.empty_like(one)
        L_ = capmoe.lib()
        import ctypes as _ct
        st_ = lambda: _ct.c_void_p(torch.cuda.current_stream().cuda_stream)
        floor_ms = timed_graph(lambda i: L_.capmoe_drop_keys(0, _ct.c_uint64(0), _ct.c_void_p(one.data_ptr()), None,
                                                             _ct.c_int64(1), cfg.E, cfg.E,
                                                             _ct.c_void_p(one_keys.data_ptr()), st_()))
        l0 = capmoe.launch_count()
        if args.mode == "token_drop":
            fn = lambda i: capmoe.token_drop(t["topk_score"], t["topk_idx"], cfg.E, layer.C, ws=t["drop_ws"])
            drop_bytes = 16 * cfg.N * cfg.k + 8 * cfg.N
        elif args.mode == "expanded_drop":
            fn = lambda i: capmoe.expanded_drop(t["scores"], t["topk_idx"], layer.C, cfg.D, ws=t["drop_ws"])
            drop_bytes = 4 * cfg.N * cfg.E + 4 * cfg.N * cfg.k + 8 * cfg.N + 4 * cfg.N * layer.slots
        else:
            fn = lambda i: capmoe.device_drop(t["scores"], t["topk_idx"], layer.C, cfg.D,
                                              args.mode == "device_expanded_drop", ws=t["drop_ws"])
            drop_bytes = 4 * cfg.N * cfg.E + 4 * cfg.N * cfg.k + 8 * cfg.N + 4 * cfg.N * layer.slots
        fn(0)
        n_launch = capmoe.launch_count() - l0
        ms = timed_graph(fn)
        latency_stages["drop"] = {"ms": ms, "kernel_launches": int(n_launch), "bytes": drop_bytes,
                                  "near_empty_launch_us": floor_ms * 1e3,
                                  "launch_floor_ms": floor_ms * n_launch,
                                  "times_launch_floor": ms / (floor_ms * n_launch) if n_launch else None}

    # ------------------------------------------------------------------ e2e through the host-buffer entry point
    # Every step copies its activations in from pinned host memory and its output back out, inside
    # the timed region.  Two layer instances (own activation buffers, shared weights) alternate on
    # two streams, so step i+1's upload and step i's download overlap the other step's kernels.
    # The input buffer is private to each instance because the entry point stages x into it.
    xh = [inp.x.clone().pin_memory() for _ in range(2)]
    yh = [torch.empty_like(xh[0]).pin_memory() for _ in range(2)]
    streams = [torch.cuda.Stream(device=dev) for _ in range(2)]

    def make_private(mode, gamma, straggler):
        return capmoe.MoELayer(torch.empty_like(g["x"]), g["w_router"], g["bias"], g["w_gate"], g["w_up"],
                               g["w_down"], cfg.k, cfg.D, mode, gamma=gamma, straggler=straggler, shared=shared)

    pipe = [layer, make_private(args.mode, args.gamma, args.straggler)]
    pipe[0] = make_private(args.mode, args.gamma, args.straggler)
    del layer

    def e2e_steps(n):
        for i in range(n):
            with torch.cuda.stream(streams[i % 2]):
                pipe[i % 2].forward_host(xh[i % 2], yh[i % 2], stream=streams[i % 2])

    e2e_steps(4)
    barrier()
    cur = torch.cuda.current_stream()
    e0.record(cur)
    for st_ in streams:
        st_.wait_event(e0)
    e2e_steps(K)
    for st_ in streams:
        cur.wait_stream(st_)
    e1.record(cur)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1) / K)
    for p_ in pipe:
        p_.check_device_status()
    # one serial step for reference (upload, layer, download back to back on one stream)
    pipe[0].forward_host(xh[0], yh[0])
    torch.cuda.synchronize()
    e0.record()
    for _ in range(3):
        pipe[0].forward_host(xh[0], yh[0])
    e1.record()
    torch.cuda.synchronize()
    ms_serial = e0.elapsed_time(e1) / 3
    nbytes = xh[0].numel() * xh[0].element_size()
    e2e = {"value": distrib.job_throughput(cfg.N, ms_e2e, info), "unit": UNIT, "ms_per_step": ms_e2e,
           "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes,
           "how": "capmoe_layer_forward_host, two instances alternating on two streams",
           "ms_per_step_single_stream": ms_serial}
    del pipe

    # ------------------------------------------------------------------ the other modes of the same workload
    modes = []
    if args.sweep and rank == 0:
        sweep_steps = max(3, min(K, 10))
        nodrop_ms = {}
        for strag in ([False, True] if cfg.straggler else [False]):
            variants = ("token_drop", "expanded_drop") + (
                ("device_token_drop", "device_expanded_drop") if cfg.D < cfg.E else ())
            for mode, gam in [("nodrop", None)] + [(m, gm) for gm in cfg.gammas for m in variants]:
                lay = make(mode, 1.0 if gam is None else gam, strag)
                ms = time_layer(lay, sweep_steps, 3, torch)
                if mode == "nodrop":
                    nodrop_ms[strag] = ms
                a = int(lay.t["expert_offsets"][-1].item())
                modes.append({"mode": mode, "gamma": gam, "straggler_emulation": strag, "ms_per_layer": ms,
                              "tokens_per_s": cfg.N / (ms * 1e-3), "A": a, "A_over_Nk": a / (cfg.N * cfg.k),
                              "speedup_vs_nodrop": nodrop_ms[strag] / ms})
                del lay

    # ------------------------------------------------------------------ the other workload shapes
    configs = []
    if args.sweep and rank == 0 and world == 1 and args.config == "mixtral":
        configs = per_config_sweep(capmoe, synth, torch, max(3, min(K, 10)))

    # ------------------------------------------------------------------ CPU baseline (rank 0, N = 1 only)
    cpu = None
    if args.cpu and rank == 0 and world == 1:
        v, detail = cpu_oracle_run(cfg, inp, args.mode, args.gamma, args.ref_tokens or 1024)
        cpu = {"value": v, "unit": UNIT, "cores": detail["cores"], "kind": "oracle",
               "sample": f"router+drop on all {cfg.N} tokens ({detail['route_drop_s_full_N']:.2f} s), expert "
                         f"FFN+combine on {detail['sample_tokens']} tokens spread over the batch "
                         f"({detail['ffn_combine_s_sample']:.2f} s); per-token times added"}

    if rank == 0:
        nbar = cfg.N * cfg.k / cfg.E
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_with_stage_events": ms_with_events,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic", "config": _config_dict(cfg, args),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu,
            "step_spread": step_spread, "stages_ms": stage_ms, "hbm_stages": hbm_stages, "hbm_kernels": hbm_kernels, "latency_stages": latency_stages,
            "workload_stats": {"A": A, "C": int(layer_C(cfg, args, capmoe)), "max_load_over_mean": max(load) / nbar,
                               "kept_fraction_of_Nk": A / (cfg.N * cfg.k), "kept_per_expert": kept,
                               "load_per_expert": load},
            "modes": modes,
            "configs": configs,
            "peaks": peaks,
        }
        print(json.dumps(line), flush=True)
    distrib.finish(info)


def layer_C(cfg, args, capmoe):
    if args.mode == "nodrop":
        return cfg.N
    if args.mode.startswith("device_"):
        return capmoe.device_capacity(cfg.N, cfg.E, cfg.k, cfg.D, args.gamma)
    return capmoe.capacity(cfg.N, cfg.E, cfg.k, args.gamma)


if __name__ == "__main__":
    main()
