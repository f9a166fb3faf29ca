"""The exchange of the expert-parallel layer among two CPU ranks (gloo): each rank lays the checker's
kept rows out in the fixed [E][C] row space, the rows and the per-expert counts cross with the same
equal-split all-to-all the GPU path uses (paper_2503_05066_b200.ep.exchange_rows), the owner runs
the checker's expert FFN on the segments it received, the results cross back, and the combined
output must equal the checker's ep_layer, which moves nothing.  This covers the host side of the
N > 1 path: block order, which block goes where, counts travelling with the rows."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2503_05066_b200 import ep, synth
from tests.util import to_np

R, N_LOCAL, MODE, GAMMA = 2, 96, "expanded_drop", 1.0


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _inputs():
    cfg = synth.CONFIGS["tiny_f32"].with_(N=R * N_LOCAL, d=64, E=8, k=2, F=48, D=R)
    inp = synth.make_layer_inputs(cfg)
    x = to_np(inp.x)
    xs = [np.ascontiguousarray(x[r * N_LOCAL:(r + 1) * N_LOCAL]) for r in range(R)]
    w = [to_np(t) for t in (inp.w_router, inp.w_gate, inp.w_up, inp.w_down)]
    return cfg, xs, w, inp.bias.numpy()


def _worker(rank, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=R)
    cfg, xs, w, bias = _inputs()
    E, m, d = cfg.E, cfg.E // R, cfg.d
    ref = oracle.ep_layer(xs, w[0], bias, w[1], w[2], w[3], cfg.k, GAMMA, MODE, cfg.dtype)
    mine = ref["ranks"][rank]                          # this rank's routing, drop and packed rows
    C = mine["C"]
    # fixed places: row e*C + i for the i-th kept row of expert e
    x_send = np.zeros((E * C, d), np.float32)
    slot_row_ep = np.full_like(mine["slot_row"], -1)
    off = mine["offsets"]
    for e in range(E):
        x_send[e * C:e * C + mine["kept"][e]] = mine["x_perm"][off[e]:off[e + 1]]
    for row in range(mine["A"]):
        e, t = int(mine["perm_expert"][row]), int(mine["perm_token"][row])
        slot_row_ep[t][mine["slot_row"][t] == row] = e * C + (row - off[e])
    x_recv = ep.exchange_rows(torch.from_numpy(x_send), R).numpy()
    cnt = ep.exchange_rows(torch.from_numpy(mine["kept"].astype(np.int32)), R).numpy()     # [source][local expert]
    # owner: segment s = (source, local expert) at rows [s*C, s*C + cnt[s])
    y_recv = np.zeros((E * C, d), np.float64)
    wl = [np.ascontiguousarray(t[rank * m:(rank + 1) * m]) for t in w[1:]]
    for s in range(R * m):
        if cnt[s]:
            rows = np.ascontiguousarray(x_recv[s * C:s * C + cnt[s]])
            y_recv[s * C:s * C + cnt[s]] = oracle.expert_ffn(rows, np.full((cnt[s],), s % m, np.int32), *wl, cfg.dtype)
    y_ret = ep.exchange_rows(torch.from_numpy(y_recv), R).numpy()
    y = oracle.combine(y_ret, slot_row_ep, mine["scores"], mine["topk_idx"], mine["Dp"], None, mine["tg"])
    np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
    np.save(os.path.join(out_dir, f"ref{rank}.npy"), ref["y"][rank])
    np.save(os.path.join(out_dir, f"cnt{rank}.npy"), np.stack([cnt, ref["send_counts"][:, rank, :].reshape(-1)]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_cpu_ranks_exchange_rows_and_counts(tmp_path):
    mp.spawn(_worker, args=(_free_port(), str(tmp_path)), nprocs=R, join=True)
    for r in range(R):
        cnt = np.load(tmp_path / f"cnt{r}.npy")
        assert np.array_equal(cnt[0], cnt[1])
        y, ref = np.load(tmp_path / f"y{r}.npy"), np.load(tmp_path / f"ref{r}.npy")
        assert np.abs(ref).max() > 0
        assert np.array_equal(y, ref)


def test_single_rank_exchange_is_a_copy():
    a = torch.arange(12.0).reshape(6, 2)
    b = ep.exchange_rows(a, 1)
    assert torch.equal(a, b) and b.data_ptr() != a.data_ptr()
    assert ep.owner_layout(2, 4, 3, 10) == (60, 30)
