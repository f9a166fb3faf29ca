"""Expert parallelism with per-rank capacity: the layer spread over R ranks, each holding its own
tokens (data parallel) and m = E/R of the experts (expert parallel), as in the paper's deployment.

The capacity is applied inside every rank (C_local from the rank's own token count), so a rank
keeps at most C_local rows per expert and tokens are dropped before anything is exchanged.  That
bound gives every row a fixed place: a rank's kept rows live in an [E][C] row space (row e*C + i =
i-th kept row of expert e), block r' of it belongs to owner r', and an owner receives [R][m][C]
rows, source-major.  Nothing about the routing result has to reach the host, and the exchange is

  transport "collective"   two equal-split all-to-alls each way (rows, and m counts per pair) over
                           torch.distributed (NCCL on GPUs; gloo works for CPU tensors)
  transport "peer"         the permute kernel stores every kept row straight into its owner's
                           buffer and the combine kernel reads every result straight from it
                           (peer-mapped memory inside one node; plain stores and loads); only the
                           counts go through the small all-to-all

Every step of the layer runs in the CUDA library (capmoe.*); this module orders the calls of one
rank (EPRank), moves buffers between ranks, and can run a whole group on ONE device, rank after
rank and stage after stage (EPGroupOnOneDevice), which is how the path is checked on a single GPU:
no kernel ever waits for another rank, the ordering between ranks is the order of the calls.
"""
from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist

from . import capmoe


def exchange_rows(send: torch.Tensor, R: int, group=None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """send [R * B, ...]: block r' goes to rank r'.  Returns recv of the same shape: block r came
    from rank r.  Equal splits: the per-rank capacity bounds every block, so no sizes are exchanged."""
    assert send.shape[0] % R == 0
    recv = torch.empty_like(send) if out is None else out
    if R == 1:
        recv.copy_(send)
    else:
        dist.all_to_all_single(recv, send.contiguous(), group=group)
    return recv


def owner_layout(rank: int, R: int, m: int, C: int):
    """Where rank `rank`'s block sits in an owner's [R][m][C] receive space: (first row, rows)."""
    return rank * m * C, m * C


class EPRank:
    """One rank of the group: its tokens, the router, its m experts, and every buffer of a forward.
    The three phases of the forward are the library's capmoe_ep_forward_* calls on one struct."""

    def __init__(self, rank: int, R: int, x, w_router, bias, w_gate_local, w_up_local, w_down_local, k: int,
                 mode: str, gamma: float = 1.0, C_buf: Optional[int] = None, round_mode: str = "ceil"):
        assert mode in capmoe.EP_MODES
        self.rank, self.R, self.k, self.mode = rank, R, k, mode
        self.x, self.w_router, self.bias = x, w_router, bias
        self.w_gate, self.w_up, self.w_down = w_gate_local, w_up_local, w_down_local
        N, d = x.shape
        E = w_router.shape[0]
        assert E % R == 0 and w_gate_local.shape[0] == E // R
        self.N, self.d, self.E, self.m = N, d, E, E // R
        self.F = w_gate_local.shape[-2]
        self.C_local = N if mode == "nodrop" else capmoe.capacity(N, E, k, gamma, round_mode)
        # the row stride every rank of the group uses (>= every rank's own capacity)
        self.C = self.C_local if C_buf is None else int(C_buf)
        assert self.C >= self.C_local
        self.expanded = mode == "expanded_drop"
        self.slots = k + self.m if self.expanded else k
        dev, dt = x.device, x.dtype
        i32 = dict(device=dev, dtype=torch.int32)
        f32 = dict(device=dev, dtype=torch.float32)
        rows = max(E * self.C, 1)
        self.token_group = torch.full((N,), rank, **i32) if self.expanded else None
        self.drop_ws = torch.empty((max(capmoe.drop_workspace_bytes(N, E, k, R, self.expanded), 1),), device=dev,
                                   dtype=torch.uint8)
        self.r = dict(logits=torch.empty((N, E), **f32), scores=torch.empty((N, E), **f32),
                      topk_idx=torch.empty((N, k), **i32), topk_score=torch.empty((N, k), **f32),
                      load=torch.zeros((E,), **i32))
        self.dr = dict(keep_mask=torch.zeros((N, (E + 63) // 64), device=dev, dtype=torch.int64),
                       cand=torch.zeros((E,), **i32), kept=torch.zeros((E,), **i32),
                       offsets=torch.zeros((E + 1,), **i32), slot_row=torch.full((N, self.slots), -1, **i32))
        self.slot_row_ep = torch.full((N, self.slots), -1, **i32)
        self.bad = torch.zeros((1,), **i32)
        self.x_send = torch.zeros((rows, d), device=dev, dtype=dt)         # [E][C] rows of this rank
        self.x_recv = torch.zeros((rows, d), device=dev, dtype=dt)         # [R][m][C] rows this rank owns
        self.h_ws = torch.empty((rows, self.F), device=dev, dtype=dt)
        self.y_recv = torch.zeros((rows, d), device=dev, dtype=dt)
        self.y_ret = torch.zeros((rows, d), device=dev, dtype=dt)
        self.perm = dict(perm_token=torch.full((rows,), -1, **i32), perm_weight=torch.zeros((rows,), **f32))
        self.cnt_recv = torch.zeros((E,), **i32)                           # [R][m] kept of (source, local expert)
        self.seg_begin = torch.zeros((E,), **i32)
        self.seg_end = torch.zeros((E,), **i32)
        self.dev_status = torch.zeros((capmoe.FFN_STATUS_WORDS,), **i32)
        self.y = torch.empty((N, d), device=dev, dtype=dt)
        self._peer_x = self._peer_y = None

    def set_peers(self, peer_x: Optional[torch.Tensor], peer_y: Optional[torch.Tensor]):
        """Device tables [R] (int64) of the ranks' x_recv / y_recv addresses: peer transport."""
        self._peer_x, self._peer_y = peer_x, peer_y

    def _struct(self):
        return capmoe.ep_rank_struct(
            N=self.N, d=self.d, E=self.E, k=self.k, F=self.F, dtype=capmoe._dt(self.x), R=self.R, rank=self.rank,
            mode=capmoe.EP_MODES[self.mode], C_local=self.C_local, C=self.C,
            x=self.x, w_router=self.w_router, bias=self.bias, w_gate=self.w_gate, w_up=self.w_up, w_down=self.w_down,
            logits=self.r["logits"], scores=self.r["scores"], topk_idx=self.r["topk_idx"],
            topk_score=self.r["topk_score"], load=self.r["load"], keep_mask=self.dr["keep_mask"], cand=self.dr["cand"],
            kept=self.dr["kept"], expert_offsets=self.dr["offsets"], slot_row=self.dr["slot_row"],
            slot_row_ep=self.slot_row_ep, token_group=self.token_group, perm_token=self.perm["perm_token"],
            perm_weight=self.perm["perm_weight"], x_send=self.x_send, y_ret=self.y_ret, peer_x=self._peer_x,
            peer_y=self._peer_y, x_recv=self.x_recv, h_ws=self.h_ws, y_recv=self.y_recv, cnt_recv=self.cnt_recv,
            seg_begin=self.seg_begin, seg_end=self.seg_end, y=self.y, drop_ws=self.drop_ws,
            drop_ws_bytes=self.drop_ws.numel(), dev_status=self.dev_status, bad=self.bad)

    def dispatch(self):
        """Stages 1-4 on the rank's own tokens: router, drop with C_local, fixed row places, and the
        rows on their way (into the owners' buffers, or into x_send).  Returns kept [E] = [R][m]:
        rows for (owner, its local expert)."""
        capmoe.ep_forward_dispatch(self._struct())
        return self.dr["kept"]

    def expert_ffn(self):
        """Stage 5 on the owner: every (source, local expert) pair is a segment at a fixed place."""
        capmoe.ep_forward_experts(self._struct())
        return self.y_recv

    def combine(self):
        """Stage 6: from the owners' buffers (peer transport) or from y_ret."""
        capmoe.ep_forward_combine(self._struct())
        return self.y

    def check(self):
        if int(self.bad.item()) != 0:
            raise capmoe.CapmoeError(capmoe.EINVAL, "an expert holds more rows than the per-rank capacity allows")
        s = int(self.dev_status[0].item())
        if s != capmoe.OK:
            raise capmoe.CapmoeError(s, "device status")


class EPLayer(EPRank):
    """A rank of a real group (one process per GPU, torch.distributed initialised): collective
    transport.  The group agrees once, at construction, on the row stride (the largest capacity)."""

    def __init__(self, rank: int, R: int, x, w_router, bias, w_gate_local, w_up_local, w_down_local, k: int,
                 mode: str, gamma: float = 1.0, round_mode: str = "ceil", group=None):
        self.group = group
        N, E = x.shape[0], w_router.shape[0]
        c_local = N if mode == "nodrop" else capmoe.capacity(N, E, k, gamma, round_mode)
        if R > 1:
            c = torch.tensor([c_local], device=x.device, dtype=torch.int64)
            dist.all_reduce(c, op=dist.ReduceOp.MAX, group=group)
            c_local = int(c.item())
        super().__init__(rank, R, x, w_router, bias, w_gate_local, w_up_local, w_down_local, k, mode, gamma,
                         C_buf=c_local, round_mode=round_mode)

    def forward(self):
        kept = self.dispatch()
        exchange_rows(self.x_send, self.R, self.group, out=self.x_recv)
        exchange_rows(kept, self.R, self.group, out=self.cnt_recv)
        self.expert_ffn()
        exchange_rows(self.y_recv, self.R, self.group, out=self.y_ret)
        return self.combine()


class EPGroupOnOneDevice:
    """All R ranks of a group on one device, for checking the whole path with a single GPU.  The
    ranks' stages run one after another on the current stream; moving a block from one rank's send
    buffer to another's receive buffer stands for the all-to-all ("collective"), or the kernels are
    given the other ranks' buffer addresses ("peer"), which on one device are ordinary pointers."""

    def __init__(self, ranks: List[EPRank], transport: str = "collective"):
        assert transport in ("collective", "peer")
        self.ranks, self.transport = ranks, transport
        self.R = len(ranks)
        assert all(rk.C == ranks[0].C and rk.R == self.R for rk in ranks)
        dev = ranks[0].x.device
        self.peer_x = torch.tensor([rk.x_recv.data_ptr() for rk in ranks], device=dev, dtype=torch.int64)
        self.peer_y = torch.tensor([rk.y_recv.data_ptr() for rk in ranks], device=dev, dtype=torch.int64)
        for rk in ranks:
            rk.set_peers(*((self.peer_x, self.peer_y) if transport == "peer" else (None, None)))

    def _all_to_all(self, bufs_send, bufs_recv):
        R = self.R
        B = bufs_send[0].shape[0] // R
        for r in range(R):
            for o in range(R):
                bufs_recv[o][r * B:(r + 1) * B].copy_(bufs_send[r][o * B:(o + 1) * B])

    def forward(self):
        kept = [rk.dispatch() for rk in self.ranks]
        if self.transport == "collective":
            self._all_to_all([rk.x_send for rk in self.ranks], [rk.x_recv for rk in self.ranks])
        self._all_to_all(kept, [rk.cnt_recv for rk in self.ranks])
        for rk in self.ranks:
            rk.expert_ffn()
        if self.transport == "collective":
            self._all_to_all([rk.y_recv for rk in self.ranks], [rk.y_ret for rk in self.ranks])
        return [rk.combine() for rk in self.ranks]
