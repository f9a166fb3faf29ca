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


def exchange_rows(send: torch.Tensor, R: int, group=None) -> torch.Tensor:
    """send [R * B, ...]: block r' goes to rank r'.  Returns recv of the same shape: block r came
    from rank r.  Equal splits: the per-rank capacity bounds every block, so no sizes are exchanged."""
    assert send.shape[0] % R == 0
    recv = torch.empty_like(send)
    if R == 1:
        recv.copy_(send)
    else:
        dist.all_to_all_single(recv, send.contiguous(), group=group)
    return recv


def owner_layout(rank: int, R: int, m: int, C: int):
    """Where rank `rank`'s block sits in an owner's [R][m][C] receive space: (first row, rows)."""
    return rank * m * C, m * C


class EPRank:
    """One rank of the group: its tokens, the router, its m experts, and every buffer of a forward."""

    def __init__(self, rank: int, R: int, x, w_router, bias, w_gate_local, w_up_local, w_down_local, k: int,
                 mode: str, gamma: float = 1.0, C_buf: Optional[int] = None, round_mode: str = "ceil"):
        assert mode in ("nodrop", "token_drop", "expanded_drop")
        self.rank, self.R, self.k, self.mode = rank, R, k, mode
        self.x, self.w_router, self.bias = x, w_router, bias
        self.w_gate, self.w_up, self.w_down = w_gate_local, w_up_local, w_down_local
        N, d = x.shape
        E = w_router.shape[0]
        assert E % R == 0 and w_gate_local.shape[0] == E // R
        self.N, self.d, self.E, self.m = N, d, E, E // R
        self.C_local = N if mode == "nodrop" else capmoe.capacity(N, E, k, gamma, round_mode)
        # the row stride every rank of the group uses (>= every rank's own capacity)
        self.C = self.C_local if C_buf is None else int(C_buf)
        assert self.C >= self.C_local
        self.expanded = mode == "expanded_drop"
        self.slots = k + self.m if self.expanded else k
        dev, dt = x.device, x.dtype
        rows = max(E * self.C, 1)
        self.token_group = torch.full((N,), rank, device=dev, dtype=torch.int32) if self.expanded else None
        self.drop_ws = torch.empty((capmoe.drop_workspace_bytes(N, E, k, R, self.expanded),), device=dev,
                                   dtype=torch.uint8)
        self.x_send = torch.zeros((rows, d), device=dev, dtype=dt)         # [E][C] rows of this rank
        self.x_recv = torch.zeros((rows, d), device=dev, dtype=dt)         # [R][m][C] rows this rank owns
        self.h_ws = torch.empty((rows, w_gate_local.shape[-2]), device=dev, dtype=dt)
        self.y_recv = torch.zeros((rows, d), device=dev, dtype=dt)
        self.y_ret = torch.zeros((rows, d), device=dev, dtype=dt)
        self.perm = dict(perm_token=torch.full((rows,), -1, device=dev, dtype=torch.int32),
                         perm_weight=torch.zeros((rows,), device=dev, dtype=torch.float32))
        self.cnt_recv = torch.zeros((E,), device=dev, dtype=torch.int32)   # [R][m] kept of (source, local expert)
        self.dev_status = torch.zeros((capmoe.FFN_STATUS_WORDS,), device=dev, dtype=torch.int32)
        self.y = torch.empty((N, d), device=dev, dtype=dt)

    # ---- stage 1-3 on the rank's own tokens, then the fixed row places
    def route_and_drop(self):
        self.r = capmoe.route(self.x, self.w_router, self.bias, self.k)
        if self.expanded:
            self.dr = capmoe.expanded_drop(self.r["scores"], self.r["topk_idx"], self.C_local, self.R,
                                           token_group=self.token_group, ws=self.drop_ws)
        else:
            self.dr = capmoe.token_drop(self.r["topk_score"], self.r["topk_idx"], self.E, self.C_local, ws=self.drop_ws)
        self.slot_row_ep, self.bad = capmoe.ep_plan(self.dr["slot_row"], self.r["topk_idx"], self.dr["offsets"], self.E,
                                                    self.C, D=self.R if self.expanded else 1,
                                                    token_group=self.token_group)
        return self.dr["kept"]                         # [E] = [R][m]: rows for (owner, its local expert)

    @property
    def _Dp(self):
        return self.R if self.expanded else 0

    # ---- stage 4, collective transport: fill the send buffer
    def fill_send_buffer(self):
        capmoe.permute(self.x, self.r["scores"], self.r["topk_idx"], self.slot_row_ep, self.x_send.shape[0], self._Dp,
                       token_group=self.token_group,
                       out=dict(x_perm=self.x_send, perm_token=self.perm["perm_token"],
                                perm_weight=self.perm["perm_weight"]))
        return self.x_send

    # ---- stage 4, peer transport: store rows straight into the owners' buffers
    def dispatch_to_peers(self, peer_x_recv: torch.Tensor):
        capmoe.ep_dispatch(self.x, self.r["scores"], self.r["topk_idx"], self.slot_row_ep, peer_x_recv, self.R,
                           self.rank, self.C, D=self._Dp, token_group=self.token_group, out=self.perm)

    # ---- stage 5 on the owner: every (source, local expert) pair is a segment at a fixed place
    def expert_ffn(self):
        self.seg_begin, self.seg_end = capmoe.ep_segments(self.cnt_recv, self.C)
        if self.E * self.C > 0:
            capmoe.grouped_ffn_segments(self.x_recv, self.seg_begin, self.seg_end, self.w_gate, self.w_up, self.w_down,
                                        self.m, h_ws=self.h_ws, y_rows=self.y_recv, dev_status=self.dev_status)
        return self.y_recv

    # ---- stage 6
    def combine_returned(self):
        return capmoe.combine(self.y_ret, self.slot_row_ep, self.perm["perm_weight"], y=self.y)

    def combine_from_peers(self, peer_y_recv: torch.Tensor):
        return capmoe.ep_combine(peer_y_recv, self.R, self.rank, self.E, self.C, self.slot_row_ep,
                                 self.perm["perm_weight"], self.d, self.x.dtype, y=self.y)

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
        kept = self.route_and_drop()
        self.fill_send_buffer()
        self.x_recv = exchange_rows(self.x_send, self.R, self.group)
        self.cnt_recv = exchange_rows(kept, self.R, self.group)
        self.expert_ffn()
        self.y_ret = exchange_rows(self.y_recv, self.R, self.group)
        return self.combine_returned()


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

    def _all_to_all(self, bufs_send, bufs_recv):
        R = self.R
        B = bufs_send[0].shape[0] // R
        for r in range(R):
            for o in range(R):
                bufs_recv[o][r * B:(r + 1) * B].copy_(bufs_send[r][o * B:(o + 1) * B])

    def forward(self):
        kept = [rk.route_and_drop() for rk in self.ranks]
        if self.transport == "collective":
            for rk in self.ranks:
                rk.fill_send_buffer()
            self._all_to_all([rk.x_send for rk in self.ranks], [rk.x_recv for rk in self.ranks])
        else:
            for rk in self.ranks:
                rk.dispatch_to_peers(self.peer_x)
        self._all_to_all(kept, [rk.cnt_recv for rk in self.ranks])
        for rk in self.ranks:
            rk.expert_ffn()
        if self.transport == "collective":
            self._all_to_all([rk.y_recv for rk in self.ranks], [rk.y_ret for rk in self.ranks])
            return [rk.combine_returned() for rk in self.ranks]
        return [rk.combine_from_peers(self.peer_y) for rk in self.ranks]
