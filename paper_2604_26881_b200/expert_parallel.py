"""Expert blocks placed on several ranks: the exchange around the expert step.

The paper's compute plane puts expert blocks on different workers and names the cost of moving tokens to them as its
main limit (Sec. 5, on latency and network); on GPUs the counterpart is one process per GPU, every rank holding the
blocks a placement table gives it, with one exchange of routed rows before the expert step and one of their outputs
after it.  This module is the host-side protocol of that exchange: which rank owns which block, which rows go where,
and the two all-to-alls; routing, the permutation and the combine stay on the rank that owns the tokens.  The compute
steps are passed in as callables, so the same protocol runs on GPUs (the library's calls over NCCL) and in CPU tests
(gloo, with any stand-in for the expert step).

What is NOT here: any overlap of the exchange with the expert GEMMs (one kernel that sends and computes tile by tile
over peer memory), and any measurement: the protocol has run as CPU ranks over gloo and as a single rank over NCCL.
"""
from __future__ import annotations

from typing import Callable, List, Sequence

import torch
import torch.distributed as dist


def place_blocks(block_rows: Sequence[int], world: int) -> List[int]:
    """Rank of every block: heaviest block first, each to the rank with the fewest rows so far (ties: lowest rank)."""
    order = sorted(range(len(block_rows)), key=lambda b: (-int(block_rows[b]), b))
    load = [0] * world
    rank_of = [0] * len(block_rows)
    for b in order:
        r = min(range(world), key=lambda q: (load[q], q))
        rank_of[b] = r
        load[r] += int(block_rows[b])
    return rank_of


def rows_per_destination(expert_off: torch.Tensor, rank_of_expert: Sequence[int], world: int):
    """For rows sorted by expert (the dispatch order): the per-expert row counts [E'] and, per destination rank, the
    list of (first row, rows) segments in expert order."""
    counts = (expert_off[1:] - expert_off[:-1]).to(torch.int64)
    segs = [[] for _ in range(world)]
    for e, c in enumerate(counts.tolist()):
        if c:
            segs[rank_of_expert[e]].append((int(expert_off[e]), c))
    return counts, segs


class ExpertParallel:
    """One rank of an expert-parallel layer.

    rank_of_expert[e]: the rank that holds expert e (all experts of a block share a rank).
    expert_step(x_rows [n, H], expert_off [E'+1]) -> y_rows [n, H_out]: the expert FFNs on rows sorted by expert, where
    expert_off counts only the rows this rank received (experts it does not own have none).
    """

    def __init__(self, rank_of_expert: Sequence[int], expert_step: Callable, group=None):
        self.rank_of_expert = list(rank_of_expert)
        self.expert_step = expert_step
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def exchange_counts(self, counts: torch.Tensor) -> torch.Tensor:
        """counts [E'] of this rank's rows per expert -> [world, E'] rows every rank sends to the experts this rank owns
        (zero elsewhere).  One small all-to-all of int64."""
        n_exp = counts.numel()
        owned = torch.tensor([1 if r == self.rank else 0 for r in self.rank_of_expert], dtype=torch.int64, device=counts.device)
        send = torch.stack([counts * torch.tensor([1 if self.rank_of_expert[e] == q else 0 for e in range(n_exp)],
                                                  dtype=torch.int64, device=counts.device) for q in range(self.world)])
        recv = torch.empty_like(send)
        dist.all_to_all_single(recv, send, group=self.group)
        return recv * owned

    def forward_rows(self, x_perm: torch.Tensor, expert_off: torch.Tensor, out_features: int, out_dtype=None):
        """x_perm [R, H]: this rank's routed rows in dispatch order; expert_off [E'+1].  Returns y_perm [R, out_features]
        in the same order: every row computed by the rank that holds its expert."""
        dev = x_perm.device
        out_dtype = out_dtype or x_perm.dtype
        counts, segs = rows_per_destination(expert_off.cpu(), self.rank_of_expert, self.world)
        recv_counts = self.exchange_counts(counts.to(dev)).cpu()              # [world, E']
        # send buffer: destination-major, expert order inside a destination
        send_rows = [sum(c for _, c in segs[q]) for q in range(self.world)]
        idx = [torch.arange(a, a + c) for q in range(self.world) for (a, c) in segs[q]]
        send_index = torch.cat(idx) if idx else torch.zeros(0, dtype=torch.int64)
        send_buf = x_perm[send_index.to(dev)] if send_index.numel() else x_perm[:0]
        recv_rows = recv_counts.sum(dim=1).tolist()
        recv_buf = torch.empty((sum(recv_rows), x_perm.shape[1]), dtype=x_perm.dtype, device=dev)
        dist.all_to_all_single(recv_buf, send_buf.contiguous(), output_split_sizes=recv_rows, input_split_sizes=send_rows,
                               group=self.group)
        # received rows are source-major; the expert step wants them expert-major (source order inside an expert)
        n_exp = counts.numel()
        src_base = [0]
        for r in recv_rows:
            src_base.append(src_base[-1] + r)
        order, local_off = [], [0]
        within = [0] * self.world                        # rows of each source consumed so far (they arrive in expert order)
        for e in range(n_exp):
            for q in range(self.world):
                c = int(recv_counts[q, e])
                if c:
                    order.append(torch.arange(src_base[q] + within[q], src_base[q] + within[q] + c))
                    within[q] += c
            local_off.append(local_off[-1] + int(recv_counts[:, e].sum()))
        order_t = (torch.cat(order) if order else torch.zeros(0, dtype=torch.int64)).to(dev)
        x_local = recv_buf[order_t] if order_t.numel() else recv_buf
        y_local = self.expert_step(x_local, torch.tensor(local_off, dtype=torch.int32, device=dev))
        # back: undo the local order, return every row to its source, undo the send order
        y_back = torch.empty((recv_buf.shape[0], out_features), dtype=out_dtype, device=dev)
        if order_t.numel():
            y_back[order_t] = y_local.to(out_dtype)
        y_recv = torch.empty((send_buf.shape[0], out_features), dtype=out_dtype, device=dev)
        dist.all_to_all_single(y_recv, y_back, output_split_sizes=send_rows, input_split_sizes=recv_rows, group=self.group)
        y_perm = torch.empty((x_perm.shape[0], out_features), dtype=out_dtype, device=dev)
        if send_index.numel():
            y_perm[send_index.to(dev)] = y_recv
        return y_perm
