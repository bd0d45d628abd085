"""Expert-parallel forward of the zero-expert MoE layer: host-side plan and exchange.

The experts are partitioned over G ranks in contiguous blocks, the tokens stay data-parallel.  Each
rank routes its own tokens, DROPS the zero-expert slots (Section 2.1: a zero expert outputs 0, so a
slot that selects one has nothing to compute anywhere) and only then packs rows for the exchange:
zero slots cost no link bytes.  The paper names expert-parallel communication as future work
(Appendix A); the arithmetic is Eq. 1 unchanged.

Per layer call and rank:
    dispatch   route, pack the x rows of the surviving pairs by (expert, token)   [library kernels]
    exchange   all-to-all of the per-expert counts, then of the rows              [this module]
    experts    grouped SwiGLU GEMMs on the received rows                          [library kernels]
    exchange   all-to-all of the result rows back                                 [this module]
    combine    Eq. 1 in token order                                               [library kernels]

The plan arithmetic lives in the small functions below; they take and return plain integers and
torch tensors on any device, so the same code runs under NCCL on GPUs and under gloo on CPU.  The
rows land in local memory first; no kernel ever reads a peer's memory.
"""
from __future__ import annotations

from typing import List, Sequence

import torch


def owner_of_expert(e: int, n_real: int, ep_size: int) -> int:
    """Rank that holds expert e: contiguous blocks of n_real / ep_size experts."""
    return e // (n_real // ep_size)


def send_counts_from_offsets(offsets: torch.Tensor, n_real: int, ep_size: int) -> List[int]:
    """Rows this rank sends to each destination: the pairs are sorted by expert and experts are
    owned in contiguous blocks, so destination r's rows are offsets[(r+1) n_local] - offsets[r n_local]."""
    n_local = n_real // ep_size
    o = offsets.tolist()
    return [int(o[(r + 1) * n_local] - o[r * n_local]) for r in range(ep_size)]


def recv_layout(recv_counts: torch.Tensor):
    """From recv_counts [G, n_local] (rows from source s for local expert j): rows per source and the
    total.  The received buffer holds source 0's block, then source 1's, ...; each block is in its
    sender's (expert, token) order."""
    per_source = [int(v) for v in recv_counts.sum(dim=1).tolist()]
    return per_source, sum(per_source)


class TorchDistExchange:
    """All-to-all over a torch.distributed process group (NCCL for device tensors, gloo for CPU)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.size = dist.get_world_size(group)

    def counts(self, expert_counts: torch.Tensor) -> torch.Tensor:
        """Sends block r of expert_counts [G * n_local] to rank r; returns recv_counts [G, n_local]."""
        n_local = expert_counts.numel() // self.size
        out = torch.empty((self.size, n_local), dtype=expert_counts.dtype, device=expert_counts.device)
        self.dist.all_to_all_single(out.view(-1), expert_counts.contiguous(), group=self.group)
        return out

    def rows(self, send: torch.Tensor, send_splits: Sequence[int], recv_splits: Sequence[int]) -> torch.Tensor:
        """Sends send[sum(splits[:r]) : sum(splits[:r+1])] to rank r; returns the received blocks in
        source order."""
        n_in = sum(send_splits)
        out = torch.empty((max(sum(recv_splits), 1), send.shape[1]), dtype=send.dtype, device=send.device)
        self.dist.all_to_all_single(out[:sum(recv_splits)], send[:n_in], output_split_sizes=list(recv_splits),
                                    input_split_sizes=list(send_splits), group=self.group)
        return out


class LoopbackExchange:
    """The exchange of a group of one: counts and rows stay where they are."""

    rank, size = 0, 1

    def counts(self, expert_counts: torch.Tensor) -> torch.Tensor:
        return expert_counts.view(1, -1).contiguous()

    def rows(self, send: torch.Tensor, send_splits: Sequence[int], recv_splits: Sequence[int]) -> torch.Tensor:
        return send


class ExpertParallelMoE:
    """One rank of an expert-parallel zero-expert MoE layer on a GPU.

    `moe` is a paper_2605_18643_b200.zeda.ZedaMoE created with ep_size = G, ep_rank = this rank and
    the weights of this rank's experts; `exchange` moves counts and rows between the ranks (None for
    a group that is stepped by forward_group_in_one_process)."""

    def __init__(self, moe, exchange):
        self.moe = moe
        self.x = exchange
        self.G = moe.cfg.ep_size
        assert self.G >= 1 and (exchange is None or exchange.size == self.G)

    def forward(self, x: torch.Tensor, out: torch.Tensor = None, launches: list = None) -> torch.Tensor:
        """One layer call of this rank.  `launches`, if given, receives the number of library kernels
        each of the three device phases enqueued (costs three host synchronisations)."""
        m = self.moe
        send_rows, send_counts, expert_counts = m.ep_dispatch(x)
        if launches is not None:
            launches.append(m.last_counters()[3])
        recv_counts = self.x.counts(expert_counts)
        # the one host synchronisation of the call: the all-to-all needs its split sizes on the host
        send_splits = [int(v) for v in send_counts.tolist()]
        recv_splits, n_rows = recv_layout(recv_counts)
        if n_rows > m.cfg.max_recv_pairs:
            raise RuntimeError("rank receives %d pair rows, handle was sized for %d" % (n_rows, m.cfg.max_recv_pairs))
        recv_rows = self.x.rows(send_rows, send_splits, recv_splits)
        out_rows = m.ep_experts(recv_rows, recv_counts, n_rows)
        if launches is not None:
            launches.append(m.last_counters()[3])
        back_rows = self.x.rows(out_rows, recv_splits, send_splits)
        y = m.ep_combine(x, back_rows, out)
        if launches is not None:
            launches.append(m.last_counters()[3])
        return y


def forward_group_in_one_process(ranks: Sequence["ExpertParallelMoE"], xs: Sequence[torch.Tensor]):
    """Runs a whole expert-parallel group step by step in ONE process (every rank's handle on the
    same GPU, device copies instead of a transport).  The phases run one after the other, so no
    kernel ever waits for another rank.  For single-GPU testing of the multi-rank data path."""
    G = len(ranks)
    packed = [r.moe.ep_dispatch(x) for r, x in zip(ranks, xs)]
    send_splits = [[int(v) for v in p[1].tolist()] for p in packed]
    n_local = ranks[0].moe.E // G
    outs = []
    recv = []
    for r in range(G):
        counts = torch.stack([packed[s][2][r * n_local:(r + 1) * n_local] for s in range(G)]).contiguous()
        blocks = []
        for s in range(G):
            start = sum(send_splits[s][:r])
            blocks.append(packed[s][0][start:start + send_splits[s][r]])
        rows = torch.cat(blocks) if sum(b.shape[0] for b in blocks) else torch.empty((1, xs[0].shape[1]), dtype=xs[0].dtype, device=xs[0].device)
        n_rows = sum(b.shape[0] for b in blocks)
        recv.append((counts, [b.shape[0] for b in blocks], n_rows))
        outs.append(ranks[r].moe.ep_experts(rows.contiguous(), counts, n_rows))
    ys = []
    for s in range(G):
        back = []
        for r in range(G):
            start = sum(recv[r][1][:s])
            back.append(outs[r][start:start + recv[r][1][s]])
        rows = torch.cat(back) if sum(b.shape[0] for b in back) else torch.empty((1, xs[0].shape[1]), dtype=xs[0].dtype, device=xs[0].device)
        ys.append(ranks[s].moe.ep_combine(xs[s], rows.contiguous()))
    return ys
