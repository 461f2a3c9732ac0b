"""Expert-parallel forward of the FP8 MoE layer: experts split across ranks in contiguous ranges of
expert ids, tokens stay where they are, two all-to-all exchanges per layer (quantized rows out,
bf16 contributions back).

The arithmetic is the library's (`moe_dispatch`, `moe_experts_fwd`, `moe_combine_sorted` run the kernels of
the single-GPU layer on the same per-row data); this module only plans and performs the exchanges, so by
the row invariance (App. C) the output equals the single-GPU layer's bit for bit for any number of ranks.

Two drivers share the three phases of `ExpertParallelMoE`:
  * `forward(...)`: one process per GPU, `torch.distributed.all_to_all_single` (NCCL on GPUs, gloo on CPU
    tensors) for the exchanges;
  * `run_local(ranks, inputs)`: all ranks' phases run in one process, one after the other, the exchanges
    done by slicing: the form to use with fewer GPUs than ranks (kernels of different ranks never wait
    on one another here, so running them in turn on one GPU is safe).

`stages` is the compute backend: `CudaStages` (the product) or any object with the same three methods
and a `contrib_dtype` (the element type of what `experts` writes).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch
import torch.distributed as dist


def expert_range(rank: int, world: int, E: int) -> tuple[int, int]:
    """Global expert ids [lo, hi) owned by `rank`."""
    if E % world:
        raise ValueError(f"E={E} must be a multiple of the number of ranks {world}")
    per = E // world
    return rank * per, (rank + 1) * per


def send_counts(offsets: torch.Tensor, world: int) -> torch.Tensor:
    """offsets [E+1] of the expert-sorted layout -> int64 [world, E/world]: rows this rank holds for each
    expert of each destination rank."""
    off = offsets.to(device="cpu", dtype=torch.int64)
    E = off.numel() - 1
    expert_range(0, world, E)
    return (off[1:] - off[:-1]).reshape(world, E // world)


def group_offsets(counts_row: torch.Tensor, device) -> torch.Tensor:
    """int64 [E_local] rows per local expert -> int32 [E_local+1] exclusive prefix sums on `device`."""
    off = torch.zeros(counts_row.numel() + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(counts_row.to("cpu"), 0)
    return off.to(device=device, dtype=torch.int32)


class CudaStages:
    """The three device stages on this rank's GPU; w13 / w2 are (codes, scales) of the LOCAL experts."""

    contrib_dtype = torch.bfloat16

    def __init__(self, ctx, w13, w2, E: int):
        self.ctx, self.w13, self.w2, self.E = ctx, w13, w2, E

    def dispatch(self, x, ids, wts):
        return self.ctx.moe_dispatch(x, ids, wts, self.E)

    def experts(self, codes, scales, weights, offsets, out):
        return self.ctx.moe_experts_fwd(codes, scales, weights, offsets, *self.w13, *self.w2, out=out)

    def combine(self, contrib_sorted, ids, pos_of_pair):
        return self.ctx.moe_combine_sorted(contrib_sorted, ids, pos_of_pair, self.E)


@dataclass
class _InFlight:
    """What a rank keeps between the phases of one forward."""
    ids: torch.Tensor
    pos_of_pair: torch.Tensor
    send: list            # [codes, scales, weights], expert-sorted = grouped by destination rank
    counts_out: torch.Tensor                      # [world, E_local] rows sent per destination expert
    counts_in: torch.Tensor | None = None         # [world, E_local] rows received per source and local expert


class ExpertParallelMoE:
    def __init__(self, stages, rank: int, world: int, E: int, group=None):
        expert_range(rank, world, E)
        self.stages, self.rank, self.world, self.E, self.group = stages, rank, world, E, group

    # -------------------------------------------------------------- the three phases
    def begin(self, x, ids, wts) -> _InFlight:
        d = self.stages.dispatch(x, ids, wts)
        return _InFlight(ids=ids, pos_of_pair=d["pos_of_pair"], send=[d["codes"], d["scales"], d["weights"]],
                         counts_out=send_counts(d["offsets"], self.world))

    def middle(self, st: _InFlight, codes, scales, weights) -> torch.Tensor:
        """Run the local experts over the received rows, source by source (each source's rows arrive sorted
        by expert); returns the contributions in the order of arrival."""
        rows = st.counts_in.sum(1).tolist()
        H = codes.shape[1]
        out = torch.empty((sum(rows), H), dtype=self.stages.contrib_dtype, device=codes.device)
        at = 0
        for s, n in enumerate(rows):
            if n:
                off = group_offsets(st.counts_in[s], codes.device)
                self.stages.experts(codes[at:at + n], scales[at:at + n], weights[at:at + n], off, out[at:at + n])
            at += n
        return out

    def finish(self, st: _InFlight, contrib_back) -> torch.Tensor:
        return self.stages.combine(contrib_back, st.ids, st.pos_of_pair)

    # -------------------------------------------------------------- one process per rank
    def forward(self, x, ids, wts) -> torch.Tensor:
        st = self.begin(x, ids, wts)
        dev = st.send[0].device
        st.counts_in = exchange_counts(st.counts_out, dev, self.group)
        rows_out, rows_in = st.counts_out.sum(1).tolist(), st.counts_in.sum(1).tolist()
        got = [exchange_rows(t, rows_out, rows_in, self.group) for t in st.send]
        contrib = self.middle(st, *got)
        back = exchange_rows(contrib, rows_in, rows_out, self.group)
        return self.finish(st, back)


def exchange_counts(counts_out: torch.Tensor, device, group=None) -> torch.Tensor:
    """counts_out [world, E_local] (row g: what this rank sends to rank g) -> counts_in [world, E_local]
    (row s: what rank s sends here).  The tensors travel on `device` (NCCL needs device memory)."""
    src = counts_out.to(device).contiguous()
    dst = torch.empty_like(src)
    dist.all_to_all_single(dst, src, group=group)
    return dst.cpu()


def exchange_rows(t: torch.Tensor, rows_out: list[int], rows_in: list[int], group=None) -> torch.Tensor:
    """Send rows_out[g] leading rows of `t` (in order) to each rank g; returns the rows_in[s] rows received
    from each rank s, in rank order."""
    out = torch.empty((sum(rows_in), *t.shape[1:]), dtype=t.dtype, device=t.device)
    dist.all_to_all_single(out, t.contiguous(), output_split_sizes=rows_in, input_split_sizes=rows_out, group=group)
    return out


def run_local(ranks: list[ExpertParallelMoE], inputs: list[tuple]) -> list[torch.Tensor]:
    """All ranks in this process: inputs[r] = (x, ids, wts) of rank r -> [out_r].  The exchanges are slices and
    concatenations of the ranks' buffers; phases of different ranks run one after the other."""
    world = len(ranks)
    sts = [ep.begin(*inp) for ep, inp in zip(ranks, inputs)]
    bounds = []                                   # bounds[s][g]: slice of rank s's sorted rows that goes to rank g
    for st in sts:
        edges = [0] + torch.cumsum(st.counts_out.sum(1), 0).tolist()
        bounds.append([slice(edges[g], edges[g + 1]) for g in range(world)])
    contribs = []
    for r, (ep, st) in enumerate(zip(ranks, sts)):
        st.counts_in = torch.stack([sts[s].counts_out[r] for s in range(world)])
        got = [_cat([sts[s].send[i][bounds[s][r]] for s in range(world)]) for i in range(3)]
        contribs.append(ep.middle(st, *got))
    outs = []
    for r, (ep, st) in enumerate(zip(ranks, sts)):
        pieces = []
        for g in range(world):                    # what rank g computed for the rows that came from rank r
            edges = [0] + torch.cumsum(sts[g].counts_in.sum(1), 0).tolist()
            pieces.append(contribs[g][edges[r]:edges[r + 1]])
        outs.append(ep.finish(st, _cat(pieces)))
    return outs


def _cat(pieces: list[torch.Tensor]) -> torch.Tensor:
    return pieces[0] if len(pieces) == 1 else torch.cat(pieces)
