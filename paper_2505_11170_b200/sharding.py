"""Sampling a tensor that is held in parts, one per rank (ZeRO / FSDP style flat shards).

Section 3.5 leaves the 2 bytes per parameter of w_hat to training parallelism.  Rank r of W then holds the
logical elements [bounds[r], bounds[r+1]) of a dense tensor whose groups are runs of ``group`` consecutive
elements (1 x G groups with G dividing cols, or whole rows).  Almost all of a shard is whole groups and goes
through the fused calls unchanged; at most one group at each end reaches into a neighbour's memory.  For those
two the steps of Eq. 3 / Eq. 4 are taken apart (see ``include/gws.h``, "tensors held in parts") around one small
all-reduce each way:

  forward   partial max of the end pieces -> all-reduce(MAX) over W+1 floats -> scale -> given-scale sampling
  backward  partial gradient of the end pieces -> all-reduce(SUM) over W+1 floats

Slot k of the reduced buffer belongs to the cut between ranks k-1 and k; a rank adds its partial result to every
cut that lies inside the same group as its piece (a group wider than a shard spans several cuts), so after the
reduction each slot holds the result for the whole group and a rank reads slot r (front) and r+1 (back).
Because a piece states its global element index, the noise, and so every bit of w_hat, equals the uncut tensor's.

``FlatShardPlan`` is pure host arithmetic (no device, no process group).  ``ShardedSampler`` runs the device
work through the CUDA library and the two reductions through ``torch.distributed``; the local and the finishing
half of each pass are separate methods so that the reduction can also be supplied by the caller.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

from . import binding
from .binding import Desc


def even_bounds(n_elements: int, world: int, align: int = 32) -> List[int]:
    """Cuts of ``n_elements`` into ``world`` runs of equal length, rounded up to ``align`` elements.  The default, 32
    elements = 64 bytes of BF16, keeps every piece on the kernels that move 64-byte chunks; 8 is the minimum."""
    if n_elements < 0 or world < 1 or align < 8 or align % 8 != 0:
        raise ValueError("even_bounds: n_elements >= 0, world >= 1 and align a multiple of 8 expected")
    per = -(-n_elements // world)
    per = -(-per // align) * align
    return [min(r * per, n_elements) for r in range(world + 1)]


@dataclass(frozen=True)
class Piece:
    """A run of a shard that lies inside ONE group which the shard does not hold completely."""
    local_begin: int          # first element, counted from the start of the rank's buffer
    n_elements: int
    elem_offset: int          # global logical index of that element
    local_group: int          # index of its group in the rank's bt / scale / grad_bt arrays
    slots: Tuple[int, ...]    # cuts inside its group: where its partial result is added
    read_slot: int            # the cut this rank reads the group's result from


@dataclass(frozen=True)
class Body:
    """The whole groups of a shard."""
    local_begin: int
    n_groups: int
    elem_offset: int
    local_group: int          # index of its first group in the rank's arrays


@dataclass(frozen=True)
class FlatShardPlan:
    rank: int
    world: int
    group: int                # elements per group
    begin: int                # global logical index of the shard's first element
    end: int
    first_group: int          # global index of the first group the shard touches
    n_local_groups: int       # groups it touches (entries of the rank's bt / scale / grad_bt arrays)
    body: Optional[Body]
    pieces: Tuple[Piece, ...]  # 0, 1 or 2

    @property
    def n_elements(self) -> int:
        return self.end - self.begin

    @property
    def n_slots(self) -> int:
        return self.world + 1


def plan_flat_shard(n_elements: int, group: int, rank: int, world: int, bounds: Optional[Sequence[int]] = None,
                    elem_offset: int = 0) -> FlatShardPlan:
    """Plan for rank ``rank``.  ``bounds`` (W+1 non-decreasing cuts from 0 to n_elements, multiples of 8) defaults to
    ``even_bounds``; ``elem_offset`` is the logical index of the tensor's element 0 (a multiple of ``group``)."""
    if group < 8 or group % 8 != 0:
        raise ValueError("plan_flat_shard: group must be a positive multiple of 8")
    if n_elements % group != 0:
        raise ValueError("plan_flat_shard: whole groups expected (n_elements a multiple of group)")
    if elem_offset % group != 0:
        raise ValueError("plan_flat_shard: elem_offset must be a multiple of group")
    if not 0 <= rank < world:
        raise ValueError("plan_flat_shard: rank outside [0, world)")
    bounds = even_bounds(n_elements, world) if bounds is None else list(bounds)
    if len(bounds) != world + 1 or bounds[0] != 0 or bounds[-1] != n_elements:
        raise ValueError("plan_flat_shard: bounds must run from 0 to n_elements in world + 1 entries")
    if any(b % 8 != 0 for b in bounds) or any(a > b for a, b in zip(bounds[:-1], bounds[1:])):
        raise ValueError("plan_flat_shard: bounds must be non-decreasing multiples of 8")

    begin, end = bounds[rank], bounds[rank + 1]
    if begin == end:
        return FlatShardPlan(rank, world, group, begin, end, begin // group, 0, None, ())

    def cuts_inside(g: int) -> Tuple[int, ...]:
        return tuple(k for k in range(1, world) if bounds[k] % group != 0 and bounds[k] // group == g)

    first_group, last_group = begin // group, (end - 1) // group
    pieces: List[Piece] = []
    body_begin, body_end = begin, end
    if begin % group != 0:                                   # front piece: up to the next group boundary (or the end)
        stop = min(end, (first_group + 1) * group)
        pieces.append(Piece(0, stop - begin, elem_offset + begin, 0, cuts_inside(first_group), rank))
        body_begin = stop
    if end % group != 0 and last_group * group >= body_begin:   # back piece: from the last group boundary
        start = last_group * group
        pieces.append(Piece(start - begin, end - start, elem_offset + start, last_group - first_group,
                            cuts_inside(last_group), rank + 1))
        body_end = start
    body = None
    if body_end > body_begin:
        body = Body(body_begin - begin, (body_end - body_begin) // group, elem_offset + body_begin,
                    body_begin // group - first_group)
    return FlatShardPlan(rank, world, group, begin, end, first_group, last_group - first_group + 1, body, tuple(pieces))


def all_reduce_slots(buf: torch.Tensor, op: str, process_group=None) -> torch.Tensor:
    """The exchange step: an all-reduce of the W+1 cut slots, MAX for maxima, SUM for gradients."""
    import torch.distributed as dist
    dist.all_reduce(buf, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM, group=process_group)
    return buf


class ShardedSampler:
    """Forward and backward sampling of one rank's shard.

    Buffers (all on the rank's GPU): ``w`` / ``w_hat`` / ``grad_w_hat`` BF16 [n_elements of the shard];
    ``bt`` / ``scale`` / ``grad_bt`` FP32 [plan.n_local_groups], entry k for global group plan.first_group + k.  The
    bit-width of a group that two ranks share is held by both and must be equal; its gradient comes back equal.
    """

    def __init__(self, plan: FlatShardPlan, seed: int, process_group=None):
        self.plan = plan
        self.seed = seed
        self.process_group = process_group

    # -- descriptors -------------------------------------------------------------------------------------------
    def _body_desc(self, step: int) -> Desc:
        b = self.plan.body
        return Desc.make(b.n_groups, self.plan.group, 1, self.plan.group, seed=self.seed, step=step, elem_offset=b.elem_offset)

    def _piece_desc(self, p: Piece, step: int) -> Desc:
        return Desc.make(1, p.n_elements, 1, 0, seed=self.seed, step=step, elem_offset=p.elem_offset)

    def _check(self, elems: Sequence[torch.Tensor], groups: Sequence[torch.Tensor]) -> None:
        for t in elems:
            if t.numel() != self.plan.n_elements or t.dtype != torch.bfloat16 or not t.is_contiguous():
                raise ValueError("ShardedSampler: contiguous BF16 buffers of the shard's length expected")
        for t in groups:
            if t.numel() != self.plan.n_local_groups or t.dtype != torch.float32 or not t.is_contiguous():
                raise ValueError("ShardedSampler: contiguous FP32 arrays of n_local_groups entries expected")

    def _slots(self, device) -> torch.Tensor:
        return torch.zeros(self.plan.n_slots, dtype=torch.float32, device=device)

    def _scatter(self, buf: torch.Tensor, partial: torch.Tensor) -> None:
        for k, p in enumerate(self.plan.pieces):
            for s in p.slots:
                buf[s:s + 1].copy_(partial[k:k + 1])     # a copy, no arithmetic

    # -- forward -----------------------------------------------------------------------------------------------
    def forward_local(self, step: int, w: torch.Tensor, bt: torch.Tensor, w_hat: torch.Tensor, scale: torch.Tensor) -> torch.Tensor:
        """Samples the whole groups and takes the partial maxima of the end pieces.  Returns the slot buffer
        (zeros where this rank has nothing to add: a maximum of magnitudes is never below zero)."""
        self._check([w, w_hat], [bt, scale])
        plan = self.plan
        buf = self._slots(w.device)
        if plan.body is not None:
            b = plan.body
            n = b.n_groups * plan.group
            binding.sample_fwd(self._body_desc(step), w[b.local_begin:b.local_begin + n], bt[b.local_group:b.local_group + b.n_groups],
                               w_hat=w_hat[b.local_begin:b.local_begin + n], scale_out=scale[b.local_group:b.local_group + b.n_groups])
        if plan.pieces:
            partial = torch.empty(len(plan.pieces), dtype=torch.float32, device=w.device)
            for k, p in enumerate(plan.pieces):
                binding.group_absmax(self._piece_desc(p, step), w[p.local_begin:p.local_begin + p.n_elements], absmax=partial[k:k + 1])
            self._scatter(buf, partial)
        return buf

    def forward_finish(self, step: int, reduced: torch.Tensor, w: torch.Tensor, bt: torch.Tensor, w_hat: torch.Tensor,
                       scale: torch.Tensor) -> None:
        """``reduced``: the slot buffers of all ranks under an elementwise maximum."""
        for p in self.plan.pieces:
            g = p.local_group
            binding.scale_from_absmax(reduced[p.read_slot:p.read_slot + 1], bt[g:g + 1], scale=scale[g:g + 1])
            binding.sample_fwd_scaled(self._piece_desc(p, step), w[p.local_begin:p.local_begin + p.n_elements], scale[g:g + 1],
                                      w_hat=w_hat[p.local_begin:p.local_begin + p.n_elements])

    def forward(self, step: int, w: torch.Tensor, bt: torch.Tensor, w_hat: torch.Tensor, scale: torch.Tensor) -> None:
        buf = self.forward_local(step, w, bt, w_hat, scale)
        if self.plan.world > 1:
            all_reduce_slots(buf, "max", self.process_group)
        self.forward_finish(step, buf, w, bt, w_hat, scale)

    # -- backward ----------------------------------------------------------------------------------------------
    def backward_local(self, step: int, grad_w_hat: torch.Tensor, scale: torch.Tensor, grad_bt: torch.Tensor) -> torch.Tensor:
        """Gradients of the whole groups, partial gradients of the end pieces.  Returns the slot buffer."""
        self._check([grad_w_hat], [scale, grad_bt])
        plan = self.plan
        buf = self._slots(grad_w_hat.device)
        if plan.body is not None:
            b = plan.body
            n = b.n_groups * plan.group
            binding.sample_bwd(self._body_desc(step), grad_w_hat[b.local_begin:b.local_begin + n],
                               scale[b.local_group:b.local_group + b.n_groups],
                               grad_bt=grad_bt[b.local_group:b.local_group + b.n_groups])
        if plan.pieces:
            partial = torch.empty(len(plan.pieces), dtype=torch.float32, device=grad_w_hat.device)
            for k, p in enumerate(plan.pieces):
                g = p.local_group
                binding.sample_bwd(self._piece_desc(p, step), grad_w_hat[p.local_begin:p.local_begin + p.n_elements], scale[g:g + 1],
                                   grad_bt=partial[k:k + 1])
            self._scatter(buf, partial)
        return buf

    def backward_finish(self, reduced: torch.Tensor, grad_bt: torch.Tensor) -> None:
        """``reduced``: the slot buffers of all ranks added up."""
        for p in self.plan.pieces:
            grad_bt[p.local_group:p.local_group + 1].copy_(reduced[p.read_slot:p.read_slot + 1])

    def backward(self, step: int, grad_w_hat: torch.Tensor, scale: torch.Tensor, grad_bt: torch.Tensor) -> None:
        buf = self.backward_local(step, grad_w_hat, scale, grad_bt)
        if self.plan.world > 1:
            all_reduce_slots(buf, "sum", self.process_group)
        self.backward_finish(buf, grad_bt)


class ShardedSetSampler:
    """All sharded tensors of a rank in a few launches per pass (the per-tensor sampler above takes several per tensor).

    Every whole-group body and every end piece is one tensor of a multi-tensor plan, so one forward pass of that plan
    samples the bodies for good and leaves, for each end piece, the factor its PART of the group would give:
    fl32(partial max * 2^(1 - b)).  Rounding is monotonic and every rank multiplies by the same power, so the
    maximum of those over the ranks is the factor of the whole group, fl32(max * 2^(1 - b)), bit for bit: the
    factors themselves go through the MAX all-reduce, and a second, small plan re-samples the end pieces with
    them (gws_sample_fwd_scaled_multi).  Backward is one pass of the plan, then the SUM all-reduce.

    ``w[t]`` / ``w_hat[t]`` / ``grad_w_hat[t]``: BF16 shard of tensor t; ``bt[t]``: FP32 [plans[t].n_local_groups].
    The sampler owns the flat ``scale_all`` / ``grad_bt_all`` arrays; ``scale[t]`` and ``grad_bt[t]`` are views.
    """

    def __init__(self, plans: Sequence[FlatShardPlan], seeds: Sequence[int], w: Sequence[torch.Tensor], bt: Sequence[torch.Tensor],
                 w_hat: Sequence[torch.Tensor], grad_w_hat: Optional[Sequence[torch.Tensor]] = None, process_group=None):
        if not (len(plans) == len(seeds) == len(w) == len(bt) == len(w_hat)) or (grad_w_hat is not None and len(grad_w_hat) != len(plans)):
            raise ValueError("ShardedSetSampler: one plan, seed and buffer set per tensor expected")
        if len({p.world for p in plans}) > 1:
            raise ValueError("ShardedSetSampler: every plan must have the same world size")
        self.plans = list(plans)
        self.process_group = process_group
        self.world = plans[0].world if plans else 1
        device = w[0].device if w else torch.device("cuda")
        offsets, total = [], 0
        for p in plans:
            offsets.append(total)
            total += p.n_local_groups
        self.scale_all = torch.zeros(max(total, 1), dtype=torch.float32, device=device)
        self.grad_bt_all = torch.zeros(max(total, 1), dtype=torch.float32, device=device)
        self.scale = [self.scale_all[o:o + p.n_local_groups] for o, p in zip(offsets, plans)]
        self.grad_bt = [self.grad_bt_all[o:o + p.n_local_groups] for o, p in zip(offsets, plans)]
        n_slots = self.world + 1
        self._buf = torch.zeros(max(len(plans) * n_slots, 1), dtype=torch.float32, device=device)

        descs, sel = [], []            # sel: (tensor, element slice, group slice) of every plan entry
        piece_entries = []
        src, dst, grp, read = [], [], [], []
        for t, p in enumerate(plans):
            for buf, name in ((w[t], "w"), (w_hat[t], "w_hat")) + (((grad_w_hat[t], "grad_w_hat"),) if grad_w_hat is not None else ()):
                if buf.numel() != p.n_elements or buf.dtype != torch.bfloat16 or not buf.is_contiguous():
                    raise ValueError(f"ShardedSetSampler: {name}[{t}] must be a contiguous BF16 buffer of the shard's length")
            if bt[t].numel() != p.n_local_groups or bt[t].dtype != torch.float32 or not bt[t].is_contiguous():
                raise ValueError(f"ShardedSetSampler: bt[{t}] must be a contiguous FP32 array of n_local_groups entries")
            if p.body is not None:
                b = p.body
                descs.append(Desc.make(b.n_groups, p.group, 1, p.group, seed=seeds[t], elem_offset=b.elem_offset))
                sel.append((t, slice(b.local_begin, b.local_begin + b.n_groups * p.group), slice(b.local_group, b.local_group + b.n_groups)))
            for piece in p.pieces:
                descs.append(Desc.make(1, piece.n_elements, 1, 0, seed=seeds[t], elem_offset=piece.elem_offset))
                sel.append((t, slice(piece.local_begin, piece.local_begin + piece.n_elements), slice(piece.local_group, piece.local_group + 1)))
                piece_entries.append(len(descs) - 1)
                for s in piece.slots:
                    src.append(offsets[t] + piece.local_group)
                    dst.append(t * n_slots + s)
                grp.append(offsets[t] + piece.local_group)
                read.append(t * n_slots + piece.read_slot)
        index = lambda v: torch.tensor(v, dtype=torch.int64, device=device)
        self._src, self._dst, self._grp, self._read = index(src), index(dst), index(grp), index(read)
        self.n_pieces = len(piece_entries)

        def views(entries):
            pick = lambda bufs, groups: [bufs[t][gs] if groups else bufs[t][es] for t, es, gs in (sel[k] for k in entries)]
            return dict(w=pick(w, False), bt=pick(bt, True), w_hat=pick(w_hat, False), scale=pick(self.scale, True),
                        grad_w_hat=pick(grad_w_hat, False) if grad_w_hat is not None else None,
                        grad_bt=pick(self.grad_bt, True) if grad_w_hat is not None else None)

        everything = list(range(len(descs)))
        self._plan_all = binding.MultiPlan(descs, **views(everything)) if descs else None
        self._plan_pieces = None
        if piece_entries:
            v = views(piece_entries)
            self._plan_pieces = binding.MultiPlan([descs[k] for k in piece_entries], w=v["w"], bt=v["bt"], w_hat=v["w_hat"], scale=v["scale"])

    def _gather(self, values: torch.Tensor) -> torch.Tensor:
        self._buf.zero_()
        if self.n_pieces:
            self._buf.index_copy_(0, self._dst, values.index_select(0, self._src))    # copies only
        return self._buf

    def _scatter(self, reduced: torch.Tensor, values: torch.Tensor) -> None:
        if self.n_pieces:
            values.index_copy_(0, self._grp, reduced.index_select(0, self._read))

    def forward_local(self, step: int) -> torch.Tensor:
        """Returns the slot buffer (W+1 slots per tensor) to be reduced with MAX over the ranks."""
        if self._plan_all is not None:
            self._plan_all.sample_fwd_multi(step)
        return self._gather(self.scale_all)

    def forward_finish(self, step: int, reduced: torch.Tensor) -> None:
        self._scatter(reduced, self.scale_all)
        if self._plan_pieces is not None:
            self._plan_pieces.sample_fwd_scaled_multi(step)

    def forward(self, step: int) -> None:
        buf = self.forward_local(step)
        if self.world > 1:
            all_reduce_slots(buf, "max", self.process_group)
        self.forward_finish(step, buf)

    def backward_local(self, step: int) -> torch.Tensor:
        """Returns the slot buffer to be reduced with SUM over the ranks."""
        if self._plan_all is not None:
            self._plan_all.sample_bwd_multi(step)
        return self._gather(self.grad_bt_all)

    def backward_finish(self, reduced: torch.Tensor) -> None:
        self._scatter(reduced, self.grad_bt_all)

    def backward(self, step: int) -> None:
        buf = self.backward_local(step)
        if self.world > 1:
            all_reduce_slots(buf, "sum", self.process_group)
        self.backward_finish(buf)

    @property
    def launches_per_forward(self) -> int:
        return (self._plan_all.launches_per_pass if self._plan_all is not None else 0) + \
               (self._plan_pieces.launches_per_pass if self._plan_pieces is not None else 0)
