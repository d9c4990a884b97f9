"""One CO3 iteration with the gradient cut into slices of d, one plan (one GPU) per slice.

Every rank holds its slice of every user's gradient and memory.  Conversion, coding, decoding and
averaging are local to a slice; the only exchange is the three moment sums per layer (entries,
sum |a|, sum a^2 of a = g + gamma m, Sec. III (i)): a layer that spans several slices must be
fitted to the sums over ALL its entries, so that every rank derives the same exponent bias and the
same header for it.  That is one all-reduce of n_segments x 3 doubles after the convert pass, and at
t = 0 one more after the statistics pass (with the bias from the current iteration's moments the later
iterations convert under the previous bias and repair the layers whose bias changed after the fit).

Slices are cut at multiples of 4096 elements, so the chunks of the slices together are exactly the
chunks of the unsliced gradient: a user's payload is the slices' payloads one after the other, and
the averaged gradient comes out already sliced.

SliceLayout is plain index arithmetic (no GPU); ShardedPlan wraps a binding.Plan of the slice and
needs the CUDA library.
"""
from typing import List, Optional, Sequence, Tuple

TILE = 4096


def slice_bounds(d: int, world: int) -> List[Tuple[int, int]]:
    """[lo, hi) of every rank: whole 4096-element tiles, as equal as they come (the first
    n_tiles % world ranks hold one tile more); the last slice ends at d."""
    n_tiles = (d + TILE - 1) // TILE
    if world < 1 or n_tiles < world:
        raise ValueError(f"d = {d} has {n_tiles} tiles of {TILE}: too few for {world} slices")
    base, extra = divmod(n_tiles, world)
    out, t = [], 0
    for r in range(world):
        n = base + (1 if r < extra else 0)
        out.append((t * TILE, min(d, (t + n) * TILE)))
        t += n
    return out


class SliceLayout:
    """The slice of rank `rank` and how its segments map to the segments of the whole gradient."""

    def __init__(self, d: int, seg_offsets: Optional[Sequence[int]], rank: int, world: int):
        off = [0, d] if seg_offsets is None else [int(x) for x in seg_offsets]
        self.d, self.rank, self.world = int(d), int(rank), int(world)
        self.n_segments = len(off) - 1
        self.lo, self.hi = slice_bounds(self.d, self.world)[self.rank]
        self.seg_ids: List[int] = []                    # global index of every local segment
        self.local_offsets: List[int] = [0]             # segment offsets of the slice, relative to lo
        for s in range(self.n_segments):
            a, b = max(off[s], self.lo), min(off[s + 1], self.hi)
            if b > a:                                   # an empty segment has no entries anywhere
                self.seg_ids.append(s)
                self.local_offsets.append(b - self.lo)

        self._index = {}                                # seg_ids as an index tensor, per device

    def _ids(self, device):
        import torch
        key = str(device)
        if key not in self._index:
            self._index[key] = torch.as_tensor(self.seg_ids, dtype=torch.int64, device=device)
        return self._index[key]

    def to_global(self, local):
        """[S_local][3] -> [n_segments][3], zero where this slice has no part of the segment."""
        import torch
        g = torch.zeros((self.n_segments, 3), dtype=local.dtype, device=local.device)
        g.index_copy_(0, self._ids(local.device), local)
        return g

    def to_local(self, glob):
        return glob.index_select(0, self._ids(glob.device))


def all_reduce_sum(glob, group=None):
    """Sum of the ranks' moment tables, in place (NCCL for CUDA tensors, gloo for CPU ones).  Without
    a process group there is one slice and nothing to add."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(glob, op=dist.ReduceOp.SUM, group=group)
    return glob


class ShardedPlan:
    """The plan of this rank's slice.  encode() runs the iteration with the two all-reduces in
    place; the phase methods (begin / statistics / convert / finish) expose the points where the
    moments are pooled, for callers that exchange them some other way."""

    def __init__(self, d, n_users, exp_bits, mant_bits, seg_offsets, rank, world, ld=None, **plan_kwargs):
        from . import binding
        if plan_kwargs.get("bias_mode", binding.BIAS_LAGGED) not in (binding.BIAS_CURRENT, binding.BIAS_LAGGED):
            raise ValueError("slices pool their moments through the tiled iteration: bias modes 0 and 1 only")
        self.layout = SliceLayout(d, seg_offsets, rank, world)
        self.plan = binding.Plan(self.layout.hi - self.layout.lo, n_users, exp_bits, mant_bits,
                                 self.layout.local_offsets, ld=ld, **plan_kwargs)
        self.U = int(n_users)

    # ---- phases: each returns this slice's sums as a [n_segments][3] table ready to be added up ----
    def begin(self) -> bool:
        return self.plan.tiled_begin()

    def statistics(self, grad, residual, stream=None):
        self.plan.tiled_statistics(grad, residual, 0, self.U, stream)
        return self.layout.to_global(self.plan.moments_export(stream=stream))

    def convert(self, grad, residual, pooled_statistics=None, stream=None):
        if pooled_statistics is not None:
            self.plan.moments_import(self.layout.to_local(pooled_statistics), stream)
        self.plan.tiled_convert(grad, residual, 0, self.U, stream)
        return self.layout.to_global(self.plan.moments_export(stream=stream))

    def finish(self, pooled, out, stream=None):
        self.plan.moments_import(self.layout.to_local(pooled), stream)
        self.plan.tiled_finish(out, stream)

    # ---- the iteration as a rank of a process group runs it ----
    def encode(self, grad, residual, out, group=None):
        """grad, residual: this slice's [U][ld] rows on the current device; all on the current stream."""
        pooled = None
        if self.begin():
            pooled = all_reduce_sum(self.statistics(grad, residual), group)
        pooled = all_reduce_sum(self.convert(grad, residual, pooled), group)
        self.finish(pooled, out)

    def decode_aggregate(self, out, avg=None):
        """The average of this slice: elements [lo, hi) of the averaged gradient."""
        return self.plan.decode_aggregate(out, avg)
