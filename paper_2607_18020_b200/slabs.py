"""One grid split into slabs along its slowest axis (x), one slab per rank.

The operators have exactly one exchange step when a grid is split: a node's residual reads the
fields `radius` planes to either side, and the gather-form adjoint reads the upstream arrays
`radius` planes to either side (and, where the Jacobian depends on the fields, the fields at
those rows' own neighbours).  So per step a rank

  1. receives 2*radius halo planes of every field from each x neighbour,
  2. runs the forward kernel on the planes [x0 - radius, x1 + radius): rows on its own planes,
  3. receives radius halo planes of every residual array,
  4. runs the adjoint kernel on the planes [x0 - 2 radius, x1 + 2 radius): with the interior-axis
     rule (rows where the stencil fits) the upstream arrays are honoured on [x0 - radius,
     x1 + radius), which is what the gradients on the own planes [x0, x1) need,
  5. adds up the ranks' shares of the loss (nresiduals + 1 doubles, one all-reduce posted before
     the adjoint so that it runs beside it): the forward call divides by the row count of the
     WHOLE grid (fpde_fwd_rows), so no loss arithmetic is done outside the library.

Every array is stored once per rank with the widest halo; the forward call is handed a
sub-range of planes (contiguous, because x is the slowest axis), so nothing is copied locally.
An operator whose x axis is an interior axis is its own slab form (at the two ends of the
domain the halo is simply absent); the periodic operators (unsteady Navier-Stokes, Gray-Scott) have
slab forms with a non-periodic x axis (`ns_3d_t_xslab`, `grayscott_2d_xslab`).  The kernels are the single-GPU kernels; this
module only plans the ranges and moves the halo planes (torch.distributed point-to-point, or
plain copies when several slabs live in one process).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence, Tuple

from . import workloads as W

# operator on the whole grid -> operator one slab runs
SLAB_OP = {
    W.POISSON_2D: W.POISSON_2D,
    W.HELMHOLTZ_3D_O4: W.HELMHOLTZ_3D_O4,
    W.NS_2D_STEADY: W.NS_2D_STEADY,
    W.NS_3D_STEADY: W.NS_3D_STEADY,
    W.NS_3D_T: W.NS_3D_T_XSLAB,
    W.GRAYSCOTT_2D: W.GRAYSCOTT_2D_XSLAB,
}
RADIUS = {W.POISSON_2D: 1, W.HELMHOLTZ_3D_O4: 2, W.NS_2D_STEADY: 1, W.NS_3D_STEADY: 1, W.NS_3D_T: 1, W.GRAYSCOTT_2D: 1}


@dataclass(frozen=True)
class Transfer:
    """`count` planes starting at global plane `start`, owned by `peer`, land at local plane `dst`."""
    peer: int
    start: int
    count: int
    dst: int


@dataclass(frozen=True)
class SlabPlan:
    op: str                    # operator on the whole grid
    shape: Tuple[int, ...]     # whole grid
    world: int
    rank: int

    @property
    def local_op(self) -> str:
        return SLAB_OP[self.op]

    @property
    def radius(self) -> int:
        return RADIUS[self.op]

    @property
    def periodic(self) -> bool:
        return W.CONFIGS[next(k for k, c in W.CONFIGS.items() if c["op"] == self.op)]["bc"][0] == W.PERIODIC

    def owned_of(self, rank: int) -> Tuple[int, int]:
        n0 = self.shape[0]
        return rank * n0 // self.world, (rank + 1) * n0 // self.world

    @property
    def owned(self) -> Tuple[int, int]:
        return self.owned_of(self.rank)

    def _range(self, halo: int) -> Tuple[int, int]:
        x0, x1 = self.owned
        if self.periodic:
            return x0 - halo, x1 + halo                      # may run past the ends: planes wrap
        return max(0, x0 - halo), min(self.shape[0], x1 + halo)

    @property
    def wide(self) -> Tuple[int, int]:
        """Planes every local array holds."""
        return self._range(2 * self.radius)

    @property
    def tight(self) -> Tuple[int, int]:
        """Planes the forward kernel is run on."""
        return self._range(self.radius)

    @property
    def local_shape(self) -> Tuple[int, ...]:
        w0, w1 = self.wide
        return (w1 - w0,) + tuple(self.shape[1:])

    @property
    def tight_shape(self) -> Tuple[int, ...]:
        t0, t1 = self.tight
        return (t1 - t0,) + tuple(self.shape[1:])

    def local_of(self, plane: int) -> int:
        """Local plane index of a global plane index of this rank's wide range."""
        return plane - self.wide[0]

    def owner(self, plane: int) -> int:
        n0 = self.shape[0]
        g = plane % n0
        for r in range(self.world):
            a, b = self.owned_of(r)
            if a <= g < b:
                return r
        raise AssertionError(plane)

    def check(self):
        if self.op not in SLAB_OP:
            raise ValueError("operator %s has no slab form" % self.op)
        for r in range(self.world):
            a, b = self.owned_of(r)
            if b - a < 2 * self.radius:
                raise ValueError("slab of rank %d has %d planes; at least %d are needed" % (r, b - a, 2 * self.radius))
        if self.periodic and self.shape[0] < 4 * self.radius:
            raise ValueError("grid too short along x")

    def halo_transfers(self, halo: int) -> List[Transfer]:
        """What this rank receives to fill `halo` planes beyond each end of its own planes: runs of
        consecutive planes with one owner, in ascending local order."""
        x0, x1 = self.owned
        lo, hi = self._range(halo)
        out: List[Transfer] = []
        for a, b in ((lo, x0), (x1, hi)):
            g = a
            while g < b:
                peer = self.owner(g)
                pa, pb = self.owned_of(peer)
                start = g % self.shape[0]
                count = min(b - g, pb - start)
                out.append(Transfer(peer, start, count, self.local_of(g)))
                g += count
        return out

    def sends(self, halo: int) -> List[Tuple[int, Transfer]]:
        """(destination rank, transfer as seen by the destination) for everything this rank owns
        that another rank's halo needs, in the destination's order."""
        out = []
        for r in range(self.world):
            plan = SlabPlan(self.op, self.shape, self.world, r)
            for t in plan.halo_transfers(halo):
                if t.peer == self.rank:
                    out.append((r, t))
        return out


def plans(op: str, shape: Sequence[int], world: int) -> List[SlabPlan]:
    ps = [SlabPlan(op, tuple(int(s) for s in shape), world, r) for r in range(world)]
    ps[0].check()
    return ps


def exchange_local(plan_list: Sequence[SlabPlan], arrays: Sequence, halo: int):
    """Fill the halo planes when all slabs live in this process.  arrays[rank] is either the list of
    that rank's local arrays (wide range, planes on axis 0) or ONE stacked tensor of them (arrays on
    axis 0, planes on axis 1): with the stacked form a transfer is one strided copy for all arrays."""
    for plan in plan_list:
        for t in plan.halo_transfers(halo):
            src_plan = plan_list[t.peer]
            s = src_plan.local_of(t.start)
            dst_set, src_set = arrays[plan.rank], arrays[t.peer]
            if hasattr(dst_set, "dim"):
                dst_set[:, t.dst:t.dst + t.count].copy_(src_set[:, s:s + t.count])
            else:
                for dst_arr, src_arr in zip(dst_set, src_set):
                    dst_arr[t.dst:t.dst + t.count].copy_(src_arr[s:s + t.count])


class Exchange:
    """A halo exchange that has been posted: `wait()` returns once every halo plane has landed."""

    def __init__(self, reqs):
        self.reqs = reqs

    def wait(self):
        for req in self.reqs:
            req.wait()
        self.reqs = []


def post_exchange(plan: SlabPlan, arrays, halo: int, dist) -> Exchange:
    """Post the receives and sends that fill `halo` planes beyond each end of this rank's own planes
    (torch.distributed point-to-point; both sides enumerate the transfers in the same order) and
    return at once: work that does not read the halo planes can be queued before `wait()`.
    `arrays`: the list of this rank's local arrays, or one stacked tensor of them.  Planes a rank needs
    from itself (one rank on a periodic axis) are copied; they never overlap the planes they come from."""
    stacked = hasattr(arrays, "dim")
    per_array = list(arrays.unbind(0)) if stacked else list(arrays)
    ops = []
    for t in plan.halo_transfers(halo):
        if t.peer == plan.rank:
            s = plan.local_of(t.start)
            if stacked:
                arrays[:, t.dst:t.dst + t.count].copy_(arrays[:, s:s + t.count])
            else:
                for arr in per_array:
                    arr[t.dst:t.dst + t.count].copy_(arr[s:s + t.count])
        else:
            for arr in per_array:
                ops.append(dist.P2POp(dist.irecv, arr[t.dst:t.dst + t.count], t.peer))
    for dst, t in plan.sends(halo):
        if dst == plan.rank:
            continue
        s = plan.local_of(t.start)
        for arr in per_array:
            ops.append(dist.P2POp(dist.isend, arr[s:s + t.count], dst))
    return Exchange(dist.batch_isend_irecv(ops) if ops else [])


def exchange_dist(plan: SlabPlan, arrays, halo: int, dist):
    """post_exchange + wait."""
    post_exchange(plan, arrays, halo, dist).wait()


class SlabRank:
    """The arrays and kernel calls of one slab."""

    def __init__(self, torch, B, plan: SlabPlan, spacing, coeffs, device="cuda"):
        plan.check()
        self.torch, self.B, self.plan = torch, B, plan
        self.spacing, self.coeffs = tuple(spacing), tuple(coeffs)
        meta = W.OP_META[plan.op]
        self.nf, self.ns, self.ne = len(meta["fields"]), len(meta["sources"]), len(meta["residuals"])
        self.bc = W.CONFIGS[next(k for k, c in W.CONFIGS.items() if c["op"] == plan.local_op)]["bc"]
        ls = plan.local_shape
        # the arrays of one kind are slices of ONE tensor, so that a halo transfer between slabs of
        # one process is a single strided copy for all of them
        stack = lambda k: torch.zeros((max(k, 1),) + tuple(ls), dtype=torch.float32, device=device)
        self.field_stack, self.res_stack = stack(self.nf), stack(self.ne)
        self.fields = list(self.field_stack.unbind(0))[:self.nf]
        self.res = list(self.res_stack.unbind(0))[:self.ne]
        new = lambda: torch.zeros(ls, dtype=torch.float32, device=device)
        self.sources = [new() for _ in range(self.ns)]
        self.grads = [new() for _ in range(self.nf)]
        self.loss = torch.zeros(self.ne + 1, dtype=torch.float64, device=device)
        self.ws = torch.empty(max(16, B.workspace_bytes(plan.local_op, plan.tight_shape)), dtype=torch.uint8, device=device) \
            if device != "cpu" else None
        self.rows_global = B.row_count(plan.op, plan.shape) if device != "cpu" else 0
        self.rows_local = B.row_count(plan.local_op, plan.tight_shape) if device != "cpu" else 0

    def _owned_slice(self):
        x0, x1 = self.plan.owned
        return slice(self.plan.local_of(x0), self.plan.local_of(x1))

    def _tight_slice(self):
        t0, t1 = self.plan.tight
        return slice(self.plan.local_of(t0), self.plan.local_of(t1))

    def owned(self, arrays):
        s = self._owned_slice()
        return [a[s] for a in arrays]

    def load_owned(self, fields, sources):
        """Copy this rank's planes of whole-grid arrays (numpy or torch) into the local arrays."""
        x0, x1 = self.plan.owned
        for dst, src in zip(self.owned(self.fields) + self.owned(self.sources), list(fields) + list(sources)):
            dst.copy_(self.torch.as_tensor(src[x0:x1]))

    def fwd(self, stream=None):
        """Forward kernel on the tight range.  The loss vector is this slab's share of the whole
        grid's loss (the library divides by the whole grid's row count), so shares add up."""
        s = self._tight_slice()
        p = self.plan
        self.B.fpde_fwd_rows(p.local_op, [a[s] for a in self.fields], [a[s] for a in self.sources], [a[s] for a in self.res],
                             self.loss, p.tight_shape, self.spacing, self.coeffs, self.bc, self.ws, self.rows_global, stream)

    def bwd(self, stream=None):
        p = self.plan
        self.B.fpde_bwd(p.local_op, self.fields, self.res, [2.0 / self.rows_global] * self.ne, self.grads,
                        p.local_shape, self.spacing, self.coeffs, self.bc, None, stream)

    # ---- launches over ranges of planes: the planes away from the halos first, while the halo
    # ---- planes are still in flight, then the planes next to them -------------------------------
    def chunk_plan(self):
        """Chunk ranges of the ranged launches, or None if the operator has no ranged launches or the
        slab is too short: ((K, lo, hi) forward, (K, lo, hi) adjoint) with K chunks in all, of which
        [lo, hi) neither hold nor read a plane that a halo exchange fills.  Forward: the field halos
        are the outer `radius` planes of the tight range.  Adjoint: the residual halos are planes
        [radius, 2 radius) and their mirror image of the wide range (field halos are complete by then)."""
        p = self.plan
        R = p.radius
        out = []
        for n, halo_end in ((p.tight_shape[0], R), (p.local_shape[0], 2 * R)):
            P = self.B.plane_chunk(p.local_op, (n,) + tuple(p.shape[1:]))
            if P <= 0:
                return None
            K = -(-n // P)
            inner = [c for c in range(K) if c * P - R >= halo_end and min((c + 1) * P, n) - 1 + R < n - halo_end]
            if not inner:
                return None
            out.append((K, inner[0], inner[-1] + 1))
        return tuple(out)

    def fwd_inner(self, plan, stream=None):
        self._fwd_chunks(plan[1], plan[2], False, stream)

    def fwd_edges(self, plan, stream=None):
        K, lo, hi = plan
        self._fwd_chunks(0, lo, hi == K, stream)
        if hi < K:
            self._fwd_chunks(hi, K, True, stream)

    def _fwd_chunks(self, lo, hi, finish, stream):
        s = self._tight_slice()
        p = self.plan
        self.B.fpde_fwd_chunks(p.local_op, [a[s] for a in self.fields], [a[s] for a in self.sources], [a[s] for a in self.res],
                               self.loss, p.tight_shape, self.spacing, self.coeffs, self.bc, self.ws, self.rows_global,
                               lo, hi, finish, stream)

    def bwd_inner(self, plan, stream=None):
        self._bwd_chunks(plan[1], plan[2], stream)

    def bwd_edges(self, plan, stream=None):
        K, lo, hi = plan
        self._bwd_chunks(0, lo, stream)
        if hi < K:
            self._bwd_chunks(hi, K, stream)

    def _bwd_chunks(self, lo, hi, stream):
        p = self.plan
        self.B.fpde_bwd_chunks(p.local_op, self.fields, self.res, [2.0 / self.rows_global] * self.ne, self.grads,
                               p.local_shape, self.spacing, self.coeffs, self.bc, lo, hi, stream)


def step_local(ranks: Sequence[SlabRank]):
    """One loss + gradient step over slabs that all live in this process (one GPU standing in for
    several: the kernels of different slabs run one after the other, nothing waits on anything).
    Returns the loss vector of the whole grid: the sum of the slabs' shares."""
    plan_list = [r.plan for r in ranks]
    R = plan_list[0].radius
    exchange_local(plan_list, [r.field_stack for r in ranks], 2 * R)
    for r in ranks:
        r.fwd()
    exchange_local(plan_list, [r.res_stack for r in ranks], R)
    for r in ranks:
        r.bwd()
    loss = ranks[0].loss.clone()
    for r in ranks[1:]:
        loss += r.loss
    return loss


def step_dist(rank: SlabRank, dist, overlap=None):
    """The same step with one slab per process.  With `overlap` (default: whenever there is more than
    one rank and the operator has launches over ranges of planes) the chunks of planes away from the
    halos are queued while the halo planes are in flight and the chunks next to the halos after they
    have landed; on one rank there is nothing to overlap and three launches per direction only cost
    their tails (measured: 0.59 against 0.50 ms per step).  The all-reduce of the loss shares is
    posted before the adjoint is queued, so it runs beside it."""
    R = rank.plan.radius
    if overlap is None:
        overlap = rank.plan.world > 1
    chunks = rank.chunk_plan() if overlap else None
    ex = post_exchange(rank.plan, rank.field_stack, 2 * R, dist)
    if chunks is not None:
        # the chunks of planes away from the halos run while the halo planes are in flight
        rank.fwd_inner(chunks[0])
        ex.wait()
        rank.fwd_edges(chunks[0])
    else:
        ex.wait()
        rank.fwd()
    ex = post_exchange(rank.plan, rank.res_stack, R, dist)
    loss = rank.loss.clone()
    work = dist.all_reduce(loss, op=dist.ReduceOp.SUM, async_op=True) if rank.plan.world > 1 else None
    if chunks is not None:
        rank.bwd_inner(chunks[1])
        ex.wait()
        rank.bwd_edges(chunks[1])
    else:
        ex.wait()
        rank.bwd()
    if work is not None:
        work.wait()
    return loss
