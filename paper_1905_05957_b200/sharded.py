"""DoubleSqueeze with one worker per GPU and the server sharded over the same GPUs.

Rank r holds worker r's error delta^(r), slice r of the server error delta, and a full copy of x.
One iteration (Algorithm 1 with the parameter server spread over the workers, which Section 3.1
allows):

  1. worker pass for row r                        ds_worker_compress_rows
  2. every rank sends slice q of its payload to rank q (an all-to-all of compressed slices: the
     first of the two compressed hops)            exchange_worker_payloads
  3. server pass over slice r of d                ds_server_aggregate_compress_slice (+ update of x on the slice)
  4. every rank sends its slice of the server payload to all the others (an all-gather: the second
     compressed hop)                              exchange_server_payload
  5. update of x on the other slices              ds_apply_update_slice

A top-k server (its threshold is a property of the whole vector) replaces 3-5 by the staged calls
ds_server_topk_slice_begin / _digit / _emit with three all-reduces of a 4096-bin histogram and one
all-gather of four words in between, then an all-gather of the slices' (index, value) lists.

Every step of the arithmetic runs in the library's kernels; this module only says which bytes
move where.  The moves go through a `transport` with two methods, so that the same plan runs over
torch.distributed point-to-point operations (NCCL between GPUs, gloo in the CPU test) and over plain
copies between buffers of one process (the single-GPU check of the arithmetic).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from .workloads import Q

SLICE_ALIGN = 8192          # ds_server_aggregate_compress_slice wants slice starts on this grid
_ELEM_BYTES = {"identity": lambda q: 4.0, "clip": lambda q: (32 - q.bits) / 8}


def slice_bounds(d: int, world: int) -> list[tuple[int, int]]:
    """Contiguous slices of [0, d) on the SLICE_ALIGN grid, as even as that allows; trailing slices may
    be empty when d is small."""
    units = -(-d // SLICE_ALIGN)
    out, start = [], 0
    for r in range(world):
        n_units = units // world + (1 if r < units % world else 0)
        lo = min(start * SLICE_ALIGN, d)
        hi = min((start + n_units) * SLICE_ALIGN, d)
        out.append((lo, hi))
        start += n_units
    return out


def payload_slice_ranges(q: Q, layout_off, lo: int, hi: int) -> list[tuple[int, int]]:
    """Byte ranges (start, length) inside ONE payload that hold entries lo .. hi-1, one per sub-array,
    for the operators whose payload is laid out along d.  lo is a multiple of SLICE_ALIGN."""
    if hi <= lo:
        return []
    if q.op == "sign1":
        return [(layout_off[0] + lo // 8, 4 * (-(-hi // 32)) - lo // 8),
                (layout_off[1] + 4 * (lo // q.chunk), 4 * (-(-hi // q.chunk) - lo // q.chunk))]
    if q.op == "qsgd":
        return [(layout_off[0] + lo, hi - lo),
                (layout_off[1] + lo // 8, 4 * (-(-hi // 32)) - lo // 8),
                (layout_off[2] + 4 * (lo // q.chunk), 4 * (-(-hi // q.chunk) - lo // q.chunk))]
    if q.op == "clip":
        b = (32 - q.bits) // 8
        return [(layout_off[0] + b * lo, b * (hi - lo))]
    if q.op == "identity":
        return [(layout_off[0] + 4 * lo, 4 * (hi - lo))]
    if q.op == "rsparse":
        S, per = q.keep_one_in, q.chunk // q.keep_one_in
        c_lo, c_hi = lo // q.chunk, -(-hi // q.chunk)          # whole chunks: a short last chunk still has `per` slots
        return [(layout_off[0] + 4 * (lo // S), 4 * (c_hi * per - lo // S)),
                (layout_off[1] + 4 * c_lo, 4 * (c_hi - c_lo))]
    raise ValueError(f"operator {q.op!r} has no slices along d")


def _gather_bytes(buf: torch.Tensor, base: int, ranges) -> torch.Tensor:
    return torch.cat([buf[base + s: base + s + n] for s, n in ranges]) if ranges else buf[:0]


def _scatter_bytes(buf: torch.Tensor, base: int, ranges, data: torch.Tensor):
    at = 0
    for s, n in ranges:
        buf[base + s: base + s + n].copy_(data[at: at + n])
        at += n


@dataclass
class ShardPlan:
    """What rank `rank` of `world` sends and receives in one iteration."""
    world: int
    rank: int
    d: int
    worker_q: Q
    server_q: Q
    worker_off: tuple       # sub-array offsets of a worker payload
    worker_stride: int
    server_off: tuple

    def __post_init__(self):
        self.bounds = slice_bounds(self.d, self.world)

    # -- hop 1: worker payload slices, rank i -> rank q ------------------------------------------
    def worker_send(self, worker_payload: torch.Tensor) -> list[torch.Tensor]:
        """For every destination q: slice q of this rank's own payload (row `rank`)."""
        base = self.rank * self.worker_stride
        return [_gather_bytes(worker_payload, base, payload_slice_ranges(self.worker_q, self.worker_off, *self.bounds[q]))
                for q in range(self.world)]

    def worker_recv_sizes(self) -> list[int]:
        n = sum(r[1] for r in payload_slice_ranges(self.worker_q, self.worker_off, *self.bounds[self.rank]))
        return [n] * self.world

    def worker_place(self, worker_payload: torch.Tensor, received: list[torch.Tensor]):
        """received[i] = slice `rank` of worker i's payload -> row i of the local payload buffer."""
        ranges = payload_slice_ranges(self.worker_q, self.worker_off, *self.bounds[self.rank])
        for i, data in enumerate(received):
            if i != self.rank:
                _scatter_bytes(worker_payload, i * self.worker_stride, ranges, data)

    # -- hop 2: server payload slices, rank q -> everyone ----------------------------------------
    def server_send(self, server_payload: torch.Tensor) -> torch.Tensor:
        return _gather_bytes(server_payload, 0, payload_slice_ranges(self.server_q, self.server_off, *self.bounds[self.rank]))

    def server_recv_sizes(self) -> list[int]:
        return [sum(r[1] for r in payload_slice_ranges(self.server_q, self.server_off, *self.bounds[q]))
                for q in range(self.world)]

    def server_place(self, server_payload: torch.Tensor, received: list[torch.Tensor]):
        for q, data in enumerate(received):
            if q != self.rank:
                _scatter_bytes(server_payload, 0, payload_slice_ranges(self.server_q, self.server_off, *self.bounds[q]), data)


class DistTransport:
    """The two hops over torch.distributed point-to-point operations (works with NCCL and gloo)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self._staging: dict = {}
        self.bytes_sent = 0          # payload bytes this rank has put on the wire so far

    def _recv_buffers(self, recv_sizes: list[int], device) -> list[torch.Tensor]:
        """Receive staging, allocated once per shape of exchange and reused every iteration."""
        key = (tuple(recv_sizes), str(device))
        if key not in self._staging:
            self._staging[key] = [torch.empty(n, dtype=torch.uint8, device=device) for n in recv_sizes]
        return list(self._staging[key])

    def _exchange(self, send: list[torch.Tensor], recv_sizes: list[int]) -> list[torch.Tensor]:
        dist = self.dist
        recv = self._recv_buffers(recv_sizes, send[0].device)
        self.bytes_sent += sum(int(t.numel()) for q, t in enumerate(send) if q != self.rank)
        ops = []
        for q in range(self.world):
            if q == self.rank:
                recv[q] = send[q]
                continue
            if send[q].numel():
                ops.append(dist.P2POp(dist.isend, send[q].contiguous(), q, self.group))
            if recv_sizes[q]:
                ops.append(dist.P2POp(dist.irecv, recv[q], q, self.group))
        if ops:
            for w in dist.batch_isend_irecv(ops):
                w.wait()
        return recv

    def all_to_all(self, send: list[torch.Tensor], recv_sizes: list[int]) -> list[torch.Tensor]:
        return self._exchange(send, recv_sizes)

    def all_gather(self, mine: torch.Tensor, recv_sizes: list[int]) -> list[torch.Tensor]:
        return self._exchange([mine] * self.world, recv_sizes)

    def all_reduce_sum(self, t: torch.Tensor):
        """In-place sum over the ranks (the 4096-bin histograms of a top-k over slices)."""
        self.bytes_sent += int(t.numel() * t.element_size())
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)

    def all_gather_small(self, t: torch.Tensor) -> list[torch.Tensor]:
        """Every rank's copy of a few words."""
        out = [torch.empty_like(t) for _ in range(self.world)]
        self.bytes_sent += int(t.numel() * t.element_size()) * (self.world - 1)
        self.dist.all_gather(out, t, group=self.group)
        return out


class ShardedDoubleSqueeze:
    """One rank of the one-worker-per-GPU deployment (see the module text).  `ds` is this rank's
    DoubleSqueeze instance, created with n = world and, to hold the error of its own worker only,
    delta_w_rows = 1 (an instance with all n rows works too and uses row `rank`)."""

    def __init__(self, ds, rank: int, world: int):
        if ds.n != world:
            raise ValueError("the instance must be created with n = world size")
        self.ds, self.rank, self.world = ds, rank, world
        self.plan = ShardPlan(world, rank, ds.d, ds.worker_q, ds.server_q, tuple(ds.worker_layout.off),
                              int(ds.worker_layout.stride), tuple(ds.server_layout.off))
        self.lo, self.hi = self.plan.bounds[rank]

    def worker_pass(self, g_row: torch.Tensor, t: int):
        self.ds.worker_compress_rows(g_row.reshape(1, -1), self.rank, t)

    def exchange_worker_payloads(self, transport):
        p = self.plan
        got = transport.all_to_all(p.worker_send(self.ds.worker_payload), p.worker_recv_sizes())
        p.worker_place(self.ds.worker_payload, got)

    def server_pass(self, t: int):
        if self.hi > self.lo:
            self.ds.server_aggregate_compress_slice(t, self.lo, self.hi, fuse_apply=True)

    def exchange_server_payload(self, transport):
        p = self.plan
        got = transport.all_gather(p.server_send(self.ds.server_payload), p.server_recv_sizes())
        p.server_place(self.ds.server_payload, got)

    def apply_other_slices(self):
        for q, (lo, hi) in enumerate(self.plan.bounds):
            if q != self.rank and hi > lo:
                self.ds.apply_update_slice(lo, hi)

    # -- a top-k server: its threshold belongs to the whole vector, so the pass is cut into stages between
    # -- which the slices' histograms are added up over the ranks ------------------------------------------
    @property
    def server_is_topk(self) -> bool:
        return self.ds.server_q.op == "topk"

    def _hists(self):
        if not hasattr(self, "_hist"):
            dev = self.ds.server_payload.device
            self._hist = [torch.zeros(4096, dtype=torch.int32, device=dev) for _ in range(2)]
        return self._hist

    def topk_begin(self, t: int) -> torch.Tensor:
        """Stage 1: v on the own slice and its first-digit histogram (to be summed over the ranks)."""
        h = self._hists()[0]
        if self.hi > self.lo:
            self.ds.server_topk_slice_begin(t, self.lo, self.hi, h)
        else:
            h.zero_()
        return h

    def topk_digit(self, level: int) -> torch.Tensor:
        """Stage 2, level 1..3: consumes the summed histogram of the previous stage, returns this slice's next one
        (after level 3: above, ties, r, tau in its first four words)."""
        a, b = self._hists()
        src, dst = (a, b) if level % 2 == 1 else (b, a)
        if self.hi > self.lo:
            self.ds.server_topk_slice_digit(level, self.lo, self.hi, src, dst)
        else:
            dst.zero_()          # an empty slice holds nothing; r and tau come from the others
        return dst

    @staticmethod
    def topk_shares(totals: list[tuple[int, int]], r: int) -> list[tuple[int, int, int]]:
        """From every slice's (entries above tau, entries equal to tau) and the vector's tie quota r: per slice
        (ties to keep, entries kept, first output slot).  Ties go to lower indices, i.e. to earlier slices, first."""
        out, ties_before, slot = [], 0, 0
        for above, ties in totals:
            keep = max(0, min(ties, r - ties_before))
            out.append((keep, above + keep, slot))
            ties_before += ties
            slot += above + keep
        return out

    def topk_emit(self, share: tuple[int, int, int]):
        keep, count, first = share
        if self.hi > self.lo:
            self.ds.server_topk_slice_emit(self.lo, self.hi, keep, count, first, fuse_apply=True)

    def topk_parts(self, share: tuple[int, int, int]) -> tuple[torch.Tensor, torch.Tensor]:
        """The own slice's part of the server payload: (indices, values) as byte tensors."""
        _, count, first = share
        v = self.ds.server_views()
        return v["idx"][first:first + count].view(torch.uint8), v["val"][first:first + count].view(torch.uint8)

    def topk_place(self, q: int, share: tuple[int, int, int], idx_bytes: torch.Tensor, val_bytes: torch.Tensor):
        """Rank q's part into the local payload, and its update of x."""
        _, count, first = share
        if q == self.rank or count == 0:
            return
        v = self.ds.server_views()
        v["idx"][first:first + count].view(torch.uint8).copy_(idx_bytes)
        v["val"][first:first + count].view(torch.uint8).copy_(val_bytes)
        self.ds.apply_update_sparse_range(first, count)

    def server_topk(self, t: int, transport):
        """The whole top-k server pass of this rank over a transport with collectives."""
        h = self.topk_begin(t)
        for level in (1, 2, 3):
            transport.all_reduce_sum(h)
            h = self.topk_digit(level)
        words = [w.cpu() for w in transport.all_gather_small(h[:4].clone())]
        r = max(int(w[2]) for w in words)                       # the same on every rank that holds a slice
        shares = self.topk_shares([(int(w[0]), int(w[1])) for w in words], r)
        self.topk_emit(shares[self.rank])
        idx_b, val_b = self.topk_parts(shares[self.rank])
        sizes = [4 * c for _, c, _ in shares]
        got_idx = transport.all_gather(idx_b, sizes)
        got_val = transport.all_gather(val_b, sizes)
        for q in range(self.world):
            self.topk_place(q, shares[q], got_idx[q], got_val[q])

    def step(self, g_row: torch.Tensor, t: int, transport):
        self.worker_pass(g_row, t)
        self.exchange_worker_payloads(transport)
        if self.server_is_topk:
            self.server_topk(t, transport)
            return
        self.server_pass(t)
        self.exchange_server_payload(transport)
        self.apply_other_slices()


def step_in_process(ranks: list[ShardedDoubleSqueeze], g: torch.Tensor, t: int):
    """One iteration for all ranks held by ONE process (their buffers on one device): the five phases
    run rank after rank, and the two hops are plain copies.  Checks the arithmetic of the sharded
    form without a second GPU; no kernel here waits for another."""
    world = len(ranks)
    for r in ranks:
        r.worker_pass(g[r.rank], t)
    sends = [r.plan.worker_send(r.ds.worker_payload) for r in ranks]
    for r in ranks:
        r.plan.worker_place(r.ds.worker_payload, [sends[i][r.rank] for i in range(world)])
    if ranks[0].server_is_topk:
        hs = [r.topk_begin(t) for r in ranks]
        for level in (1, 2, 3):
            total = torch.stack(hs).sum(dim=0, dtype=torch.int32)      # what the all-reduce would leave on every rank
            for h in hs:
                h.copy_(total)
            hs = [r.topk_digit(level) for r in ranks]
        words = [h[:4].cpu() for h in hs]
        rr = max(int(w[2]) for w in words)
        shares = ShardedDoubleSqueeze.topk_shares([(int(w[0]), int(w[1])) for w in words], rr)
        for r in ranks:
            r.topk_emit(shares[r.rank])
        parts = [r.topk_parts(shares[r.rank]) for r in ranks]
        for r in ranks:
            for q in range(world):
                r.topk_place(q, shares[q], parts[q][0], parts[q][1])
        return
    for r in ranks:
        r.server_pass(t)
    slices = [r.plan.server_send(r.ds.server_payload) for r in ranks]
    for r in ranks:
        r.plan.server_place(r.ds.server_payload, slices)
    for r in ranks:
        r.apply_other_slices()
