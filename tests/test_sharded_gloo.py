"""The two compressed hops of the one-worker-per-GPU form over torch.distributed (gloo, CPU): every
rank must end with exactly the bytes that plain copies between the ranks' buffers would give."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1905_05957_b200 import binding as b
from paper_1905_05957_b200.sharded import DistTransport, ShardPlan, payload_slice_ranges, slice_bounds
from paper_1905_05957_b200.workloads import Q

D = 3 * 8192 + 777
WQ, SQ = Q("qsgd", chunk=2048, levels=255), Q("sign1", chunk=4096)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _plan(rank: int, world: int) -> tuple[ShardPlan, int, int]:
    cfg = b.make_config(world, D, 0.1, WQ, SQ, 1)
    wl, sl = b.get_layout(cfg, 0), b.get_layout(cfg, 1)
    return ShardPlan(world, rank, D, WQ, SQ, tuple(wl.off), int(wl.stride), tuple(sl.off)), int(wl.stride), int(sl.stride)


def _buffers(rank: int, world: int, wstride: int, sstride: int):
    """What rank `rank` holds before the hops: its own payload row and its own server slice carry
    data, everything else is a marker byte."""
    gen = torch.Generator().manual_seed(100 + rank)
    wp = torch.full((world * wstride,), 0xEE, dtype=torch.uint8)
    wp[rank * wstride:(rank + 1) * wstride] = torch.randint(0, 256, (wstride,), generator=gen, dtype=torch.uint8)
    sp = torch.randint(0, 256, (sstride,), generator=gen, dtype=torch.uint8)
    return wp, sp


def _rank_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    plan, wstride, sstride = _plan(rank, world)
    wp, sp = _buffers(rank, world, wstride, sstride)
    tr = DistTransport()
    plan.worker_place(wp, tr.all_to_all(plan.worker_send(wp), plan.worker_recv_sizes()))
    plan.server_place(sp, tr.all_gather(plan.server_send(sp), plan.server_recv_sizes()))
    dist.barrier()
    out.put((rank, wp.numpy().tobytes(), sp.numpy().tobytes()))
    dist.destroy_process_group()


def test_hops_over_gloo_equal_plain_copies():
    world, port = 3, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = {}
    for _ in range(world):
        r, wp, sp = out.get(timeout=180)
        got[r] = (torch.frombuffer(bytearray(wp), dtype=torch.uint8), torch.frombuffer(bytearray(sp), dtype=torch.uint8))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    plans = [_plan(r, world) for r in range(world)]
    before = [_buffers(r, world, plans[r][1], plans[r][2]) for r in range(world)]
    bounds = slice_bounds(D, world)
    for r in range(world):
        plan, wstride, _ = plans[r]
        want_wp, want_sp = before[r][0].clone(), before[r][1].clone()
        for i in range(world):          # slice r of worker i's payload lands in row i of rank r
            for s, n in payload_slice_ranges(WQ, plan.worker_off, *bounds[r]):
                want_wp[i * wstride + s: i * wstride + s + n] = before[i][0][i * wstride + s: i * wstride + s + n]
        for q in range(world):          # slice q of the server payload comes from rank q
            for s, n in payload_slice_ranges(SQ, plan.server_off, *bounds[q]):
                want_sp[s: s + n] = before[q][1][s: s + n]
        assert torch.equal(got[r][0], want_wp) and torch.equal(got[r][1], want_sp)
        # bytes outside the received slices are untouched (still the marker) in the other rows
        other = (r + 1) % world
        lo_b = payload_slice_ranges(WQ, plan.worker_off, *bounds[r])[0][0]
        if lo_b > plan.worker_off[0]:
            assert int(got[r][0][other * wstride + plan.worker_off[0]]) == 0xEE


def test_slices_tile_the_vector_and_the_payload():
    for d, world in [(D, 3), (11_689_512, 8), (100, 4), (8192, 2)]:
        bounds = slice_bounds(d, world)
        assert bounds[0][0] == 0 and bounds[-1][1] == d
        assert all(a[1] == b_[0] for a, b_ in zip(bounds, bounds[1:]))
        assert all(lo % 8192 == 0 for lo, _ in bounds if lo < d)
        cfg = b.make_config(world, d, 0.1, WQ, SQ, 1)
        for q, lay in ((WQ, b.get_layout(cfg, 0)), (SQ, b.get_layout(cfg, 1))):
            covered = sorted(r for lo, hi in bounds for r in payload_slice_ranges(q, tuple(lay.off), lo, hi))
            # per sub-array the slices are disjoint, in order, and end where the sub-array ends
            for j in range(3):
                if lay.count[j] == 0:
                    continue
                sub = [(s, n) for s, n in covered if lay.off[j] <= s < lay.off[j] + max(1, lay.count[j] * 4)]
                assert all(a[0] + a[1] <= b_[0] for a, b_ in zip(sub, sub[1:]))


# ------------------------------------------------------------------ the whole iteration, phase by phase

class _StandInInstance:
    """What ShardedDoubleSqueeze needs of a DoubleSqueeze instance, on the CPU: the payload buffers and
    layouts are the library's, the three passes write recognisable bytes and keep a log instead of
    launching kernels.  The worker pass fills the rank's own payload row with a byte that names
    (rank, step); the server pass fills this rank's slice of the server payload with the sum (mod 256)
    of the first byte of that slice in every worker's row, so it can only come out right if hop 1
    delivered every worker's slice before it ran; apply records which slices it was asked for."""

    def __init__(self, rank, world):
        self.n, self.d, self.worker_q, self.server_q = world, D, WQ, SQ
        cfg = b.make_config(world, D, 0.1, WQ, SQ, 1)
        self.worker_layout, self.server_layout = b.get_layout(cfg, 0), b.get_layout(cfg, 1)
        self.worker_payload = torch.zeros(world * int(self.worker_layout.stride), dtype=torch.uint8)
        self.server_payload = torch.zeros(int(self.server_layout.stride), dtype=torch.uint8)
        self.rank, self.log = rank, []

    def worker_compress_rows(self, g_rows, row0, t):
        self.log.append(("worker", row0, t))
        stride = int(self.worker_layout.stride)
        self.worker_payload[row0 * stride:(row0 + 1) * stride] = (17 * row0 + 3 * t + 1) % 256

    def server_aggregate_compress_slice(self, t, lo, hi, fuse_apply=False):
        self.log.append(("server", lo, hi, t, fuse_apply))
        stride = int(self.worker_layout.stride)
        wr = payload_slice_ranges(WQ, tuple(self.worker_layout.off), lo, hi)
        total = sum(int(self.worker_payload[i * stride + wr[0][0]]) for i in range(self.n)) % 256
        for s_, n_ in payload_slice_ranges(SQ, tuple(self.server_layout.off), lo, hi):
            self.server_payload[s_: s_ + n_] = total

    def apply_update_slice(self, lo, hi):
        self.log.append(("apply", lo, hi))


def _step_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1905_05957_b200.sharded import ShardedDoubleSqueeze
    inst = _StandInInstance(rank, world)
    sh = ShardedDoubleSqueeze(inst, rank, world)
    tr = DistTransport()
    sent = []
    for t in range(2):
        before = tr.bytes_sent
        sh.step(torch.zeros(D), t, tr)
        sent.append(tr.bytes_sent - before)
    staging = sum(len(v) for v in tr._staging.values())
    dist.barrier()
    out.put((rank, inst.log, inst.server_payload.numpy().tobytes(), sent, staging))
    dist.destroy_process_group()


def test_whole_iteration_over_gloo_runs_its_phases_in_order_and_moves_the_planned_bytes():
    world, port = 3, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_step_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = {}
    for _ in range(world):
        r, log, sp, sent, staging = out.get(timeout=180)
        got[r] = (log, torch.frombuffer(bytearray(sp), dtype=torch.uint8), sent, staging)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    bounds = slice_bounds(D, world)
    cfg = b.make_config(world, D, 0.1, WQ, SQ, 1)
    wl, sl = b.get_layout(cfg, 0), b.get_layout(cfg, 1)
    # what the last step's server payload must be on EVERY rank: slice q filled by rank q from all workers' bytes
    t = 1
    want = torch.zeros(int(sl.stride), dtype=torch.uint8)
    for q, (lo, hi) in enumerate(bounds):
        total = sum((17 * i + 3 * t + 1) % 256 for i in range(world)) % 256
        for s_, n_ in payload_slice_ranges(SQ, tuple(sl.off), lo, hi):
            want[s_: s_ + n_] = total
    for r in range(world):
        log, sp, sent, staging = got[r]
        lo, hi = bounds[r]
        per_step = [("worker", r, None), ("server", lo, hi, None, True)] + \
                   [("apply", *bounds[q]) for q in range(world) if q != r and bounds[q][1] > bounds[q][0]]
        assert len(log) == 2 * len(per_step)
        for t_ in range(2):
            chunk = log[t_ * len(per_step):(t_ + 1) * len(per_step)]
            assert chunk[0] == ("worker", r, t_) and chunk[1] == ("server", lo, hi, t_, True)
            assert chunk[2:] == per_step[2:]
        assert torch.equal(sp, want), f"server payload on rank {r}"
        # bytes on the wire per step: slice q of the own payload to every other rank, the own server slice to every other rank
        hop1 = sum(sum(n_ for _, n_ in payload_slice_ranges(WQ, tuple(wl.off), *bounds[q])) for q in range(world) if q != r)
        hop2 = (world - 1) * sum(n_ for _, n_ in payload_slice_ranges(SQ, tuple(sl.off), lo, hi))
        assert sent == [hop1 + hop2, hop1 + hop2]
        assert staging == 2 * world        # one set of receive buffers per hop, reused by the second step
    # the compressed hops move a small fraction of what the dense vector would: 9/32 and 1/32 of 4 bytes per entry here
    dense = 4 * D
    assert got[0][2][0] < 0.25 * dense


# ------------------------------------------------------------------ collectives of the top-k server over slices

def _collectives_main(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1905_05957_b200.sharded import ShardedDoubleSqueeze
    tr = DistTransport()
    hist = (torch.arange(4096, dtype=torch.int32) % 7) * (rank + 1)        # this slice's histogram
    tr.all_reduce_sum(hist)
    words = tr.all_gather_small(torch.tensor([10 * rank + 1, rank, 5, 1234], dtype=torch.int32))
    shares = ShardedDoubleSqueeze.topk_shares([(int(w[0]), int(w[1])) for w in words], max(int(w[2]) for w in words))
    dist.barrier()
    out.put((rank, hist.tolist()[:16], [w.tolist() for w in words], shares, tr.bytes_sent))
    dist.destroy_process_group()


def test_histogram_sum_and_totals_gather_over_gloo():
    world, port = 3, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_collectives_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = [out.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want_hist = [(i % 7) * (1 + 2 + 3) for i in range(16)]
    want_words = [[10 * r + 1, r, 5, 1234] for r in range(world)]
    # ties 0, 1, 2 per slice and a quota of 5: every tie is kept; the slots follow the kept counts
    want_shares = [(0, 1, 0), (1, 12, 1), (2, 23, 13)]
    for rank, hist, words, shares, sent in got:
        assert hist == want_hist and words == want_words and shares == want_shares
        assert sent == 4096 * 4 + 16 * (world - 1)
