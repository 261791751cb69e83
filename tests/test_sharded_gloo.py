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
