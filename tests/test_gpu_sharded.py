"""One worker per GPU with a sharded server (rows / slice entry points of the C ABI), checked on ONE
GPU: all ranks live in this process, run one after the other, and exchange by plain copies.  The
result must equal the whole-vector step bit for bit, which the other tests check against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_05957_b200 import DoubleSqueeze, Q
from paper_1905_05957_b200.sharded import ShardedDoubleSqueeze, slice_bounds, step_in_process
from tests.helpers import compare_state, to_oracle_q

pytestmark = pytest.mark.gpu

SIGN = Q("sign1", chunk=4096)
PAIRS = [(SIGN, SIGN), (Q("qsgd", chunk=2048, levels=255), Q("qsgd", chunk=2048, levels=255)),
         (Q("sign1", chunk=1024, norm=2), Q("clip", bits=16)), (Q("clip", bits=24), Q("qsgd", chunk=512, levels=7)),
         (Q("identity"), SIGN), (Q("qsgd", chunk=8192, levels=31), Q("identity")),
         (Q("rsparse", chunk=4096, keep_one_in=32), Q("rsparse", chunk=4096, keep_one_in=32)),
         (Q("rsparse", chunk=256, keep_one_in=4, scaled=1), SIGN), (Q("clip", bits=16), Q("rsparse", chunk=1024, keep_one_in=8))]


def _bits(t):
    return t.contiguous().view(torch.uint8).cpu()


@pytest.mark.parametrize("wq,sq", PAIRS)
@pytest.mark.parametrize("world,d", [(4, 5 * 8192 + 1234), (3, 8192 * 3), (5, 20_000), (2, 100)])
def test_sharded_step_equals_whole_vector_step(wq, sq, world, d):
    gamma, seed, T = 0.1, 77, 3
    gen = torch.Generator().manual_seed(world * 1000 + d)
    gs = [torch.randn(world, d, generator=gen).cuda() for _ in range(T)]
    whole = DoubleSqueeze(world, d, gamma, wq, sq, seed)
    st = oracle.State.zeros(world, d)
    # every rank keeps the error of its own worker only (delta_w_rows = 1); rank 0 keeps all rows, which must work too
    ranks = [ShardedDoubleSqueeze(DoubleSqueeze(world, d, gamma, wq, sq, seed, delta_w_rows=1 if r else 0), r, world)
             for r in range(world)]
    bounds = slice_bounds(d, world)
    assert bounds[0][0] == 0 and bounds[-1][1] == d and all(a[1] == b[0] for a, b in zip(bounds, bounds[1:]))
    for t, g in enumerate(gs):
        whole.step(g, t)
        step_in_process(ranks, g, t)
        torch.cuda.synchronize()
        oracle.step(st, g.cpu().numpy(), to_oracle_q(wq), to_oracle_q(sq), gamma, seed, t)
        compare_state(whole, st, g.cpu().numpy(), tag=f"whole, step {t}: ")
        for r in ranks:
            lo, hi = bounds[r.rank]
            assert torch.equal(_bits(r.ds.x), _bits(whole.x)), f"x on rank {r.rank}, step {t}"
            own = r.ds.delta_w[r.rank] if r.ds.delta_w.shape[0] == world else r.ds.delta_w[0]
            assert r.rank == 0 or r.ds.delta_w.shape[0] == 1      # one row of errors, not n
            assert torch.equal(_bits(own), _bits(whole.delta_w[r.rank]))
            assert torch.equal(_bits(r.ds.delta_s[lo:hi]), _bits(whole.delta_s[lo:hi]))
            for name, view in r.ds.server_views().items():
                assert torch.equal(_bits(view), _bits(whole.server_views()[name])), f"server payload {name} on rank {r.rank}"
            mine, ref = r.ds.worker_views()[r.rank], whole.worker_views()[r.rank]
            for name in mine:
                assert torch.equal(_bits(mine[name]), _bits(ref[name])), f"worker payload {name} of rank {r.rank}"
            assert r.ds.device_status() == 0
    # the whole-vector result is itself the oracle's
    assert np.array_equal(whole.x.cpu().numpy().view(np.uint32), st.x.view(np.uint32))


TOPK_PAIRS = [(SIGN, 1), (Q("qsgd", chunk=2048, levels=255), 2), (Q("clip", bits=16), 3), (Q("identity"), 4),
              (Q("rsparse", chunk=1024, keep_one_in=8), 5)]


@pytest.mark.parametrize("wq,kdiv", TOPK_PAIRS)
@pytest.mark.parametrize("world,d", [(4, 5 * 8192 + 1234), (3, 8192 * 3), (5, 200_000), (2, 100)])
def test_sharded_top_k_server_equals_whole_vector_step(wq, kdiv, world, d):
    """A top-k server whose vector is spread over the ranks: the staged calls with the histograms summed over the ranks
    in between must select exactly what the whole-vector pass selects (and that is the oracle's selection)."""
    gamma, seed, T = 0.1, 78, 3
    k = max(1, d // (20 * kdiv))
    sq = Q("topk", k=k)
    gen = torch.Generator().manual_seed(world * 1000 + d + kdiv)
    gs = [torch.randn(world, d, generator=gen).cuda() for _ in range(T)]
    if kdiv == 4:   # identity workers: integer-valued gradients, so that many entries tie at the threshold across slices
        gs = [torch.randint(-3, 4, (world, d), generator=gen).float().cuda() for _ in range(T)]
    whole = DoubleSqueeze(world, d, gamma, wq, sq, seed)
    st = oracle.State.zeros(world, d)
    ranks = [ShardedDoubleSqueeze(DoubleSqueeze(world, d, gamma, wq, sq, seed, delta_w_rows=1), r, world) for r in range(world)]
    bounds = slice_bounds(d, world)
    for t, g in enumerate(gs):
        whole.step(g, t)
        step_in_process(ranks, g, t)
        torch.cuda.synchronize()
        oracle.step(st, g.cpu().numpy(), to_oracle_q(wq), to_oracle_q(sq), gamma, seed, t)
        compare_state(whole, st, g.cpu().numpy(), tag=f"whole, step {t}: ")
        for r in ranks:
            lo, hi = bounds[r.rank]
            assert torch.equal(_bits(r.ds.x), _bits(whole.x)), f"x on rank {r.rank}, step {t}"
            assert torch.equal(_bits(r.ds.delta_w[0]), _bits(whole.delta_w[r.rank]))
            assert torch.equal(_bits(r.ds.delta_s[lo:hi]), _bits(whole.delta_s[lo:hi]))
            for name, view in r.ds.server_views().items():
                assert torch.equal(_bits(view), _bits(whole.server_views()[name])), f"server payload {name} on rank {r.rank}"
            assert r.ds.device_status() == 0


def test_tie_quota_is_dealt_to_earlier_slices_first():
    shares = ShardedDoubleSqueeze.topk_shares([(5, 2), (0, 3), (7, 0), (1, 4)], r=4)
    assert shares == [(2, 7, 0), (2, 2, 7), (0, 7, 9), (0, 1, 16)]
    assert ShardedDoubleSqueeze.topk_shares([(0, 0), (3, 1)], r=1) == [(0, 0, 0), (1, 4, 0)]


def test_slices_reject_what_they_cannot_do():
    ds = DoubleSqueeze(2, 40_000, 0.1, SIGN, SIGN)
    g = torch.randn(2, 40_000, device="cuda")
    ds.worker_compress_rows(g[1:2].contiguous(), 1, 0)
    with pytest.raises(Exception, match="-1"):
        ds.server_aggregate_compress_slice(0, 100, 8192)          # start off the grid
    with pytest.raises(Exception, match="-1"):
        ds.server_aggregate_compress_slice(0, 0, 8000)            # end neither on the grid nor d
    with pytest.raises(Exception, match="-1"):
        ds.worker_compress_rows(g, 1, 0)                          # rows 1..2 of 2
    one = DoubleSqueeze(4, 40_000, 0.1, SIGN, SIGN, delta_w_rows=2)
    g4 = torch.randn(4, 40_000, device="cuda")
    with pytest.raises(Exception, match="-6"):
        one.worker_compress(g4, 0)                                # the errors of one block of workers only
    with pytest.raises(Exception, match="-1"):
        one.worker_compress_rows(g4[1:3].contiguous(), 1, 0)      # rows 1..2 straddle two blocks of 2
    one.worker_compress_rows(g4[2:4].contiguous(), 2, 0)
    tk = DoubleSqueeze(2, 40_000, 0.1, Q("topk", k=10), SIGN)
    with pytest.raises(Exception, match="-6"):
        tk.worker_compress_rows(g[:1].contiguous(), 0, 0)
    with pytest.raises(Exception, match="-6"):
        tk.server_aggregate_compress_slice(0, 0, 8192)
    torch.cuda.synchronize()
