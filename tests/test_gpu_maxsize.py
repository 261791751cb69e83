"""Sizes beyond 2^31 entries per vector: 64-bit offsets and 32-bit indices near their limits."""
import numpy as np
import psutil
import pytest
import torch

import oracle
from paper_1905_05957_b200 import DoubleSqueeze, Q
from tests.helpers import compare_state, to_oracle_q

pytestmark = pytest.mark.gpu

D_BIG = (1 << 31) + 4100          # more than 2^31 entries, ragged against every tile size


def _enough(host_gib: float, dev_gib: float) -> bool:
    free, _ = torch.cuda.mem_get_info()
    return psutil.virtual_memory().available > host_gib * 2**30 and free > dev_gib * 2**30


def test_sign1_beyond_two_to_the_31_entries_matches_the_oracle():
    if not _enough(60, 40):
        pytest.skip("needs 60 GiB of host and 40 GiB of device memory")
    n, d = 1, D_BIG
    wq = sq = Q("sign1", chunk=4096)
    ds = DoubleSqueeze(n, d, 0.1, wq, sq, seed=1)
    gen = torch.Generator(device="cuda").manual_seed(5)
    g = torch.empty(n, d, device="cuda").normal_(0.0, 1.0, generator=gen)
    ds.delta_w.normal_(0.0, 0.3, generator=gen)
    ds.delta_s.normal_(0.0, 0.1, generator=gen)
    st = oracle.State(ds.x.cpu().numpy().copy(), ds.delta_w.cpu().numpy().copy(), ds.delta_s.cpu().numpy().copy())
    ds.step(g, 2)
    torch.cuda.synchronize()
    g_host = g.cpu().numpy()
    del g
    oracle.step(st, g_host, to_oracle_q(wq), to_oracle_q(sq), 0.1, 1, 2)
    compare_state(ds, st, g_host, tag="2^31+: ")
    ds.close()


def test_topk_beyond_two_to_the_31_entries_finds_planted_entries():
    """Closed form instead of the oracle's full sort: small noise everywhere, k large values planted
    at known places up to the very last entry; top-k must return exactly those, in order."""
    if not _enough(8, 70):
        pytest.skip("needs 70 GiB of device memory")
    n, d, k = 1, D_BIG, 1000
    ds = DoubleSqueeze(n, d, 0.1, Q("topk", k=k), Q("identity"), seed=1)
    gen = torch.Generator(device="cuda").manual_seed(6)
    g = torch.empty(n, d, device="cuda").uniform_(-1e-3, 1e-3, generator=gen)
    where = torch.linspace(0, d - 1, k, dtype=torch.float64).round().to(torch.int64).cuda()
    where[-1] = d - 1
    where[-2] = (1 << 31) + 1
    where[-3] = (1 << 31) - 1
    where = torch.unique(where)          # sorted, distinct
    k = int(where.numel())
    ds.close()
    ds = DoubleSqueeze(n, d, 0.1, Q("topk", k=k), Q("identity"), seed=1)
    vals = (1.0 + torch.arange(k, device="cuda", dtype=torch.float32) / k) * torch.where(
        torch.arange(k, device="cuda") % 2 == 0, 1.0, -1.0)
    g[0, where] = vals
    before = g[0].clone()
    for step in range(2):                # the second step runs with a threshold history
        ds.delta_w.zero_()
        ds.worker_compress(g, step)
        torch.cuda.synchronize()
        v = ds.worker_views()[0]
        idx = v["idx"].to(torch.int64) & 0xFFFFFFFF
        assert torch.equal(idx, where)
        assert torch.equal(v["val"], vals)
        assert ds.device_status() == 0
        kept = ds.delta_w[0, where]
        assert not kept.any()
        ds.delta_w[0, where] = vals      # put them back: everything else must be untouched v
        assert torch.equal(ds.delta_w[0].view(torch.int32), before.view(torch.int32))
        ds.server_aggregate_compress(step, fuse_apply=True)   # completes the step (identity server)
    ds.close()
