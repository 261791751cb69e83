"""The benchmark workloads at full size, in the launch configuration the benchmark times: one step from
a seeded random state (non-zero errors and model), compared with the oracle element by element."""
import numpy as np
import psutil
import pytest
import torch

import oracle
from paper_1905_05957_b200 import DoubleSqueeze, WORKLOADS, make_gradients
from tests.helpers import compare_state, to_oracle_q

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wid", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12])
def test_full_size_step_matches_oracle(wid):
    wl = WORKLOADS[wid]
    need = 4 * wl.n * wl.d * 4 + (2 << 30)
    if psutil.virtual_memory().available < need:
        pytest.skip(f"host memory: need {need >> 30} GiB for the oracle's copy of workload {wid}")
    dev = "cuda"
    ds = DoubleSqueeze.for_workload(wl, dev)
    gen = torch.Generator(device=dev).manual_seed(1000 + wid)
    g = make_gradients(wl, 3, device=dev)
    scale = float(g[0, :100_000].abs().mean())
    ds.x.normal_(0.0, 1.0, generator=gen)
    if wl.compensate:
        ds.delta_w.normal_(0.0, 0.5 * scale, generator=gen)
        ds.delta_s.normal_(0.0, 0.25 * scale, generator=gen)
        st = oracle.State(ds.x.cpu().numpy().copy(), ds.delta_w.cpu().numpy().copy(), ds.delta_s.cpu().numpy().copy())
    else:
        st = oracle.State.zeros(wl.n, wl.d, ds.x.cpu().numpy())
    ds.step(g, 3, fuse_apply=True)
    torch.cuda.synchronize()
    g_host = g.cpu().numpy()
    del g
    oracle.step(st, g_host, to_oracle_q(wl.worker_q), to_oracle_q(wl.server_q), wl.gamma, wl.seed, 3, compensate=wl.compensate)
    compare_state(ds, st, g_host, tag=f"workload {wid}: ")
    ds.close()


@pytest.mark.parametrize("wid", [3, 5])
def test_full_size_top_k_on_the_predicted_route_matches_oracle(wid):
    """The route the benchmark times in its steady state: after a few steps the top-k threshold band is
    predicted from the earlier thresholds and v is read only once.  Four GPU steps from a seeded
    state; the state before the last one goes to the oracle, which takes that one step, and every
    output must agree.  The route counters say which path each selection took."""
    wl = WORKLOADS[wid]
    need = 4 * wl.n * wl.d * 4 + (2 << 30)
    if psutil.virtual_memory().available < need:
        pytest.skip(f"host memory: need {need >> 30} GiB for the oracle's copy of workload {wid}")
    dev = "cuda"
    ds = DoubleSqueeze.for_workload(wl, dev)
    gen = torch.Generator(device=dev).manual_seed(2000 + wid)
    selections = (wl.n if wl.worker_q.op == "topk" else 0) + (1 if wl.server_q.op == "topk" else 0)
    g = make_gradients(wl, 0, device=dev)
    scale = float(g[0, :100_000].abs().mean())
    ds.delta_w.normal_(0.0, 0.5 * scale, generator=gen)
    ds.delta_s.normal_(0.0, 0.25 * scale, generator=gen)
    ds.x.normal_(0.0, 1.0, generator=gen)
    T = 4
    for t in range(T - 1):
        make_gradients(wl, t, device=dev, out=g)
        ds.step(g, t, fuse_apply=True)
        if t == 0:
            assert ds.topk_routes() == (0, selections)       # no history yet: the full route
    before = ds.topk_routes()
    st = oracle.State(ds.x.cpu().numpy().copy(), ds.delta_w.cpu().numpy().copy(), ds.delta_s.cpu().numpy().copy())
    make_gradients(wl, T - 1, device=dev, out=g)
    ds.step(g, T - 1, fuse_apply=True)
    torch.cuda.synchronize()
    after = ds.topk_routes()
    assert (after[0] - before[0], after[1] - before[1]) == (selections, 0), \
        f"the last step was meant to run on predicted bands: routes {before} -> {after}"
    g_host = g.cpu().numpy()
    del g
    oracle.step(st, g_host, to_oracle_q(wl.worker_q), to_oracle_q(wl.server_q), wl.gamma, wl.seed, T - 1)
    compare_state(ds, st, g_host, tag=f"workload {wid}, predicted route: ")
    ds.close()
