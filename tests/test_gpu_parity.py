"""CUDA library against the oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1905_05957_b200 import DoubleSqueeze, Q, WORKLOADS, make_gradients
from tests.helpers import compare_state, to_oracle_q

pytestmark = pytest.mark.gpu

SIGN = lambda L=4096: Q("sign1", chunk=L)
SIGN_L2 = lambda L=4096: Q("sign1", chunk=L, norm=2)
QSGD = lambda L=2048, s=255: Q("qsgd", chunk=L, levels=s)
TOPK = lambda k: Q("topk", k=k)
IDENT = Q("identity")
CLIP = lambda b=16: Q("clip", bits=b)
RSP = lambda S=4, L=4096, scaled=0: Q("rsparse", chunk=L, keep_one_in=S, scaled=scaled)
SIGN_WHOLE = lambda norm=1: Q("sign1", chunk=0, norm=norm)      # one factor for the whole vector
TERN = Q("ternary")


def run_lockstep(n, d, wq, sq, gs, gamma=0.1, seed=190505957, fuse=True, x0=None, state0=None, scribble=False,
                 compensate=True):
    """Free-running: both sides start from the same state and see the same gradients; after every
    step every output must agree."""
    # every buffer sits between sentinel bytes and the payloads start out as 0xFF: a write outside a
    # buffer, or a payload byte the library leaves to chance, fails the comparison
    ds = DoubleSqueeze(n, d, gamma, wq, sq, seed, x0=x0, guard=True, payload_fill=0xFF, compensate=compensate)
    st = oracle.State.zeros(n, d, None if x0 is None else x0.cpu().numpy())
    if state0 is not None:
        dw, dsv = state0
        ds.delta_w.copy_(dw)
        ds.delta_s.copy_(dsv)
        st.delta_w = dw.cpu().numpy().copy()
        st.delta_s = dsv.cpu().numpy().copy()
    for t, g in enumerate(gs):
        if scribble:   # the workspace only ever holds hints: any contents must give the same results
            ds.workspace.random_(0, 256)
        g_dev = g.cuda().contiguous()
        ds.step(g_dev, t, fuse_apply=fuse)
        torch.cuda.synchronize()
        g_host = g.cpu().numpy()
        oracle.step(st, g_host, to_oracle_q(wq), to_oracle_q(sq), gamma, seed, t, compensate=compensate)
        compare_state(ds, st, g_host, tag=f"step {t}: ")
        assert ds.check_guards(), f"step {t}: bytes outside a buffer were overwritten"
    ds.close()
    return ds, st


def randn_steps(n, d, T, seed=0, scale=1.0):
    gen = torch.Generator().manual_seed(seed)
    return [torch.randn(n, d, generator=gen) * scale for _ in range(T)]


# ------------------------------------------------------------------ operators, several tiles + ragged tail

@pytest.mark.parametrize("d", [4096, 10_000, 65_536 + 4 * 37, 33, 1])
@pytest.mark.parametrize("L", [128, 1024, 4096, 8192])
def test_sign1_both_passes(d, L):
    run_lockstep(3, d, SIGN(L), SIGN(L), randn_steps(3, d, 3, seed=d + L))


@pytest.mark.parametrize("d", [4096, 10_000, 65_536 + 4 * 37, 33, 1])
@pytest.mark.parametrize("L", [128, 2048, 4096, 8192])
def test_sign1_l2_magnitudes_both_passes(d, L):
    run_lockstep(3, d, SIGN_L2(L), SIGN_L2(L), randn_steps(3, d, 3, seed=d + L + 1))


def test_sign1_l2_mixed_with_other_operators_and_unaligned_rows():
    d = 50_000 + 13
    for wq, sq in [(SIGN_L2(4096), TOPK(500)), (SIGN_L2(512), SIGN(2048)), (QSGD(1024, 31), SIGN_L2(4096)),
                   (TOPK(700), SIGN_L2(1024)), (IDENT, SIGN_L2(128))]:
        run_lockstep(4, d, wq, sq, randn_steps(4, d, 2, seed=41))
    run_lockstep(3, 30_000, SIGN_L2(4096), SIGN_L2(4096), randn_steps(3, 30_000, 3, seed=42), fuse=False)


@pytest.mark.parametrize("d", [2048, 10_000, 40_000 + 4, 5])
@pytest.mark.parametrize("L,s", [(128, 255), (2048, 255), (2048, 1), (512, 15), (8192, 200)])
def test_qsgd_both_passes(d, L, s):
    run_lockstep(3, d, QSGD(L, s), QSGD(L, s), randn_steps(3, d, 3, seed=d + L + s, scale=1e-3))


@pytest.mark.parametrize("d,k", [(10_000, 100), (70_000, 700), (70_000, 1), (8192, 8192), (300, 0), (33, 7), (1, 1)])
def test_topk_both_passes(d, k):
    run_lockstep(3, d, TOPK(k), TOPK(k), randn_steps(3, d, 3, seed=d + k))


@pytest.mark.parametrize("d", [4096, 10_000, 65_536 + 4 * 37, 33, 5, 1])
@pytest.mark.parametrize("b", [16, 24])
def test_clip_both_passes(d, b):
    run_lockstep(3, d, CLIP(b), CLIP(b), randn_steps(3, d, 3, seed=d + b))


def test_clip_mixed_with_other_operators_unaligned_rows_and_unfused_update():
    d = 50_000 + 13
    for wq, sq in [(CLIP(16), TOPK(500)), (CLIP(24), SIGN(2048)), (QSGD(1024, 31), CLIP(16)), (TOPK(700), CLIP(24)),
                   (CLIP(16), QSGD(2048)), (SIGN(4096), CLIP(16)), (IDENT, CLIP(16)), (CLIP(16), IDENT),
                   (CLIP(16), SIGN_L2(1024))]:
        run_lockstep(5, d, wq, sq, randn_steps(5, d, 2, seed=43))
    run_lockstep(3, 30_000, CLIP(16), CLIP(16), randn_steps(3, 30_000, 3, seed=44), fuse=False)
    run_lockstep(3, 30_001, CLIP(24), CLIP(24), randn_steps(3, 30_001, 2, seed=45), fuse=False)
    run_lockstep(37, 9000, CLIP(16), CLIP(16), randn_steps(37, 9000, 2, seed=46))


@pytest.mark.parametrize("d", [4096, 10_000, 65_536 + 4 * 37, 33, 5, 1])
@pytest.mark.parametrize("S,L,scaled", [(4, 4096, 0), (2, 128, 0), (32, 4096, 0), (128, 1024, 0), (4, 512, 1), (8, 8192, 1)])
def test_rsparse_both_passes(d, S, L, scaled):
    run_lockstep(3, d, RSP(S, L, scaled), RSP(S, L, scaled), randn_steps(3, d, 4, seed=d + S + L))


def test_rsparse_mixed_with_other_operators_unaligned_rows_and_unfused_update():
    d = 50_000 + 13
    for wq, sq in [(RSP(8), TOPK(500)), (RSP(4, 256), SIGN(2048)), (QSGD(1024, 31), RSP(16)), (TOPK(700), RSP(2, 128)),
                   (RSP(32), QSGD(2048)), (SIGN(4096), RSP(4)), (IDENT, RSP(8, 512)), (RSP(4), IDENT), (RSP(4), CLIP(16)),
                   (CLIP(24), RSP(8, 1024, 1))]:
        run_lockstep(5, d, wq, sq, randn_steps(5, d, 3, seed=47))
    run_lockstep(3, 30_000, RSP(4), RSP(4), randn_steps(3, 30_000, 3, seed=48), fuse=False)
    run_lockstep(3, 30_001, RSP(8, 256), RSP(8, 256), randn_steps(3, 30_001, 3, seed=49), fuse=False)
    run_lockstep(37, 9000, RSP(4, 128), RSP(4, 128), randn_steps(37, 9000, 2, seed=50))


# ------------------------------------------------------------------ one factor for the whole vector

@pytest.mark.parametrize("d", [1, 33, 4096, 10_000, 65_536 + 4 * 37, 5 * 4096 * 1024 // 16 + 12])
@pytest.mark.parametrize("norm", [1, 2])
def test_sign1_whole_vector_both_passes(d, norm):
    run_lockstep(3, d, SIGN_WHOLE(norm), SIGN_WHOLE(norm), randn_steps(3, d, 3, seed=d + norm))


def test_sign1_whole_vector_many_tiles_exercises_the_block_sums():
    # more than 1024 tiles per vector: every thread of the combining kernel sums a block of tile sums
    d = 4096 * 2500 + 777
    run_lockstep(2, d, SIGN_WHOLE(1), SIGN_WHOLE(2), randn_steps(2, d, 2, seed=3))


@pytest.mark.parametrize("d", [1, 5, 33, 4096, 10_000, 65_536 + 4 * 37, 300_001])
def test_ternary_both_passes(d):
    run_lockstep(3, d, TERN, TERN, randn_steps(3, d, 3, seed=d, scale=1e-2))


def test_whole_vector_operators_mixed_unaligned_unfused_and_degenerate():
    d = 50_000 + 13
    for wq, sq in [(TERN, IDENT), (TERN, TOPK(500)), (TERN, SIGN(2048)), (SIGN_WHOLE(), TERN), (QSGD(1024, 31), TERN),
                   (TOPK(700), SIGN_WHOLE(2)), (SIGN_WHOLE(2), QSGD(2048)), (CLIP(16), TERN), (TERN, RSP(8)),
                   (RSP(4), SIGN_WHOLE()), (IDENT, TERN), (SIGN_WHOLE(), CLIP(24))]:
        run_lockstep(5, d, wq, sq, randn_steps(5, d, 2, seed=51))
    run_lockstep(3, 30_000, TERN, TERN, randn_steps(3, 30_000, 3, seed=52), fuse=False)
    run_lockstep(3, 30_001, SIGN_WHOLE(), SIGN_WHOLE(2), randn_steps(3, 30_001, 3, seed=53), fuse=False)
    run_lockstep(37, 9000, TERN, SIGN_WHOLE(), randn_steps(37, 9000, 2, seed=54))
    n, dd = 2, 3 * 4096
    g = torch.randn(n, dd) * 1e-3
    g[:, :4096] = 0.0
    g[:, 4096:4096 + 64] = -0.0
    g[:, 5000:5100] = 1e-41
    for wq in (TERN, SIGN_WHOLE(1), SIGN_WHOLE(2)):
        run_lockstep(n, dd, wq, wq, [g, g.clone(), -g, torch.zeros(n, dd)])


# ------------------------------------------------------------------ without error compensation

@pytest.mark.parametrize("wq,sq", [
    (TOPK(500), IDENT), (TERN, IDENT), (SIGN(4096), SIGN(4096)), (QSGD(2048), QSGD(2048)), (TOPK(700), TOPK(300)),
    (SIGN(1024), TOPK(200)), (CLIP(16), RSP(8)), (RSP(4), CLIP(24)), (IDENT, IDENT), (SIGN_WHOLE(), TERN),
    (TOPK(0), SIGN(128)), (SIGN_L2(512), SIGN_WHOLE(2)),
])
def test_without_compensation_matches_the_oracle(wq, sq):
    d = 50_000 + 12
    run_lockstep(5, d, wq, sq, randn_steps(5, d, 3, seed=61), compensate=False)
    run_lockstep(3, 30_001, wq, sq, randn_steps(3, 30_001, 2, seed=62), compensate=False, fuse=False)


def test_without_compensation_top_k_on_predicted_bands_and_after_jumps():
    n, d, k = 3, 120_000, 1200
    gen = torch.Generator().manual_seed(9)
    scales = [1, 1, 1, 1, 1.02, 8.0, 8.0, 0.01, 0.01, 1]
    gs = [torch.randn(n, d, generator=gen) * s for s in scales]
    ds, _ = run_lockstep(n, d, TOPK(k), TOPK(k), gs, compensate=False)
    predicted, full = ds.topk_routes()
    assert predicted >= 3 * (n + 1) and full >= 3 * (n + 1)
    assert ds.delta_w.numel() == 0          # no worker error exists at all


def test_identity_is_parallel_sgd():
    run_lockstep(4, 10_001, IDENT, IDENT, randn_steps(4, 10_001, 3))


@pytest.mark.parametrize("wq,sq", [
    (SIGN(4096), TOPK(500)), (TOPK(2000), SIGN(1024)), (QSGD(2048), TOPK(300)), (TOPK(1000), QSGD(256, 7)),
    (SIGN(256), QSGD(4096, 255)), (QSGD(1024, 3), SIGN(2048)), (IDENT, TOPK(100)), (SIGN(512), IDENT),
    (TOPK(50), IDENT), (QSGD(128, 9), IDENT), (IDENT, SIGN(128)), (IDENT, QSGD(128, 31)),
])
def test_mixed_operators(wq, sq):
    d = 50_000 + 12
    run_lockstep(5, d, wq, sq, randn_steps(5, d, 3, seed=11))


# ------------------------------------------------------------------ layout and alignment edge cases

@pytest.mark.parametrize("d", [4097, 4098, 4099, 12_345, 31, 127])
@pytest.mark.parametrize("wq,sq", [(SIGN(1024), SIGN(1024)), (QSGD(1024, 255), QSGD(1024, 255)), ("topk", "topk"),
                                   (IDENT, IDENT)])
def test_rows_not_16_byte_aligned(d, wq, sq):
    if wq == "topk":
        wq = sq = TOPK(max(1, d // 50))
    run_lockstep(3, d, wq, sq, randn_steps(3, d, 2, seed=d))


@pytest.mark.parametrize("wq,sq", [(SIGN(4096), SIGN(4096)), (QSGD(2048), QSGD(2048)), (TOPK(300), TOPK(300)),
                                   (SIGN(4096), TOPK(150)), (IDENT, IDENT)])
def test_unfused_apply_equals_fused(wq, sq):
    d = 30_000
    run_lockstep(4, d, wq, sq, randn_steps(4, d, 3, seed=5), fuse=False)


# ------------------------------------------------------------------ degenerate data

def test_topk_ties_all_equal_and_integer_valued():
    n, d = 2, 70_000
    gen = torch.Generator().manual_seed(3)
    ties = [torch.randint(-3, 4, (n, d), generator=gen).float() for _ in range(2)]
    for k in (1, 777, 35_000, d - 1):
        run_lockstep(n, d, TOPK(k), TOPK(k), ties)
    same = [torch.full((n, d), -2.5), torch.full((n, d), 2.5)]
    run_lockstep(n, d, TOPK(1234), TOPK(4321), same)
    zeros = [torch.zeros(n, d), torch.zeros(n, d)]
    run_lockstep(n, d, TOPK(10), TOPK(10), zeros)


def test_zero_signed_zero_subnormal_and_zero_chunks():
    n, d = 2, 3 * 4096
    g = torch.randn(n, d) * 1e-3
    g[:, :4096] = 0.0            # an all-zero chunk
    g[:, 4096:4096 + 64] = -0.0
    g[:, 5000:5100] = 1e-41      # subnormals
    g[:, 5100:5200] = -1e-41
    g[0, 8192:] = 1e-30          # squares underflow: a quantisation chunk of norm ~0
    for wq in (SIGN(4096), QSGD(2048), TOPK(100), SIGN(128), QSGD(128, 5), SIGN_L2(4096), SIGN_L2(128), CLIP(16), CLIP(24)):
        run_lockstep(n, d, wq, wq, [g, g.clone(), -g])


def test_topk_threshold_prediction_hits_misses_and_garbage():
    """Top-k marks candidates during its first pass from the previous steps' threshold bins.  Steady
    magnitudes make the prediction hit, jumps make it miss (the slow path runs), and a workspace
    full of random bytes must change nothing."""
    n, d, k = 3, 120_000, 1200
    gen = torch.Generator().manual_seed(8)
    scales = [1, 1, 1, 1, 1.02, 1.05, 8.0, 8.0, 0.01, 0.01, 0.01, 1, 1]
    gs = [torch.randn(n, d, generator=gen) * s for s in scales]
    ds, _ = run_lockstep(n, d, TOPK(k), TOPK(k), gs)
    predicted, full = ds.topk_routes()
    assert predicted + full == (n + 1) * len(gs)
    # the first step and the jump by 8x cannot be predicted (after the jump down the errors still carry
    # the large magnitudes, so the threshold comes down slowly); the steady stretches are
    assert full >= 2 * (n + 1)
    assert predicted >= 4 * (n + 1)
    run_lockstep(n, d, SIGN(4096), TOPK(k // 2), gs[:6])
    run_lockstep(n, d, TOPK(k), TOPK(k), gs[:5], scribble=True)


def test_qsgd_stream_depends_on_seed_and_step():
    n, d = 2, 8192
    g = randn_steps(n, d, 1, seed=2)[0]
    a = DoubleSqueeze(n, d, 0.1, QSGD(), QSGD(), seed=1)
    b = DoubleSqueeze(n, d, 0.1, QSGD(), QSGD(), seed=(1 << 40) + 1)
    a.worker_compress(g.cuda(), 0)
    b.worker_compress(g.cuda(), 0)
    la, lb = a.worker_views()[0]["lvl"].cpu(), b.worker_views()[0]["lvl"].cpu()
    assert not torch.equal(la, lb)          # high word of the seed reaches the key
    assert not torch.equal(la, a.worker_views()[1]["lvl"].cpu())


def test_many_workers_and_one_worker():
    run_lockstep(1, 9000, SIGN(4096), SIGN(4096), randn_steps(1, 9000, 2))
    run_lockstep(33, 5000, QSGD(2048), SIGN(4096), randn_steps(33, 5000, 2))
    run_lockstep(7, 20_000, TOPK(200), TOPK(200), randn_steps(7, 20_000, 2))


# ------------------------------------------------------------------ the workloads, scaled down

@pytest.mark.parametrize("wid", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12])
def test_workload_recipes_scaled(wid):
    wl = WORKLOADS[wid]
    wl = wl if wid == 1 else wl.scaled(d=200_000 + 40, n=min(wl.n, 8), steps=4)
    gs = [make_gradients(wl, t, device="cpu") for t in range(min(wl.steps, 4))]
    run_lockstep(wl.n, wl.d, wl.worker_q, wl.server_q, gs, gamma=wl.gamma, seed=wl.seed, compensate=wl.compensate)


@pytest.mark.parametrize("wid", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10])
def test_telescoping_identity_free_running_on_the_gpu(wid):
    """Eq. 5-6 on the GPU alone, with no oracle in the loop: after T steps of any Q,
    x_T - gamma (delta_T + mean_i delta_T^(i)) = x_0 - gamma sum_t mean_i g_t^(i), up to fp32 rounding."""
    wl = WORKLOADS[wid]
    wl = wl if wid == 1 else wl.scaled(d=300_000 + 8, n=min(wl.n, 8))
    T = 20
    ds = DoubleSqueeze.for_workload(wl, "cuda")
    x0 = torch.randn(wl.d, generator=torch.Generator().manual_seed(wid)).cuda()
    ds.x.copy_(x0)
    rhs = x0.double()
    gmax = 0.0
    for t in range(T):
        g = make_gradients(wl, t, device="cuda")
        ds.step(g, t)
        rhs -= wl.gamma * g.double().mean(dim=0)
        gmax = max(gmax, float(g.abs().max()))
    torch.cuda.synchronize()
    omega = ds.delta_s.double() + ds.delta_w.double().mean(dim=0)
    lhs = ds.x.double() - wl.gamma * omega
    scale = max(float(rhs.abs().max()), gmax, float(omega.abs().max()))
    assert float((lhs - rhs).abs().max()) <= 40 * T * 2.0**-24 * scale
    assert ds.device_status() == 0
    ds.close()


def test_state_copied_into_a_fresh_instance_continues_identically():
    """x, delta_w and delta_s are the whole state (Algorithm 1): T steps, copy them into a new
    instance (which has no threshold history), T more steps -- same bits as 2T steps in one go."""
    n, d, T = 4, 60_000, 4
    for wq, sq in [(TOPK(600), TOPK(600)), (QSGD(2048), QSGD(2048)), (SIGN(4096), TOPK(300))]:
        gs = [g.cuda() for g in randn_steps(n, d, 2 * T, seed=17)]
        one = DoubleSqueeze(n, d, 0.1, wq, sq, seed=5)
        for t, g in enumerate(gs):
            one.step(g, t)
        first = DoubleSqueeze(n, d, 0.1, wq, sq, seed=5)
        for t, g in enumerate(gs[:T]):
            first.step(g, t)
        second = DoubleSqueeze(n, d, 0.1, wq, sq, seed=5, x0=first.x)
        second.delta_w.copy_(first.delta_w)
        second.delta_s.copy_(first.delta_s)
        for t, g in enumerate(gs[T:]):
            second.step(g, T + t)
        torch.cuda.synchronize()
        for a, b in ((one.x, second.x), (one.delta_w, second.delta_w), (one.delta_s, second.delta_s),
                     (one.server_payload, second.server_payload), (one.worker_payload, second.worker_payload)):
            assert torch.equal(a.view(torch.uint8) if a.dtype == torch.uint8 else a.view(torch.int32),
                               b.view(torch.uint8) if b.dtype == torch.uint8 else b.view(torch.int32))
        assert one.device_status() == 0 and second.device_status() == 0


def test_calls_out_of_order_are_refused_on_a_live_handle():
    ds = DoubleSqueeze(2, 5000, 0.1, SIGN(1024), SIGN(1024))
    g = torch.randn(2, 5000, device="cuda")
    with pytest.raises(Exception, match="-4"):
        ds.server_aggregate_compress(0)
    ds.worker_compress(g, 0)
    with pytest.raises(Exception, match="-4"):
        ds.worker_compress(g, 0)
    with pytest.raises(Exception, match="-4"):
        ds.apply_update()
    ds.server_aggregate_compress(0, fuse_apply=False)
    ds.apply_update()
    ds.step(g, 1)
    torch.cuda.synchronize()


def test_host_buffer_step_equals_device_step_and_counts_launches():
    from paper_1905_05957_b200 import load_library
    n, d = 3, 40_000 + 8
    wq, sq = SIGN(4096), TOPK(400)
    gs = randn_steps(n, d, 3, seed=23)
    a = DoubleSqueeze(n, d, 0.1, wq, sq, seed=9)
    b = DoubleSqueeze(n, d, 0.1, wq, sq, seed=9)
    stage = torch.empty(n, d, device="cuda")
    out = torch.empty(b.server_payload.numel(), dtype=torch.uint8).pin_memory()
    x_host = torch.empty(d).pin_memory()
    before = load_library().ds_kernel_launches()
    for t, g in enumerate(gs):
        a.step(g.cuda(), t)
        b.step_host(g.contiguous().pin_memory(), stage, t, server_payload_host=out, x_host=x_host)
        torch.cuda.synchronize()
        assert torch.equal(a.x.view(torch.int32), b.x.view(torch.int32))
        assert torch.equal(a.server_payload, b.server_payload)
        assert torch.equal(out, b.server_payload.cpu())
        assert torch.equal(x_host.view(torch.int32), b.x.cpu().view(torch.int32))
    assert load_library().ds_kernel_launches() > before


def test_more_workers_than_one_batch_of_the_server_loops():
    # 150 sparse payloads (the ordered sum walks them in batches of 128) and 150 one-bit payloads
    run_lockstep(150, 9000, TOPK(90), TOPK(90), randn_steps(150, 9000, 2, seed=31))
    run_lockstep(150, 4096 + 100, SIGN(1024), QSGD(512, 63), randn_steps(150, 4096 + 100, 2, seed=32))


# ------------------------------------------------------------------ seeded random configurations

def _random_q(r, d):
    kind = r.choice(["sign1", "sign1_l2", "qsgd", "topk", "clip", "identity", "rsparse"])
    if kind == "rsparse":
        return RSP(int(r.choice([2, 4, 16, 64])), int(r.choice([128, 1024, 4096])), int(r.integers(0, 2)))
    if kind == "sign1":
        return SIGN(int(r.choice([128, 256, 512, 1024, 2048, 4096, 8192])))
    if kind == "sign1_l2":
        return SIGN_L2(int(r.choice([128, 512, 2048, 4096])))
    if kind == "qsgd":
        return QSGD(int(r.choice([128, 256, 1024, 2048, 4096])), int(r.choice([1, 2, 7, 100, 255])))
    if kind == "topk":
        return TOPK(int(r.integers(0, max(1, d // 20) + 1)))
    if kind == "clip":
        return CLIP(int(r.choice([16, 24])))
    return IDENT


@pytest.mark.parametrize("case", range(24))
def test_random_configurations(case):
    """Operator pair, sizes, scale of the data and the form of the update all drawn from the case number."""
    r = np.random.default_rng(1905 + case)
    n = int(r.integers(1, 10))
    d = int(r.choice([r.integers(1, 200), r.integers(200, 20_000), r.integers(20_000, 150_000)]))
    if r.random() < 0.5:
        d = max(4, d // 4 * 4)
    wq, sq = _random_q(r, d), _random_q(r, d)
    scale = float(10.0 ** r.uniform(-4, 2))
    gs = randn_steps(n, d, 3, seed=case, scale=scale)
    run_lockstep(n, d, wq, sq, gs, gamma=float(r.choice([0.1, 0.01, 1.0])), seed=int(r.integers(0, 2**62)),
                 fuse=bool(r.random() < 0.5))
