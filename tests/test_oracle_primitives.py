"""Pins for the oracle's building blocks: summation order, Philox, elementwise steps."""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _cases():
    out = []
    with open(os.path.join(GOLDEN, "pairwise_sum_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            exp, inp = line.split("|")
            out.append((eval(exp), [eval(t) for t in inp.split(",")]))
    return out


@pytest.mark.parametrize("expected,inputs", _cases())
def test_pairwise_sum_hand_derived(expected, inputs):
    got = oracle.pairwise_sum(np.array(inputs, dtype=np.float32))
    assert float(got) == float(np.float32(expected))


def test_pairwise_sum_exact_on_integers_and_error_bound():
    rng = np.random.default_rng(1)
    a = rng.integers(-1000, 1000, size=4096).astype(np.float32)
    assert float(oracle.pairwise_sum(a)) == float(a.astype(np.int64).sum())
    for L in (128, 2048, 4096):
        b = np.abs(rng.standard_normal(L)).astype(np.float32)
        exact = math.fsum(b.astype(np.float64))
        got = float(oracle.pairwise_sum(b))
        # pairwise summation error bound: log2(L) * u * sum|a| (Higham, Accuracy and Stability, ch. 4)
        assert abs(got - exact) <= math.log2(L) * 2.0**-24 * exact * 1.01


def test_pairwise_sum_rejects_non_power_of_two():
    assert math.isnan(float(oracle.pairwise_sum(np.ones(3, dtype=np.float32))))


def test_philox_matches_independent_library():
    """Philox4x32-10 against Triton's own implementation run by its CPU interpreter."""
    os.environ["TRITON_INTERPRET"] = "1"
    try:
        import torch
        import triton
        import triton.language as tl
    except Exception as e:  # pragma: no cover
        pytest.skip(f"triton unavailable: {e}")

    @triton.jit
    def kern(out_ptr, cptr, seed, N: tl.constexpr):
        offs = tl.arange(0, N)
        c0 = tl.load(cptr + offs)
        c1 = tl.load(cptr + N + offs)
        c2 = tl.load(cptr + 2 * N + offs)
        c3 = tl.load(cptr + 3 * N + offs)
        a, b, c, d = tl.philox(seed, c0, c1, c2, c3, 10)
        tl.store(out_ptr + offs, a)
        tl.store(out_ptr + N + offs, b)
        tl.store(out_ptr + 2 * N + offs, c)
        tl.store(out_ptr + 3 * N + offs, d)

    N = 64
    rng = np.random.default_rng(7)
    ctr = rng.integers(0, 2**32, size=(4, N), dtype=np.uint64).astype(np.uint32)
    ctr[:, 0] = 0
    ctr[:, 1] = 0xFFFFFFFF
    for seed in (0, 12345, 190505957, (0xDEADBEEF << 32) | 0x01234567):
        out = torch.zeros(4 * N, dtype=torch.int32)
        try:
            kern[(1,)](out, torch.from_numpy(ctr.view(np.int32).reshape(-1).copy()), seed, N)
        except Exception as e:  # pragma: no cover
            pytest.skip(f"triton interpreter unavailable: {e}")
        ref = out.numpy().view(np.uint32).reshape(4, N)
        key = [seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF]
        for j in range(N):
            got = oracle.philox4x32_10(ctr[:, j], key)
            assert got.tolist() == ref[:, j].tolist(), (seed, j)


def test_philox_structure_and_uniformity():
    key = [190505957 & 0xFFFFFFFF, 0]
    # distinct counters -> distinct outputs (the rounds are a bijection of the counter)
    outs = {tuple(oracle.philox4x32_10([c, 0, 0, 0], key).tolist()) for c in range(2000)}
    assert len(outs) == 2000
    # changing any one input word changes the block
    base = oracle.philox4x32_10([1, 2, 3, 4], key)
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] ^= 1
        assert oracle.philox4x32_10(c, key).tolist() != base.tolist()
    assert oracle.philox4x32_10([1, 2, 3, 4], [key[0] ^ 1, 0]).tolist() != base.tolist()
    assert oracle.philox4x32_10([1, 2, 3, 4], [key[0], 1]).tolist() != base.tolist()
    # 24-bit uniforms: chi-square over 64 buckets, mean 1/2
    words = np.concatenate([oracle.philox4x32_10([c, 5, 6, 7], key) for c in range(8192)])
    u = (words >> 8).astype(np.float64) * 2.0**-24
    assert abs(u.mean() - 0.5) < 4 * (1 / 12) ** 0.5 / len(u) ** 0.5
    hist, _ = np.histogram(u, bins=64, range=(0, 1))
    chi2 = ((hist - len(u) / 64) ** 2 / (len(u) / 64)).sum()
    assert chi2 < 63 + 6 * (2 * 63) ** 0.5
    # bit balance of every output bit
    bits = ((words[:, None] >> np.arange(32)) & 1).mean(axis=0)
    assert np.all(np.abs(bits - 0.5) < 5 * 0.5 / len(words) ** 0.5)


def test_elementwise_steps_are_single_roundings():
    rng = np.random.default_rng(3)
    g = rng.standard_normal(1000).astype(np.float32)
    dl = (rng.standard_normal(1000) * 1e-3).astype(np.float32)
    assert np.array_equal(oracle.ef_add(g, dl), g + dl)          # Eq. 2, numpy fp32 add
    assert np.array_equal(oracle.residual(g, dl), g - dl)        # Eq. 3
    x = rng.standard_normal(1000).astype(np.float32)
    gam = np.float32(0.1)
    assert np.array_equal(oracle.apply_update(x, g, 0.1), x - gam * g)
    # a fused multiply-add would differ on some of these; make sure the data can tell
    fused = (x.astype(np.float64) - np.float64(gam) * g.astype(np.float64)).astype(np.float32)
    assert not np.array_equal(fused, x - gam * g)


def test_server_mean_special_cases():
    rng = np.random.default_rng(4)
    d = 513
    ds = rng.standard_normal(d).astype(np.float32)
    c0 = rng.standard_normal(d).astype(np.float32)
    # n = 1: v = C_0 + delta_s
    assert np.array_equal(oracle.server_mean_add(c0[None], ds), c0 + ds)
    # two identical workers: c + c and the halving are exact, so the mean is each of them
    assert np.array_equal(oracle.server_mean_add(np.tile(c0, (2, 1)), ds), c0 + ds)
    # eight identical workers: 3c, 5c, ... round, so only close
    got8 = oracle.server_mean_add(np.tile(c0, (8, 1)), ds)
    assert np.max(np.abs(got8 - (c0.astype(np.float64) + ds))) <= 8 * 2.0**-24 * np.max(np.abs(c0) + np.abs(ds))
    # general n against float64 (n = 3: 1/3 is rounded, so allow a few ulps)
    Call = rng.standard_normal((3, d)).astype(np.float32)
    ref = Call.astype(np.float64).mean(axis=0) + ds
    got = oracle.server_mean_add(Call, ds)
    assert np.max(np.abs(got - ref)) <= 4 * 2.0**-24 * np.max(np.abs(Call).sum(axis=0) + np.abs(ds))
    # order of accumulation is worker 0 first: [big, -big, small] keeps small, a reversed sum too,
    # but [small, big, -big] loses it
    big, small = np.float32(2**25), np.float32(1)
    z = np.zeros(1, dtype=np.float32)
    kept = oracle.server_mean_add(np.array([[big], [-big], [small], [0]], dtype=np.float32), z)
    lost = oracle.server_mean_add(np.array([[small], [big], [-big], [0]], dtype=np.float32), z)
    assert kept[0] == 0.25 and lost[0] == 0.0
