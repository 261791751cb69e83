"""Pins for the oracle functions that work on a whole vector at once: the 1-bit operator with one
scaling factor (Section 3.2 "1-Bit Quantization", Section 5.1 "1-bit compression"), the ternary
quantiser (Section 5.1, "Implementations and setups", item 2) and the passes without error
compensation (items 2 and 5)."""
import numpy as np
import pytest

import oracle
from oracle import QSpec


def _v(d, seed=0, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(d) * scale).astype(np.float32)


# ------------------------------------------------------------------ padded pairwise sum

@pytest.mark.parametrize("n,L", [(1, 1), (1, 8), (3, 4), (5, 8), (1000, 1024), (1025, 2048), (4096, 4096)])
def test_padded_pairwise_sum_equals_the_sum_over_the_written_out_padding(n, L):
    a = np.abs(_v(n, seed=n + L, scale=3.0))
    padded = np.zeros(L, dtype=np.float32)
    padded[:n] = a
    assert oracle.pairwise_sum_padded(a, L).view(np.uint32) == oracle.pairwise_sum(padded).view(np.uint32)


def test_padded_pairwise_sum_is_not_a_running_sum():
    # 2^24 + 1 + 1 + 1 ...: a running sum in binary32 never moves off 2^24, the pairwise tree does
    a = np.ones(6, dtype=np.float32)
    a[0] = 2.0**24
    got = float(oracle.pairwise_sum_padded(a, 8))
    assert got == 2.0**24 + 4.0      # (2^24+1 -> 2^24) + (1+1) = 2^24+2 ; (1+1) + 0 = 2 ; total 2^24 + 4


# ------------------------------------------------------------------ 1-bit with one factor

@pytest.mark.parametrize("d", [1, 7, 1000, 4097, 100_003])
def test_whole_vector_sign_scale_is_the_ratio_of_magnitudes(d):
    v = _v(d, seed=d, scale=0.01)
    C1, p1 = oracle.q_sign1(v, 0, 1)
    C2, p2 = oracle.q_sign1(v, 0, 2)
    v64 = v.astype(np.float64)
    assert p1["scale"].shape == (1,) and p2["scale"].shape == (1,)
    # magnitude of v over magnitude of sign(v): ||v||_1 / d and ||v||_2 / sqrt(d)
    assert abs(p1["scale"][0] - np.abs(v64).sum() / d) <= 1e-6 * np.abs(v64).mean()
    assert abs(p2["scale"][0] - np.sqrt((v64**2).sum() / d)) <= 1e-6 * np.sqrt((v64**2).mean())
    want_bits = np.packbits(np.concatenate([v >= 0, np.zeros((-d) % 32, bool)]), bitorder="little").view(np.uint32)
    assert np.array_equal(p1["bits"], want_bits) and np.array_equal(p2["bits"], want_bits)
    assert np.array_equal(C1, np.where(v >= 0, p1["scale"][0], -p1["scale"][0]).astype(np.float32))
    # the recovered vector has the magnitude of v in the chosen norm
    assert abs(np.abs(C1.astype(np.float64)).sum() - np.abs(v64).sum()) <= 1e-5 * np.abs(v64).sum()
    assert abs(np.linalg.norm(C2.astype(np.float64)) - np.linalg.norm(v64)) <= 1e-5 * np.linalg.norm(v64)
    assert np.array_equal(oracle.decode_sign1(p1["bits"], p1["scale"], d, 0), C1)
    # closed form of the residual energy for the l1 factor: ||v - Q[v]||^2 = ||v||^2 - ||v||_1^2 / d
    r = (v64 - C1.astype(np.float64))
    assert abs((r**2).sum() - ((v64**2).sum() - np.abs(v64).sum() ** 2 / d)) <= 1e-4 * (v64**2).sum()


@pytest.mark.parametrize("d", [128, 4096, 8192])
def test_whole_vector_sign_equals_one_chunk_of_the_same_length(d):
    """A vector that is exactly one chunk long: the whole-vector form and the chunked form are the same
    sum over the same tree, so they agree bit for bit."""
    v = _v(d, seed=3)
    for norm in (1, 2):
        Ca, pa = oracle.q_sign1(v, 0, norm)
        Cb, pb = oracle.q_sign1(v, d, norm)
        assert pa["scale"].view(np.uint32)[0] == pb["scale"].view(np.uint32)[0]
        assert np.array_equal(Ca, Cb) and np.array_equal(pa["bits"], pb["bits"])


def test_whole_vector_sign_short_vector_divides_by_its_true_length():
    v = np.full(1000, 2.0, dtype=np.float32)     # padded to 1024 for the sum; the length that divides is 1000
    v[::2] = -2.0
    for norm in (1, 2):
        C, p = oracle.q_sign1(v, 0, norm)
        assert p["scale"][0] == 2.0 and np.array_equal(C, v)


# ------------------------------------------------------------------ ternary quantiser

def test_ternary_structure_scale_and_the_documented_philox_word():
    d, seed, step, wid = 1003, (7 << 32) + 11, 5, 2
    v = _v(d, seed=1, scale=0.02)
    v[17] = 0.0
    C, p = oracle.q_ternary(v, seed, step, wid)
    m = np.float32(np.abs(v).max())
    assert p["max"][0] == m
    nz = np.unpackbits(p["nz"].view(np.uint8), bitorder="little")[:d].astype(bool)
    sg = np.unpackbits(p["sgn"].view(np.uint8), bitorder="little")[:d].astype(bool)
    assert np.array_equal(sg, v >= 0)
    assert not np.unpackbits(p["nz"].view(np.uint8), bitorder="little")[d:].any()      # pad bits are 0
    # entry j survives iff u < |v_j| / m, u the top 24 bits of word j % 4 of counter (j / 4, 0xFFFFFFFE, wid, step)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for j in list(range(0, 40)) + [d - 1, d - 2, 500]:
        w = oracle.philox4x32_10([j // 4, 0xFFFFFFFE, wid, step], key)[j % 4]
        u = np.float32(int(w) >> 8) * np.float32(2.0**-24)
        assert bool(nz[j]) == bool(u < np.float32(abs(v[j])) / m), j
    assert nz[np.argmax(np.abs(v))] and not nz[17]
    # one factor: magnitude of v over magnitude of the ternary vector, l1: ||v||_1 / (number of non-zeros)
    count = int(nz.sum())
    want = np.abs(v.astype(np.float64)).sum() / count
    assert abs(p["scale"][0] - want) <= 1e-6 * want
    s = p["scale"][0]
    assert np.array_equal(C, np.where(nz, np.where(sg, s, -s), 0.0).astype(np.float32))
    assert abs(np.abs(C.astype(np.float64)).sum() - np.abs(v.astype(np.float64)).sum()) <= 1e-5 * np.abs(v).sum()
    assert np.array_equal(oracle.decode_ternary(p["sgn"], p["nz"], p["scale"], d), C)
    # other worker / step / seed: other draws
    for other in [(seed, step, wid + 1), (seed, step + 1, wid), (seed + 1, step, wid), (seed, step, oracle.SERVER_WID)]:
        assert not np.array_equal(oracle.q_ternary(v, *other)[1]["nz"], p["nz"])


def test_ternary_is_unbiased_before_scaling_and_keeps_the_largest_entry_always():
    """P(kept) = |e| / |m| (Section 5.1, item 2), so m * sign(e) * kept has mean e: Monte Carlo over
    independent streams; the entry equal to m is kept in every one of them."""
    d, M = 64, 4000
    v = _v(d, seed=9)
    v[5] = 0.0
    top = int(np.argmax(np.abs(v)))
    m = float(np.abs(v).max())
    acc = np.zeros(d)
    kept_top = 0
    for s in range(M):
        _, p = oracle.q_ternary(v, 1000 + s, s % 7, s % 3)
        nz = np.unpackbits(p["nz"].view(np.uint8), bitorder="little")[:d].astype(np.float64)
        kept_top += int(nz[top])
        acc += m * np.sign(v) * nz
    assert kept_top == M
    mean = acc / M
    prob = np.abs(v) / m
    sigma = m * np.sqrt(prob * (1 - prob) / M)
    assert np.all(np.abs(mean - v) <= 4.5 * sigma + 1e-12)
    assert mean[5] == 0.0


def test_ternary_degenerate_vectors():
    z = np.zeros(100, dtype=np.float32)
    C, p = oracle.q_ternary(z, 1, 0, 0)
    assert not C.any() and p["scale"][0] == 0.0 and not p["nz"].any() and p["max"][0] == 0.0
    one = np.zeros(70, dtype=np.float32)
    one[33] = -3.5
    C, p = oracle.q_ternary(one, 1, 0, 0)
    assert np.array_equal(C, one) and p["scale"][0] == 3.5      # the only non-zero entry is the maximum: kept, factor |m|
    c = np.full(257, 0.25, dtype=np.float32)                     # constant magnitude: every entry is a maximum
    c[::3] = -0.25
    C, p = oracle.q_ternary(c, 1, 0, 0)
    assert np.array_equal(C, c)


# ------------------------------------------------------------------ passes without compensation

OPS = {"topk": QSpec(oracle.TOPK, k=29), "sign1": QSpec(oracle.SIGN1, chunk=128), "ternary": QSpec(oracle.TERNARY),
       "identity": QSpec(oracle.IDENTITY), "qsgd": QSpec(oracle.QSGD, chunk=128, levels=7)}


def _grads(n, d, T, seed=0):
    r = np.random.default_rng(seed)
    mu = r.standard_normal((n, d)).astype(np.float32)
    return [(mu + 0.5 * r.standard_normal((n, d))).astype(np.float32) for _ in range(T)]


@pytest.mark.parametrize("wq,sq", [("topk", "identity"), ("ternary", "identity"), ("sign1", "topk"), ("qsgd", "sign1")])
def test_without_compensation_the_model_follows_plain_compressed_sgd(wq, sq):
    """Section 5.1, items 2 and 5: x <- x - gamma Q_s[(1/n) sum_i Q_w[g_i]], nothing else: the errors are
    neither read nor written."""
    n, d, T, gamma, seed = 3, 500, 5, 0.1, 12
    gs = _grads(n, d, T, seed=3)
    st = oracle.State.zeros(n, d)
    r = np.random.default_rng(5)
    st.delta_w[:] = r.standard_normal((n, d)).astype(np.float32)      # must be ignored and left alone
    st.delta_s[:] = r.standard_normal(d).astype(np.float32)
    dw0, ds0 = st.delta_w.copy(), st.delta_s.copy()
    x = np.zeros(d, dtype=np.float32)
    for t, g in enumerate(gs):
        oracle.step(st, g, OPS[wq], OPS[sq], gamma, seed, t, compensate=False)
        acc = np.zeros(d, dtype=np.float32)
        for i in range(n):
            acc = acc + oracle.compress(OPS[wq], g[i], seed, t, i)[0]
        mean = acc * np.float32(1.0 / n)
        x = x - np.float32(gamma) * oracle.compress(OPS[sq], mean, seed, t, oracle.SERVER_WID)[0]
        assert np.array_equal(st.x, x)
        assert np.array_equal(st.delta_w, dw0) and np.array_equal(st.delta_s, ds0)


def test_without_compensation_identity_is_parallel_sgd_and_top_k_loses_what_it_drops():
    n, d, T, gamma = 4, 640, 25, 0.1
    gs = _grads(n, d, T, seed=9)
    sgd = -gamma * sum(g.astype(np.float64).mean(axis=0) for g in gs)
    a, b = oracle.State.zeros(n, d), oracle.State.zeros(n, d)
    for t, g in enumerate(gs):
        oracle.step(a, g, OPS["identity"], OPS["identity"], gamma, 0, t, compensate=False)
        oracle.step(b, g, OPS["identity"], OPS["identity"], gamma, 0, t, compensate=True)
    assert np.array_equal(a.x, b.x) and np.max(np.abs(a.x - sgd)) < 1e-4
    # top-k: with compensation x - gamma * Omega telescopes onto the SGD path (Eq. 5-6); without it the
    # dropped entries are gone for good and x alone is far from the SGD path
    with_c, without = oracle.State.zeros(n, d), oracle.State.zeros(n, d)
    for t, g in enumerate(gs):
        oracle.step(with_c, g, OPS["topk"], OPS["topk"], gamma, 0, t, compensate=True)
        oracle.step(without, g, OPS["topk"], OPS["topk"], gamma, 0, t, compensate=False)
    omega = with_c.delta_s.astype(np.float64) + with_c.delta_w.astype(np.float64).mean(axis=0)
    assert np.max(np.abs(with_c.x - gamma * omega - sgd)) < 1e-4
    assert np.max(np.abs(without.x - sgd)) > 0.5
    assert not without.delta_w.any() and not without.delta_s.any()
