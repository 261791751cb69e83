"""Pins for the oracle's compression operators (Section 3.2 / Section 5.1 of the paper)."""
import math

import numpy as np
import pytest

import oracle


def _rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ 1-bit with scale

@pytest.mark.parametrize("d,L", [(4096, 4096), (10000, 4096), (777, 128), (33, 4096), (1, 128)])
def test_sign1_scale_is_l1_mean_per_chunk_and_bits_are_signs(d, L):
    v = _rng(d).standard_normal(d).astype(np.float32)
    v[::7] = 0.0
    if d > 5:
        v[5] = -0.0
    C, p = oracle.q_sign1(v, L)
    nc = (d + L - 1) // L
    for c in range(nc):
        seg = v[c * L:(c + 1) * L].astype(np.float64)
        s = np.abs(seg).sum() / len(seg)        # ||v_c||_1 / len_c in float64
        assert abs(float(p["scale"][c]) - s) <= 1e-6 * s + 1e-30
        # recovered chunk has the same l1 magnitude as the compensated one
        assert abs(np.abs(C[c * L:(c + 1) * L].astype(np.float64)).sum() - np.abs(seg).sum()) <= 2e-6 * np.abs(seg).sum()
    want_bits = np.packbits((v >= 0).astype(np.uint8), bitorder="little")
    want_bits = np.concatenate([want_bits, np.zeros((-len(want_bits)) % 4, np.uint8)]).view(np.uint32)
    assert np.array_equal(p["bits"], want_bits)
    # +0 and -0 both map to +scale
    assert not np.signbit(C[v == 0]).any()
    assert np.array_equal(np.signbit(C), v < 0)
    assert np.array_equal(oracle.decode_sign1(p["bits"], p["scale"], d, L), C)


def test_sign1_residual_energy_closed_form_and_constant_chunk():
    L = 4096
    v = _rng(11).standard_normal(3 * L).astype(np.float32)
    C, p = oracle.q_sign1(v, L)
    delta = oracle.residual(v, C).astype(np.float64)
    for c in range(3):
        seg = v[c * L:(c + 1) * L].astype(np.float64)
        closed = (seg**2).sum() - np.abs(seg).sum() ** 2 / L   # ||v||^2 - ||v||_1^2 / len
        got = (delta[c * L:(c + 1) * L] ** 2).sum()
        assert abs(got - closed) <= 1e-5 * (seg**2).sum()
    # a chunk of constant magnitude is represented exactly: residual identically zero
    w = np.where(_rng(12).random(L) < 0.5, np.float32(0.375), np.float32(-0.375)).astype(np.float32)
    C, p = oracle.q_sign1(w, L)
    assert float(p["scale"][0]) == 0.375 and np.array_equal(C, w)
    assert not oracle.residual(w, C).any()


def test_sign1_short_last_chunk_divides_by_true_length():
    L = 128
    v = np.full(L + 3, 2.0, dtype=np.float32)
    _, p = oracle.q_sign1(v, L)
    assert p["scale"].tolist() == [2.0, 2.0]   # a divide by L would give 6/128


@pytest.mark.parametrize("d,L", [(4096, 4096), (10000, 4096), (777, 128), (33, 4096), (1, 128)])
def test_sign1_l2_scale_is_rms_and_keeps_the_l2_magnitude(d, L):
    """With l2 magnitudes (the norm Section 3.2 prints) the factor of Section 5.1 is
    ||v_c||_2 / ||sign(v_c)||_2 = ||v_c||_2 / sqrt(len_c), and the recovered chunk has the l2
    magnitude of the compensated one."""
    v = _rng(3 * d + 1).standard_normal(d).astype(np.float32)
    v[::5] = 0.0
    C, p = oracle.q_sign1(v, L, norm=2)
    C1, p1 = oracle.q_sign1(v, L, norm=1)
    nc = (d + L - 1) // L
    for c in range(nc):
        seg = v[c * L:(c + 1) * L].astype(np.float64)
        rms = math.sqrt((seg**2).sum() / len(seg))
        assert abs(float(p["scale"][c]) - rms) <= 1e-6 * rms + 1e-30
        got = math.sqrt((C[c * L:(c + 1) * L].astype(np.float64) ** 2).sum())
        assert abs(got - math.sqrt((seg**2).sum())) <= 2e-6 * math.sqrt((seg**2).sum()) + 1e-30
        # root mean square >= mean absolute value (Cauchy-Schwarz), equal only for constant |v|
        assert float(p["scale"][c]) >= float(p1["scale"][c]) * (1 - 1e-6)
    assert np.array_equal(p["bits"], p1["bits"])           # the signs do not depend on the norm
    assert np.array_equal(oracle.decode_sign1(p["bits"], p["scale"], d, L), C)


def test_sign1_l2_constant_chunk_short_chunk_and_residual_energy():
    L = 4096
    # constant magnitude: l2 and l1 factors coincide and the chunk is represented exactly
    w = np.where(_rng(13).random(L) < 0.5, np.float32(0.375), np.float32(-0.375)).astype(np.float32)
    C, p = oracle.q_sign1(w, L, norm=2)
    assert float(p["scale"][0]) == 0.375 and np.array_equal(C, w)
    # short last chunk: the root of the TRUE length divides (sqrt(4 * 9) / sqrt(4) = 3)
    v = np.full(128 + 4, 3.0, dtype=np.float32)
    _, p = oracle.q_sign1(v, 128, norm=2)
    assert p["scale"].tolist() == [3.0, 3.0]
    # residual energy: ||v - s sign(v)||^2 = 2 ||v||_2^2 - 2 s ||v||_1 with s = ||v||_2 / sqrt(len)
    v = _rng(14).standard_normal(2 * L).astype(np.float32)
    C, p = oracle.q_sign1(v, L, norm=2)
    delta = oracle.residual(v, C).astype(np.float64)
    for c in range(2):
        seg = v[c * L:(c + 1) * L].astype(np.float64)
        s = math.sqrt((seg**2).sum() / L)
        closed = 2 * (seg**2).sum() - 2 * s * np.abs(seg).sum()
        assert abs((delta[c * L:(c + 1) * L] ** 2).sum() - closed) <= 1e-5 * (seg**2).sum()


def test_sign1_rejects_unknown_norm():
    with pytest.raises(ValueError):
        oracle.q_sign1(np.ones(8, np.float32), 128, norm=3)


# ------------------------------------------------------------------ top-k

def _brute_topk(v, k):
    key = v.view(np.uint32) & 0x7FFFFFFF
    order = sorted(range(len(v)), key=lambda j: (-int(key[j]), j))
    return np.array(sorted(order[:k]), dtype=np.uint32)


@pytest.mark.parametrize("d,k", [(1, 0), (1, 1), (17, 0), (17, 1), (17, 16), (17, 17), (200, 13), (64, 32)])
def test_topk_matches_brute_force_with_ties(d, k):
    r = _rng(100 * d + k)
    v = r.integers(-3, 4, size=d).astype(np.float32)   # few distinct magnitudes => many ties
    if d > 3:
        v[1] = -0.0
        v[2] = 0.0
    C, p = oracle.q_topk(v, k)
    want = _brute_topk(v, k)
    assert np.array_equal(p["idx"], want)
    assert np.array_equal(p["val"].view(np.uint32), v[want].view(np.uint32))
    dense = np.zeros(d, dtype=np.float32)
    dense[want] = v[want]
    assert np.array_equal(C.view(np.uint32), dense.view(np.uint32))
    assert np.array_equal(oracle.decode_topk(p["idx"], p["val"], d).view(np.uint32), dense.view(np.uint32))


def test_topk_all_equal_takes_lowest_indices_and_matches_partition():
    v = np.full(50, -1.5, dtype=np.float32)
    _, p = oracle.q_topk(v, 7)
    assert p["idx"].tolist() == list(range(7))
    r = _rng(5)
    v = r.standard_normal(5000).astype(np.float32)     # distinct magnitudes almost surely
    k = 123
    _, p = oracle.q_topk(v, k)
    want = np.sort(np.argpartition(-np.abs(v), k - 1)[:k]).astype(np.uint32)   # library selection
    assert np.array_equal(p["idx"], want)
    # energy identity ||delta||^2 = ||v||^2 - sum_sel v^2 and the (1 - k/d) contraction
    C, _ = oracle.q_topk(v, k)
    delta = oracle.residual(v, C).astype(np.float64)
    v64 = v.astype(np.float64)
    assert abs((delta**2).sum() - ((v64**2).sum() - (v64[want] ** 2).sum())) < 1e-9
    assert (delta**2).sum() <= (1 - k / len(v)) * (v64**2).sum()
    # residual is exactly v off the support and +0 on it
    assert np.array_equal(delta[np.setdiff1d(np.arange(len(v)), want)], v64[np.setdiff1d(np.arange(len(v)), want)])
    assert not delta[want].any()


def test_topk_rejects_k_above_d():
    with pytest.raises(ValueError):
        oracle.q_topk(np.zeros(4, dtype=np.float32), 5)


# ------------------------------------------------------------------ randomised quantisation

def test_qsgd_unbiased_and_variance_by_monte_carlo():
    L, s = 128, 4            # few levels => large quantisation noise, a sharp test
    r = _rng(21)
    v = (r.standard_normal(L) * np.exp(r.standard_normal(L))).astype(np.float32)
    M = 4000
    acc = np.zeros(L)
    acc2 = np.zeros(L)
    for m in range(M):
        C, p = oracle.q_qsgd(v, L, s, seed=99, step=m, wid=3)
        acc += C
        acc2 += C.astype(np.float64) ** 2
    N = float(p["norm"][0])
    q = N / s
    rr = np.minimum(np.abs(v.astype(np.float64)) / q, s)
    pfrac = rr - np.floor(rr)
    var = q * q * pfrac * (1 - pfrac)              # two-point law on {a, b}: (b-a)^2 p (1-p)
    mean = acc / M
    sd = np.sqrt(var / M)
    assert np.all(np.abs(mean - v) <= 4.5 * sd + 1e-6 * np.abs(v))
    emp_var = acc2 / M - mean**2
    big = var > 0.05 * q * q
    assert np.all(np.abs(emp_var[big] - var[big]) <= 0.15 * var[big])
    # chunk norm is the l2 norm
    assert abs(N - math.sqrt((v.astype(np.float64) ** 2).sum())) <= 1e-6 * N


def test_qsgd_deterministic_special_cases():
    L, s = 128, 255
    # single non-zero entry: |v| = N, so it sits on the top grid point with probability one
    v = np.zeros(L, dtype=np.float32)
    v[17] = -3.0
    for step in range(20):
        C, p = oracle.q_qsgd(v, L, s, 1, step, 0)
        assert p["lvl"][17] == s and p["lvl"].sum() == s
        assert C[17] == np.float32(-(np.float32(s) * (np.float32(3.0) / np.float32(s))))
        assert not (p["sgn"][0] >> 17) & 1 and bin(int(p["sgn"][0])).count("1") == 31
    # all-zero chunk -> all zero, stored norm 0, residual equals v
    z = np.zeros(L, dtype=np.float32)
    C, p = oracle.q_qsgd(z, L, s, 1, 0, 0)
    assert not C.any() and not p["lvl"].any() and p["norm"][0] == 0
    # entries exactly on grid points stay there: v = (3,4) scaled => N = 5 * scale, s = 5
    v = np.zeros(L, dtype=np.float32)
    v[0], v[1] = 3.0, -4.0
    for step in range(20):
        C, p = oracle.q_qsgd(v, L, 5, 7, step, 2)
        assert p["lvl"][0] == 3 and p["lvl"][1] == 4 and p["norm"][0] == 5.0
        assert C[0] == 3.0 and C[1] == -4.0
    # norm so small that s/N overflows, and a norm that overflows: both sent as zeros
    tiny = np.zeros(L, dtype=np.float32)
    tiny[0] = 1e-30     # square underflows to a subnormal; s/N = inf
    C, p = oracle.q_qsgd(tiny, L, s, 1, 0, 0)
    assert not C.any() and p["norm"][0] == 0
    huge = np.full(L, 3e19, dtype=np.float32)
    C, p = oracle.q_qsgd(huge, L, s, 1, 0, 0)
    assert not C.any() and p["norm"][0] == 0


def test_qsgd_levels_bracket_the_value_and_decode_roundtrip():
    d, L, s = 5000, 2048, 255
    v = (_rng(31).standard_t(3, d) * 1e-3).astype(np.float32)
    C, p = oracle.q_qsgd(v, L, s, 5, 9, 1)
    q = np.repeat(p["norm"].astype(np.float64) / s, L)[:d]
    rr = np.abs(v.astype(np.float64)) / q
    lv = p["lvl"].astype(np.float64)
    assert np.all(lv >= np.floor(rr) - 1e-3) and np.all(lv <= np.floor(rr) + 1 + 1e-3)
    assert np.all(np.abs(C.astype(np.float64) - v) <= q * (1 + 1e-5))
    assert np.array_equal(oracle.decode_qsgd(p["lvl"], p["sgn"], p["step"], d, L), C)
    assert np.array_equal(p["step"], p["norm"] / np.float32(s))     # what is sent is q = N / s
    # the random stream depends on step, worker and seed, and on nothing else
    C2, p2 = oracle.q_qsgd(v, L, s, 5, 9, 1)
    assert np.array_equal(p["lvl"], p2["lvl"])
    for kw in (dict(seed=6, step=9, wid=1), dict(seed=5, step=10, wid=1), dict(seed=5, step=9, wid=2)):
        _, p3 = oracle.q_qsgd(v, L, s, **kw)
        assert not np.array_equal(p["lvl"], p3["lvl"])
    # the uniform used by entry j is word (t % 4) of the Philox block with counter (t // 4, chunk, wid, step)
    j = 2048 + 6
    w = oracle.philox4x32_10([6 // 4, 1, 1, 9], [5, 0])[6 % 4]
    u = (int(w) >> 8) * 2.0**-24
    inv_q = np.float32(s) / p["norm"][1]
    r = np.float32(abs(v[j])) * inv_q
    want = int(np.floor(r)) + (1 if u < float(r - np.floor(r)) else 0)
    assert p["lvl"][j] == want


# ------------------------------------------------------------------ clipping

def test_clip_worked_binary_cases():
    """The clipping option of Section 3.2 drops low-order bits of a number (its example drops decimal
    digits); for binary32 with b = 16 the sign, the exponent and 7 fraction bits survive."""
    one = np.float32(1.0)
    cases16 = [
        (1.0, 1.0), (-2.0, -2.0), (1.5, 1.5), (0.0, 0.0),
        (1.0 + 2.0**-7, 1.0 + 2.0**-7),          # the last surviving fraction bit
        (1.0 + 2.0**-8, 1.0),                    # the first cleared one
        (1.0 + 2.0**-7 + 2.0**-9, 1.0 + 2.0**-7),
        (-(3.0 + 2.0**-10), -3.0),               # truncation is toward zero for negatives too
        (1.9999999, 1.9921875),                  # 1 + 127/128: never rounds up to 2
        (float(np.float32(3.14159265)), 3.140625),
    ]
    v = np.array([c[0] for c in cases16], dtype=np.float32)
    want = np.array([c[1] for c in cases16], dtype=np.float32)
    C, p = oracle.q_clip(v, 16)
    assert np.array_equal(C, want)
    assert p["hi"].dtype == np.uint16 and int(p["hi"][0]) == 0x3F80 and int(p["hi"][1]) == 0xC000
    # b = 24 keeps the sign and the seven high bits of the biased exponent: 1.0 = 0x3F800000 has
    # exponent field 127 = 0b01111111, whose low bit goes, leaving 126, i.e. 0.5; 3.0 = 0x40400000
    # keeps field 128, i.e. 2.0; 2^-126 (field 1) falls to 0; 1e30 = 0x7149F2CA -> 0x71000000 = 2^99
    C, p = oracle.q_clip(np.array([1.0, -1.0, 3.0, 0.75, 2.0**-126, 1e30], dtype=np.float32), 24)
    assert C.tolist() == [0.5, -0.5, 2.0, 0.5, 0.0, float(2.0**99)]
    assert p["hi"].dtype == np.uint8 and p["hi"].tolist() == [0x3F, 0xBF, 0x40, 0x3F, 0x00, 0x71] and one == 1.0
    with pytest.raises(ValueError):
        oracle.q_clip(v, 12)


@pytest.mark.parametrize("b", [16, 24])
def test_clip_error_bound_idempotence_exact_residual_and_decode(b):
    r = _rng(50 + b)
    v = (r.standard_normal(20000) * 10.0 ** r.uniform(-6, 6, 20000)).astype(np.float32)
    v[:4] = [0.0, -0.0, 1e-41, -1e-41]
    C, p = oracle.q_clip(v, b)
    # never grows, never changes sign, and equals the value with its low b bits cleared
    assert np.all(np.abs(C) <= np.abs(v)) and np.array_equal(np.signbit(C), np.signbit(v))
    mask = np.uint32((0xFFFFFFFF << b) & 0xFFFFFFFF)
    assert np.array_equal(C.view(np.uint32), v.view(np.uint32) & mask)
    if b == 16:   # truncating 16 of the 23 fraction bits: relative error below 2^-7 on normal numbers
        normal = np.abs(v) >= 2.0**-126
        assert np.all(np.abs(v[normal].astype(np.float64) - C[normal]) < 2.0**-7 * np.abs(v[normal]))
    # clipping what is already clipped changes nothing
    C2, p2 = oracle.q_clip(C, b)
    assert np.array_equal(C2.view(np.uint32), C.view(np.uint32)) and np.array_equal(p2["hi"], p["hi"])
    # the residual is exact: Q[v] + (v - Q[v]) gives v back bit for bit
    delta = oracle.residual(v, C)
    assert np.array_equal(C.astype(np.float64) + delta.astype(np.float64), v.astype(np.float64))
    assert np.array_equal(oracle.decode_clip(p["hi"], v.size, b).view(np.uint32), C.view(np.uint32))
    # a contraction (Section 4 needs ||v - Q[v]|| <= alpha ||v|| with alpha < 1 on what it is applied to)
    assert np.linalg.norm(delta.astype(np.float64)) < np.linalg.norm(v.astype(np.float64))


# ------------------------------------------------------------------ randomised sparsification

@pytest.mark.parametrize("scaled", [0, 1])
def test_rsparse_structure_of_what_is_sent(scaled):
    """One draw per chunk: exactly L/S survivors per full chunk, S apart; scaled by S exactly or kept."""
    L, S, d = 256, 8, 3 * 256 + 100
    v = _rng(61).standard_normal(d).astype(np.float32)
    C, p = oracle.q_rsparse(v, L, S, scaled, seed=5, step=2, wid=1)
    f = np.float32(S if scaled else 1)
    assert p["off"].shape == (4,) and np.all(p["off"] < S) and p["val"].shape == (4 * L // S,)
    for c in range(4):
        seg = slice(c * L, min((c + 1) * L, d))
        o = int(p["off"][c])
        want = np.arange(o, seg.stop - seg.start, S)
        mask = np.zeros(seg.stop - seg.start, bool)
        mask[want] = True
        assert np.array_equal(C[seg][mask], f * v[seg][mask]) and not C[seg][~mask].any()   # power of two: exact
        slots = p["val"][c * (L // S):(c + 1) * (L // S)]
        assert np.array_equal(slots[:len(want)], C[seg][want]) and not slots[len(want):].any()
        w = oracle.philox4x32_10([0xFFFFFFFF, c, 1, 2], [5, 0])     # the draw: first word, counter as documented
        assert o == int(w[0]) % S
    assert np.array_equal(oracle.decode_rsparse(p["val"], p["off"], d, L, S), C)
    others = [oracle.q_rsparse(v, L, S, scaled, 5, 2, 2)[1]["off"], oracle.q_rsparse(v, L, S, scaled, 5, 3, 1)[1]["off"],
              oracle.q_rsparse(v, L, S, scaled, 6, 2, 1)[1]["off"]]
    assert all(not np.array_equal(o2, p["off"]) for o2 in others)   # other worker, step, seed: other draws
    with pytest.raises(ValueError):
        oracle.q_rsparse(v, L, 3, scaled, 5, 2, 1)
    with pytest.raises(ValueError):
        oracle.q_rsparse(v, L, 2 * L, scaled, 5, 2, 1)


def test_rsparse_keeps_each_entry_with_probability_one_in_S_and_scaled_form_is_unbiased():
    """Section 3.2: survive with probability p (here 1/S) and scale by 1/p, else 0 => E Q[v] = v."""
    L, S, d, M = 128, 4, 512, 4000
    v = _rng(62).standard_normal(d).astype(np.float32)
    acc = np.zeros(d)
    kept = np.zeros(d)
    err2 = [0.0, 0.0]
    for t in range(M):
        C, _ = oracle.q_rsparse(v, L, S, 1, seed=9, step=t, wid=0)
        acc += C
        kept += C != 0
        err2[1] += float(((v - C).astype(np.float64) ** 2).sum())
        C0, _ = oracle.q_rsparse(v, L, S, 0, seed=9, step=t, wid=0)
        err2[0] += float(((v - C0).astype(np.float64) ** 2).sum())
    freq = kept / M
    sigma = math.sqrt((1 / S) * (1 - 1 / S) / M)
    assert np.all(np.abs(freq - 1 / S) < 5 * sigma)                 # per-entry keep frequency
    tol = 5 * np.abs(v) * math.sqrt((S - 1) / M) + 1e-12            # Var Q_j = v_j^2 (S - 1)
    assert np.all(np.abs(acc / M - v) <= tol)
    # the four offsets of a chunk are equally likely (chi-square, 3 degrees of freedom)
    offs = np.array([oracle.q_rsparse(v[:L], L, S, 1, 9, t, 0)[1]["off"][0] for t in range(M)])
    counts = np.bincount(offs, minlength=S)
    assert ((counts - M / S) ** 2 / (M / S)).sum() < 21.1           # P(chi2_3 > 21.1) ~ 1e-4
    # mean squared error: (S - 1) ||v||^2 scaled (no contraction), (1 - 1/S) ||v||^2 unscaled (a contraction)
    n2 = float((v.astype(np.float64) ** 2).sum())
    assert abs(err2[1] / M / n2 - (S - 1)) < 0.05 * (S - 1) and abs(err2[0] / M / n2 - (1 - 1 / S)) < 0.05
