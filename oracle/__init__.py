"""CPU oracle for the DoubleSqueeze step -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front of ``dsq_oracle.c`` plus the composition of one
iteration of Algorithm 1 in the paper's order (worker: Eq. 2, compress, Eq. 3;
server: Eq. 4, compress, residual; worker: model update).  Nothing in the CUDA
package imports this module and this module imports nothing from it.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass, field

import numpy as np

from . import build as _build

IDENTITY, SIGN1, TOPK, QSGD, CLIP, RSPARSE, TERNARY = "identity", "sign1", "topk", "qsgd", "clip", "rsparse", "ternary"
SERVER_WID = 0xFFFFFFFF

_lib = None


def load(path: str):
    """Opens an oracle shared library and declares its signatures."""
    L = C.CDLL(path)
    f32p, u32p, u8p = C.POINTER(C.c_float), C.POINTER(C.c_uint32), C.POINTER(C.c_uint8)
    u64, u32 = C.c_uint64, C.c_uint32
    L.orc_pairwise_sum.restype = C.c_float
    L.orc_pairwise_sum.argtypes = [f32p, u64]
    L.orc_pairwise_sum_padded.restype = C.c_float
    L.orc_pairwise_sum_padded.argtypes = [f32p, u64, u64]
    L.orc_server_mean.restype = None
    L.orc_server_mean.argtypes = [f32p, u32, u64, f32p]
    L.orc_q_ternary.argtypes = [f32p, u64, u64, u32, u32, u32p, u32p, f32p, f32p, f32p]
    L.orc_decode_ternary.argtypes = [u32p, u32p, f32p, u64, f32p]
    L.orc_philox4x32_10.restype = None
    L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
    L.orc_ef_add.restype = None
    L.orc_ef_add.argtypes = [f32p, f32p, u64, f32p]
    L.orc_residual.restype = None
    L.orc_residual.argtypes = [f32p, f32p, u64, f32p]
    L.orc_server_mean_add.restype = None
    L.orc_server_mean_add.argtypes = [f32p, u32, u64, f32p, f32p]
    L.orc_apply_update.restype = None
    L.orc_apply_update.argtypes = [f32p, f32p, C.c_float, u64]
    L.orc_q_identity.argtypes = [f32p, u64, f32p]
    L.orc_q_sign1.argtypes = [f32p, u64, u32, u32, u32p, f32p, f32p]
    L.orc_decode_sign1.argtypes = [u32p, f32p, u64, u32, f32p]
    L.orc_q_topk.argtypes = [f32p, u64, u64, u32p, f32p, f32p]
    L.orc_decode_topk.argtypes = [u32p, f32p, u64, u64, f32p]
    L.orc_q_qsgd.argtypes = [f32p, u64, u32, u32, u64, u32, u32, u8p, u32p, f32p, f32p, f32p]
    L.orc_decode_qsgd.argtypes = [u8p, u32p, f32p, u64, u32, f32p]
    L.orc_q_clip.argtypes = [f32p, u64, u32, u8p, f32p]
    L.orc_decode_clip.argtypes = [u8p, u64, u32, f32p]
    L.orc_q_rsparse.argtypes = [f32p, u64, u32, u32, u32, u64, u32, u32, f32p, u32p, f32p]
    L.orc_decode_rsparse.argtypes = [f32p, u32p, u64, u32, u32, f32p]
    return L


def lib():
    global _lib
    if _lib is None:
        _lib = load(_build.build())
    return _lib


def _p(a: np.ndarray, ct):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ct))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with code {rc}")


# ----------------------------------------------------------------------------
# primitives
# ----------------------------------------------------------------------------

def pairwise_sum(a) -> np.float32:
    a = _f32(a)
    return np.float32(lib().orc_pairwise_sum(_p(a, C.c_float), a.size))


def pairwise_sum_padded(a, L) -> np.float32:
    """Pairwise sum of a padded with +0 to L entries (L a power of two >= len(a))."""
    a = _f32(a)
    return np.float32(lib().orc_pairwise_sum_padded(_p(a, C.c_float), a.size, L))


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def ef_add(g, delta) -> np.ndarray:
    g, delta = _f32(g), _f32(delta)
    v = np.empty_like(g)
    lib().orc_ef_add(_p(g, C.c_float), _p(delta, C.c_float), g.size, _p(v, C.c_float))
    return v


def residual(v, Cv) -> np.ndarray:
    v, Cv = _f32(v), _f32(Cv)
    out = np.empty_like(v)
    lib().orc_residual(_p(v, C.c_float), _p(Cv, C.c_float), v.size, _p(out, C.c_float))
    return out


def server_mean_add(C_all, delta_s) -> np.ndarray:
    C_all, delta_s = _f32(C_all), _f32(delta_s)
    n, d = C_all.shape
    v = np.empty(d, dtype=np.float32)
    lib().orc_server_mean_add(_p(C_all, C.c_float), n, d, _p(delta_s, C.c_float), _p(v, C.c_float))
    return v


def server_mean(C_all) -> np.ndarray:
    """(1/n) sum_i Q[v_i] alone: the server's vector when no error is carried."""
    C_all = _f32(C_all)
    n, d = C_all.shape
    v = np.empty(d, dtype=np.float32)
    lib().orc_server_mean(_p(C_all, C.c_float), n, d, _p(v, C.c_float))
    return v


def apply_update(x, Cv, gamma) -> np.ndarray:
    x = _f32(x).copy()
    Cv = _f32(Cv)
    lib().orc_apply_update(_p(x, C.c_float), _p(Cv, C.c_float), C.c_float(gamma), x.size)
    return x


# ----------------------------------------------------------------------------
# compression operators Q (Section 3.2).  Each returns (C, payload dict).
# ----------------------------------------------------------------------------

@dataclass(frozen=True)
class QSpec:
    op: str = IDENTITY
    chunk: int = 0      # sign1 / qsgd / rsparse: chunk length L (power of two); sign1: 0 = one factor for the whole vector
    norm: int = 1       # sign1: the scale is the ratio of l1 (1) or l2 (2) magnitudes
    k: int = 0          # topk
    levels: int = 0     # qsgd: s
    keep_one_in: int = 0  # rsparse: S, an element survives with probability 1/S
    scaled: int = 0     # rsparse: 1 = survivors are multiplied by S (unbiased), 0 = kept as they are
    bits: int = 0       # clip: how many low bits of each binary32 number are set to zero (16 or 24)


def qspec_from(q) -> "QSpec":
    """A QSpec with the fields of any object that names an operator the same way (duck-typed: the
    oracle imports nothing from the code it checks)."""
    return QSpec(**{f: getattr(q, f) for f in QSpec.__dataclass_fields__ if hasattr(q, f)})


def q_identity(v):
    v = _f32(v)
    Cv = np.empty_like(v)
    _check(lib().orc_q_identity(_p(v, C.c_float), v.size, _p(Cv, C.c_float)), "identity")
    return Cv, {"c": Cv.copy()}


def q_sign1(v, L, norm=1):
    v = _f32(v)
    d = v.size
    bits = np.zeros((d + 31) // 32, dtype=np.uint32)
    scale = np.zeros((d + L - 1) // L if L else 1, dtype=np.float32)
    Cv = np.empty_like(v)
    _check(lib().orc_q_sign1(_p(v, C.c_float), d, L, norm, _p(bits, C.c_uint32), _p(scale, C.c_float),
                             _p(Cv, C.c_float)), "sign1")
    return Cv, {"bits": bits, "scale": scale}


def decode_sign1(bits, scale, d, L):
    Cv = np.empty(d, dtype=np.float32)
    bits = np.ascontiguousarray(bits, dtype=np.uint32)
    scale = _f32(scale)
    _check(lib().orc_decode_sign1(_p(bits, C.c_uint32), _p(scale, C.c_float), d, L, _p(Cv, C.c_float)),
           "decode_sign1")
    return Cv


def q_ternary(v, seed, step, wid):
    v = _f32(v)
    d = v.size
    sgn = np.zeros((d + 31) // 32, dtype=np.uint32)
    nz = np.zeros((d + 31) // 32, dtype=np.uint32)
    scale = np.zeros(1, dtype=np.float32)
    vmax = np.zeros(1, dtype=np.float32)
    Cv = np.empty_like(v)
    _check(lib().orc_q_ternary(_p(v, C.c_float), d, C.c_uint64(seed), step, wid, _p(sgn, C.c_uint32), _p(nz, C.c_uint32),
                               _p(scale, C.c_float), _p(vmax, C.c_float), _p(Cv, C.c_float)), "ternary")
    # the payload is (sgn, nz, scale); the largest magnitude is returned as well for the tests that pin it
    return Cv, {"sgn": sgn, "nz": nz, "scale": scale, "max": vmax}


def decode_ternary(sgn, nz, scale, d):
    sgn = np.ascontiguousarray(sgn, dtype=np.uint32)
    nz = np.ascontiguousarray(nz, dtype=np.uint32)
    scale = _f32(scale)
    Cv = np.empty(d, dtype=np.float32)
    _check(lib().orc_decode_ternary(_p(sgn, C.c_uint32), _p(nz, C.c_uint32), _p(scale, C.c_float), d, _p(Cv, C.c_float)),
           "decode_ternary")
    return Cv


def q_topk(v, k):
    v = _f32(v)
    d = v.size
    idx = np.zeros(max(k, 1), dtype=np.uint32)
    val = np.zeros(max(k, 1), dtype=np.float32)
    Cv = np.empty_like(v)
    _check(lib().orc_q_topk(_p(v, C.c_float), d, k, _p(idx, C.c_uint32), _p(val, C.c_float),
                            _p(Cv, C.c_float)), "topk")
    return Cv, {"idx": idx[:k], "val": val[:k]}


def decode_topk(idx, val, d):
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    val = _f32(val)
    Cv = np.empty(d, dtype=np.float32)
    _check(lib().orc_decode_topk(_p(idx, C.c_uint32), _p(val, C.c_float), idx.size, d, _p(Cv, C.c_float)),
           "decode_topk")
    return Cv


def q_qsgd(v, L, s, seed, step, wid):
    v = _f32(v)
    d = v.size
    lvl = np.zeros(d, dtype=np.uint8)
    sgn = np.zeros((d + 31) // 32, dtype=np.uint32)
    norm = np.zeros((d + L - 1) // L, dtype=np.float32)
    qstep = np.zeros_like(norm)
    Cv = np.empty_like(v)
    _check(lib().orc_q_qsgd(_p(v, C.c_float), d, L, s, C.c_uint64(seed), step, wid, _p(lvl, C.c_uint8),
                            _p(sgn, C.c_uint32), _p(norm, C.c_float), _p(qstep, C.c_float), _p(Cv, C.c_float)), "qsgd")
    # the payload is (lvl, sgn, step); the chunk norm N is returned as well for the tests that pin it
    return Cv, {"lvl": lvl, "sgn": sgn, "step": qstep, "norm": norm}


def decode_qsgd(lvl, sgn, qstep, d, L):
    lvl = np.ascontiguousarray(lvl, dtype=np.uint8)
    sgn = np.ascontiguousarray(sgn, dtype=np.uint32)
    qstep = _f32(qstep)
    Cv = np.empty(d, dtype=np.float32)
    _check(lib().orc_decode_qsgd(_p(lvl, C.c_uint8), _p(sgn, C.c_uint32), _p(qstep, C.c_float), d, L,
                                 _p(Cv, C.c_float)), "decode_qsgd")
    return Cv


def q_clip(v, b):
    v = _f32(v)
    d = v.size
    hi = np.zeros(d * ((32 - b) // 8 if b in (16, 24) else 1), dtype=np.uint8)
    Cv = np.empty_like(v)
    _check(lib().orc_q_clip(_p(v, C.c_float), d, b, _p(hi, C.c_uint8), _p(Cv, C.c_float)), "clip")
    return Cv, {"hi": hi.view(np.uint16) if b == 16 else hi}


def decode_clip(hi, d, b):
    hi = np.ascontiguousarray(hi).view(np.uint8)
    Cv = np.empty(d, dtype=np.float32)
    _check(lib().orc_decode_clip(_p(hi, C.c_uint8), d, b, _p(Cv, C.c_float)), "decode_clip")
    return Cv


def q_rsparse(v, L, S, scaled, seed, step, wid):
    v = _f32(v)
    d = v.size
    nc = (d + L - 1) // L
    val = np.zeros(nc * max(L // max(S, 1), 1), dtype=np.float32)
    off = np.zeros(nc, dtype=np.uint32)
    Cv = np.empty_like(v)
    _check(lib().orc_q_rsparse(_p(v, C.c_float), d, L, S, scaled, C.c_uint64(seed), step, wid, _p(val, C.c_float),
                               _p(off, C.c_uint32), _p(Cv, C.c_float)), "rsparse")
    return Cv, {"val": val, "off": off}


def decode_rsparse(val, off, d, L, S):
    val = _f32(val)
    off = np.ascontiguousarray(off, dtype=np.uint32)
    Cv = np.empty(d, dtype=np.float32)
    _check(lib().orc_decode_rsparse(_p(val, C.c_float), _p(off, C.c_uint32), d, L, S, _p(Cv, C.c_float)), "decode_rsparse")
    return Cv


def compress(q: QSpec, v, seed=0, step=0, wid=0):
    """Q_omega[v] for the operator ``q``; omega = (seed, step, wid) where Q is random."""
    if q.op == IDENTITY:
        return q_identity(v)
    if q.op == SIGN1:
        return q_sign1(v, q.chunk, q.norm)
    if q.op == TOPK:
        return q_topk(v, q.k)
    if q.op == QSGD:
        return q_qsgd(v, q.chunk, q.levels, seed, step, wid)
    if q.op == CLIP:
        return q_clip(v, q.bits)
    if q.op == RSPARSE:
        return q_rsparse(v, q.chunk, q.keep_one_in, q.scaled, seed, step, wid)
    if q.op == TERNARY:
        return q_ternary(v, seed, step, wid)
    raise ValueError(q.op)


# ----------------------------------------------------------------------------
# Algorithm 1, one iteration
# ----------------------------------------------------------------------------

@dataclass
class State:
    """x, the n worker errors delta^(i) and the server error delta (all zero at t = 0)."""
    x: np.ndarray
    delta_w: np.ndarray
    delta_s: np.ndarray
    worker_payloads: list = field(default_factory=list)
    server_payload: dict = field(default_factory=dict)

    @staticmethod
    def zeros(n: int, d: int, x0=None) -> "State":
        x = np.zeros(d, dtype=np.float32) if x0 is None else _f32(x0).copy()
        return State(x, np.zeros((n, d), dtype=np.float32), np.zeros(d, dtype=np.float32))


def worker_pass(st: State, g, worker_q: QSpec, seed: int, step: int, compensate: bool = True) -> np.ndarray:
    """Worker side of Algorithm 1 for all n workers; returns the dense [n, d] Q[v_i].
    compensate=False: Section 5.1's methods without compensation: Q[g_i] is sent, no error is kept."""
    g = _f32(g)
    n, d = g.shape
    C_all = np.empty((n, d), dtype=np.float32)
    st.worker_payloads = []
    for i in range(n):
        if compensate:
            v = ef_add(g[i], st.delta_w[i])                    # Eq. 2
        else:
            v = g[i]
        Cv, payload = compress(worker_q, v, seed, step, i)     # compress
        if compensate:
            st.delta_w[i] = residual(v, Cv)                    # Eq. 3
        C_all[i] = Cv
        st.worker_payloads.append(payload)
    return C_all


def server_pass(st: State, C_all, server_q: QSpec, seed: int, step: int, compensate: bool = True) -> np.ndarray:
    """Server side of Algorithm 1 (Eq. 4); returns the dense Q[v] sent to the workers."""
    v = server_mean_add(C_all, st.delta_s) if compensate else server_mean(C_all)
    Cv, payload = compress(server_q, v, seed, step, SERVER_WID)
    if compensate:
        st.delta_s = residual(v, Cv)
    st.server_payload = payload
    return Cv


def step(st: State, g, worker_q: QSpec, server_q: QSpec, gamma: float, seed: int, t: int,
         compensate: bool = True) -> np.ndarray:
    """One full iteration of Algorithm 1; mutates ``st`` and returns the dense server Q[v]."""
    C_all = worker_pass(st, g, worker_q, seed, t, compensate)
    Cv = server_pass(st, C_all, server_q, seed, t, compensate)
    st.x = apply_update(st.x, Cv, gamma)
    return Cv
