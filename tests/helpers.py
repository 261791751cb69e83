"""Shared test plumbing: run the oracle and the CUDA library side by side and compare."""
from __future__ import annotations

import numpy as np

import oracle
from paper_1905_05957_b200.workloads import Q

REL_TOL = 1e-5   # bar for fp32 values, scales and delta (reduction order may differ)


def to_oracle_q(q: Q) -> oracle.QSpec:
    return oracle.qspec_from(q)


def u32(t) -> np.ndarray:
    """Device int32/uint8 tensor -> host array with unsigned bits."""
    a = t.detach().cpu().numpy()
    if a.dtype == np.int16:
        return a.view(np.uint16)
    return a.view(np.uint32) if a.dtype == np.int32 else a


def assert_float_match(name: str, got: np.ndarray, want: np.ndarray, scale: np.ndarray | float | None = None):
    """The stated bar (max relative error 1e-5 against |want|, or against `scale` where the value is a
    difference of larger numbers), and then the stronger fact that holds because both sides use the
    same summation tree: identical bits."""
    got = np.asarray(got, dtype=np.float32)
    want = np.asarray(want, dtype=np.float32)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    ref = np.abs(want).astype(np.float64) if scale is None else np.broadcast_to(np.asarray(scale, np.float64), want.shape)
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bad = err > REL_TOL * ref + 1e-45
    assert not bad.any(), f"{name}: {int(bad.sum())} of {bad.size} beyond 1e-5 relative; worst {err.max()}"
    same = got.view(np.uint32) == want.view(np.uint32)
    assert same.all(), f"{name}: {int((~same).sum())} of {same.size} differ in bits (first at {np.argmin(same.reshape(-1))})"


def assert_bits_match(name: str, got: np.ndarray, want: np.ndarray):
    assert got.shape == want.shape, (name, got.shape, want.shape)
    same = got == want
    assert same.all(), f"{name}: {int((~same).sum())} of {same.size} differ (first at {np.argmin(same.reshape(-1))})"


def compare_payload(name: str, op: str, gpu_views: dict, ora: dict):
    if op == "identity":
        assert_float_match(f"{name}.c", u32(gpu_views["c"]).view(np.float32), ora["c"])
    elif op == "sign1":
        assert_bits_match(f"{name}.bits", u32(gpu_views["bits"]), ora["bits"])
        assert_float_match(f"{name}.scale", gpu_views["scale"].cpu().numpy(), ora["scale"])
    elif op == "topk":
        assert_bits_match(f"{name}.idx", u32(gpu_views["idx"]), ora["idx"])
        assert_bits_match(f"{name}.val", u32(gpu_views["val"].view(dtype=__import__("torch").int32)),
                          ora["val"].view(np.uint32))
    elif op == "qsgd":
        assert_bits_match(f"{name}.lvl", u32(gpu_views["lvl"]), ora["lvl"])
        assert_bits_match(f"{name}.sgn", u32(gpu_views["sgn"]), ora["sgn"])
        assert_float_match(f"{name}.step", gpu_views["step"].cpu().numpy(), ora["step"])
    elif op == "rsparse":
        assert_bits_match(f"{name}.off", u32(gpu_views["off"]), ora["off"])
        assert_bits_match(f"{name}.val", u32(gpu_views["val"].view(dtype=__import__("torch").int32)), ora["val"].view(np.uint32))
    elif op == "ternary":
        assert_bits_match(f"{name}.sgn", u32(gpu_views["sgn"]), ora["sgn"])
        assert_bits_match(f"{name}.nz", u32(gpu_views["nz"]), ora["nz"])
        assert_float_match(f"{name}.scale", gpu_views["scale"].cpu().numpy(), ora["scale"])
    elif op == "clip":
        assert_bits_match(f"{name}.hi", u32(gpu_views["hi"]), ora["hi"])
    else:
        raise ValueError(op)


def compare_state(ds, st: oracle.State, g_host: np.ndarray, tag: str = ""):
    """Everything one step leaves behind: payloads, both errors, the model."""
    wq, sq = ds.worker_q.op, ds.server_q.op
    for i, (gv, ov) in enumerate(zip(ds.worker_views(), st.worker_payloads)):
        compare_payload(f"{tag}worker[{i}]", wq, gv, ov)
    compare_payload(f"{tag}server", sq, ds.server_views(), st.server_payload)
    # delta = v - Q[v] is a difference: relative to |v| + |Q[v]|, bounded here by |g| + |delta| scale
    mag = float(np.abs(g_host).max()) + float(np.abs(st.delta_w).max()) + 1e-30
    if ds.compensate:   # without compensation there are no errors (delta_s may exist as scratch: not compared)
        assert_float_match(f"{tag}delta_w", ds.delta_w.cpu().numpy(), st.delta_w, scale=mag)
        assert_float_match(f"{tag}delta_s", ds.delta_s.cpu().numpy(), st.delta_s, scale=mag)
    assert_float_match(f"{tag}x", ds.x.cpu().numpy(), st.x, scale=np.abs(st.x).astype(np.float64) + ds.gamma * mag)
    assert ds.device_status() == 0, f"{tag}device status {ds.device_status():#x}"
