"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, lays payloads out as documented, and rejects bad arguments."""
import ctypes as C
import os
import re

import pytest

from paper_1905_05957_b200 import binding as b
from paper_1905_05957_b200 import build as libbuild
from paper_1905_05957_b200.workloads import Q

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return b.load_library()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "dsq.h")).read()
    declared = set(re.findall(r"^\s*(?:int|const char\*|uint64_t)\s+(ds_\w+)\s*\(", header, flags=re.M))
    assert declared == set(b.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert lib.ds_version() >= 100


def test_struct_sizes_match_the_header():
    assert C.sizeof(b.ds_qspec) == 24
    assert C.sizeof(b.ds_config) == 24 + 24 + 24 + 8
    assert C.sizeof(b.ds_buffers) == 13 * 8
    assert C.sizeof(b.ds_payload_layout) == 56


def test_layouts(lib):
    d, n = 11_689_512, 8
    cfg = b.make_config(n, d, 0.1, Q("sign1", chunk=4096), Q("qsgd", chunk=2048, levels=255), 1)
    w = b.get_layout(cfg, 0)
    nw, nc = (d + 31) // 32, (d + 4095) // 4096
    assert list(w.count)[:2] == [nw, nc] and w.off[0] == 0 and w.off[1] == (4 * nw + 15) // 16 * 16
    assert w.stride % 16 == 0 and w.stride >= w.off[1] + 4 * nc
    s = b.get_layout(cfg, 1)
    assert list(s.count) == [d, nw, (d + 2047) // 2048]
    assert s.off[1] % 16 == 0 and s.off[1] >= d and s.off[2] % 16 == 0 and s.off[2] >= s.off[1] + 4 * nw
    cfg = b.make_config(2, 1000, 0.1, Q("topk", k=10), Q("identity"), 1)
    t = b.get_layout(cfg, 0)
    assert list(t.count)[:2] == [10, 10] and t.off[1] == 48 and t.stride == 96
    assert b.get_layout(cfg, 1).count[0] == 1000
    cfg = b.make_config(2, 1000, 0.1, Q("topk", k=0), Q("topk", k=0), 1)
    assert b.get_layout(cfg, 0).stride == 16     # never a zero stride
    cfg = b.make_config(2, 1001, 0.1, Q("clip", bits=16), Q("clip", bits=24), 1)
    c16, c24 = b.get_layout(cfg, 0), b.get_layout(cfg, 1)
    assert c16.count[0] == 1001 and c16.stride == (2 * 1001 + 15) // 16 * 16
    assert c24.count[0] == 1001 and c24.stride == (1001 + 15) // 16 * 16
    cfg = b.make_config(2, 10_000, 0.1, Q("rsparse", chunk=4096, keep_one_in=32), Q("identity"), 1)
    rs = b.get_layout(cfg, 0)
    assert list(rs.count)[:2] == [3 * 128, 3] and rs.off[1] == 3 * 128 * 4
    # the l2-magnitude variant of the 1-bit operator shares the payload format
    a = b.get_layout(b.make_config(2, 5000, 0.1, Q("sign1", chunk=128), Q("identity"), 1), 0)
    l2 = b.get_layout(b.make_config(2, 5000, 0.1, Q("sign1", chunk=128, norm=2), Q("identity"), 1), 0)
    assert (a.stride, list(a.off), list(a.count)) == (l2.stride, list(l2.off), list(l2.count))


def test_layouts_of_the_whole_vector_operators_and_sizes_without_compensation(lib):
    d, n = 100_003, 4
    nw = (d + 31) // 32
    cfg = b.make_config(n, d, 0.1, Q("sign1", chunk=0), Q("ternary"), 1)
    w, s = b.get_layout(cfg, 0), b.get_layout(cfg, 1)
    assert list(w.count)[:2] == [nw, 1] and w.off[1] == (4 * nw + 15) // 16 * 16 and w.stride == w.off[1] + 16
    assert list(s.count) == [nw, nw, 1] and s.off[1] == w.off[1] and s.off[2] == 2 * w.off[1] and s.stride == s.off[2] + 16
    bufs = b.ds_buffers()
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    ntile = (d + 4095) // 4096
    assert bufs.workspace_bytes >= 2 * n * ntile * 4 + 16 * n        # tile sums, tile maxima / counts, per-vector results
    assert bufs.delta_w_bytes == 4 * n * d and bufs.delta_s_bytes == 4 * d
    # without compensation no error buffer is asked for, except delta_s as the top-k server's scratch
    cfg = b.make_config(n, d, 0.1, Q("topk", k=10), Q("identity"), 1, compensate=False)
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    assert bufs.delta_w_bytes == 0 and bufs.delta_s_bytes == 0
    cfg = b.make_config(n, d, 0.1, Q("ternary"), Q("topk", k=10), 1, compensate=False)
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    assert bufs.delta_w_bytes == 0 and bufs.delta_s_bytes == 4 * d
    # a handle without error buffers
    cfg = b.make_config(2, 1000, 0.1, Q("sign1", chunk=128), Q("identity"), 0, compensate=False)
    bufs = b.ds_buffers()
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    bufs.x, bufs.worker_payload, bufs.server_payload, bufs.dev_status = 0x10000, 0x20000, 0x30000, 0x40000
    h = C.c_void_p()
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), C.byref(h)) == b.DS_OK
    assert lib.ds_destroy(h) == b.DS_OK
    # unknown flag bits are refused
    cfg.flags = 2
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_ERR_INVALID_ARG
    # an instance that keeps the errors of one block of workers: delta_w shrinks, the payload buffers do not
    bufs = b.ds_buffers()
    cfg = b.make_config(8, d, 0.1, Q("sign1", chunk=4096), Q("sign1", chunk=4096), 1, delta_w_rows=2)
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    assert bufs.delta_w_bytes == 2 * 4 * d and bufs.worker_payload_bytes == 8 * b.get_layout(cfg, 0).stride
    cfg = b.make_config(8, d, 0.1, Q("sign1", chunk=4096), Q("sign1", chunk=4096), 1, delta_w_rows=9)
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_ERR_INVALID_ARG


def test_query_mode_reports_sizes(lib):
    cfg = b.make_config(16, 25_557_032, 0.1, Q("topk", k=255_570), Q("topk", k=255_570), 1)
    bufs = b.ds_buffers()
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    assert bufs.x_bytes == 4 * 25_557_032 and bufs.delta_w_bytes == 16 * bufs.x_bytes
    assert bufs.worker_payload_bytes == 16 * b.get_layout(cfg, 0).stride
    assert bufs.workspace_bytes > 4 * 25_557_032           # bitmaps + dense accumulator
    cfg = b.make_config(8, 1 << 20, 0.1, Q("sign1", chunk=4096), Q("sign1", chunk=4096), 1)
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    assert bufs.workspace_bytes == 0


@pytest.mark.parametrize("kw", [
    dict(n=0), dict(d=0), dict(d=1 << 32), dict(gamma=float("nan")), dict(gamma=float("inf")), dict(n=70_000),
    dict(worker_q=Q("sign1", chunk=1000)), dict(worker_q=Q("sign1", chunk=64)), dict(worker_q=Q("sign1", chunk=16384)),
    dict(server_q=Q("qsgd", chunk=2048, levels=0)), dict(server_q=Q("qsgd", chunk=2048, levels=256)),
    dict(worker_q=Q("topk", k=1001)),
    dict(worker_q=Q("sign1", chunk=4096, norm=3)), dict(server_q=Q("clip", bits=12)), dict(server_q=Q("clip", bits=0)),
    dict(worker_q=Q("clip", bits=32)),
    dict(worker_q=Q("rsparse", chunk=4096, keep_one_in=3)), dict(server_q=Q("rsparse", chunk=4096, keep_one_in=256)),
    dict(server_q=Q("rsparse", chunk=100, keep_one_in=4)), dict(worker_q=Q("rsparse", chunk=4096, keep_one_in=4, scaled=2)),
    dict(worker_q=Q("ternary", chunk=4096)), dict(worker_q=Q("qsgd", chunk=0, levels=255)),
])
def test_bad_configs_are_rejected(lib, kw):
    args = dict(n=4, d=1000, gamma=0.1, worker_q=Q("identity"), server_q=Q("identity"), seed=0)
    args.update(kw)
    cfg = b.make_config(**args)
    bufs = b.ds_buffers()
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_ERR_INVALID_ARG
    assert lib.ds_get_layout(C.byref(cfg), 0, C.byref(b.ds_payload_layout())) == b.DS_ERR_INVALID_ARG


def test_bad_buffers_are_rejected_without_touching_a_gpu(lib):
    cfg = b.make_config(2, 1000, 0.1, Q("sign1", chunk=128), Q("topk", k=10), 0)
    bufs = b.ds_buffers()
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_NEED_BUFFERS
    h = C.c_void_p()
    base = 0x10000     # fake, never dereferenced: ds_create is host-only
    def fill(bb):
        bb.x, bb.delta_w, bb.delta_s = base, base + 0x10000, base + 0x20000
        bb.worker_payload, bb.server_payload, bb.workspace, bb.dev_status = (base + 0x30000, base + 0x40000,
                                                                              base + 0x50000, base + 0x60000)
    fill(bufs)
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), C.byref(h)) == b.DS_OK
    # calls out of order
    assert lib.ds_server_aggregate_compress(h, 0, 0, None) == b.DS_ERR_STATE
    assert lib.ds_apply_update(h, None) == b.DS_ERR_STATE
    assert lib.ds_worker_compress(h, None, 0, None) == b.DS_ERR_INVALID_ARG
    assert lib.ds_server_aggregate_compress(h, 0, 8, None) == b.DS_ERR_INVALID_ARG
    assert lib.ds_destroy(h) == b.DS_OK
    assert lib.ds_destroy(None) == b.DS_ERR_INVALID_ARG
    bad = b.ds_buffers.from_buffer_copy(bufs)
    bad.delta_s = base + 0x20004
    assert lib.ds_create(C.byref(cfg), C.byref(bad), C.byref(h)) == b.DS_ERR_ALIGN
    bad = b.ds_buffers.from_buffer_copy(bufs)
    bad.worker_payload_bytes -= 1
    assert lib.ds_create(C.byref(cfg), C.byref(bad), C.byref(h)) == b.DS_ERR_BUFFER_TOO_SMALL
    bad = b.ds_buffers.from_buffer_copy(bufs)
    bad.workspace = None
    assert lib.ds_create(C.byref(cfg), C.byref(bad), C.byref(h)) == b.DS_ERR_INVALID_ARG
    bad = b.ds_buffers.from_buffer_copy(bufs)
    bad.dev_status = None
    assert lib.ds_create(C.byref(cfg), C.byref(bad), C.byref(h)) == b.DS_ERR_INVALID_ARG
    assert lib.ds_create(C.byref(cfg), C.byref(bufs), None) == b.DS_ERR_INVALID_ARG


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError, match="no CPU path"):
        b.DoubleSqueeze(2, 100, 0.1, Q("identity"), Q("identity"))
