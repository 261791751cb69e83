"""ctypes binding of the C ABI in include/dsq.h.  Argument marshalling only.

PyTorch appears here for device memory and streams; every step of the path runs in the
library's kernels.  There is no CPU fallback: a missing library or device raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from .workloads import Q, Workload

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libdsq.so")

DS_OK, DS_NEED_BUFFERS = 0, 1
DS_ERR_INVALID_ARG, DS_ERR_ALIGN, DS_ERR_BUFFER_TOO_SMALL = -1, -2, -3
DS_ERR_STATE, DS_ERR_CUDA, DS_ERR_UNSUPPORTED = -4, -5, -6
DS_FUSE_APPLY = 1
DS_DEV_TOPK_INCONSISTENT = 1
OPS = {"identity": 0, "sign1": 1, "topk": 2, "qsgd": 3, "clip": 4, "rsparse": 5, "ternary": 6}
DS_NO_COMPENSATION = 1
EXPORTS = ("ds_get_layout", "ds_create", "ds_worker_compress", "ds_server_aggregate_compress",
           "ds_apply_update", "ds_destroy", "ds_step_host", "ds_last_error", "ds_version",
           "ds_kernel_launches", "ds_topk_worker_static", "ds_worker_compress_rows",
           "ds_server_aggregate_compress_slice", "ds_apply_update_slice", "ds_server_topk_slice_begin",
           "ds_server_topk_slice_digit", "ds_server_topk_slice_emit", "ds_apply_update_sparse_range")
DS_SLICE_ALIGN = 8192


class ds_qspec(C.Structure):
    _fields_ = [("op", C.c_int32), ("chunk", C.c_uint32), ("k", C.c_uint64), ("levels", C.c_uint32),
                ("norm", C.c_uint32)]


class ds_config(C.Structure):
    _fields_ = [("n", C.c_uint32), ("delta_w_rows", C.c_uint32), ("d", C.c_uint64), ("gamma", C.c_float),
                ("flags", C.c_uint32), ("worker_q", ds_qspec), ("server_q", ds_qspec), ("seed", C.c_uint64)]


class ds_buffers(C.Structure):
    _fields_ = [("x", C.c_void_p), ("delta_w", C.c_void_p), ("delta_s", C.c_void_p),
                ("worker_payload", C.c_void_p), ("server_payload", C.c_void_p), ("workspace", C.c_void_p),
                ("dev_status", C.c_void_p),
                ("x_bytes", C.c_size_t), ("delta_w_bytes", C.c_size_t), ("delta_s_bytes", C.c_size_t),
                ("worker_payload_bytes", C.c_size_t), ("server_payload_bytes", C.c_size_t),
                ("workspace_bytes", C.c_size_t)]


class ds_payload_layout(C.Structure):
    _fields_ = [("stride", C.c_uint64), ("off", C.c_uint64 * 3), ("count", C.c_uint64 * 3)]


class DsqError(RuntimeError):
    def __init__(self, code: int, what: str, detail: str = ""):
        super().__init__(f"{what} failed with ds_status {code}" + (f": {detail}" if detail else ""))
        self.code = code


_lib = None


def load_library() -> C.CDLL:
    """Loads csrc/libdsq.so (built by build.py).  Raises if it is absent: there is no other path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_1905_05957_b200.build` "
                           "(or __graft_entry__.build()); this package has no fallback implementation")
    L = C.CDLL(LIB_PATH)
    vp, u32 = C.c_void_p, C.c_uint32
    L.ds_get_layout.argtypes = [C.POINTER(ds_config), C.c_int, C.POINTER(ds_payload_layout)]
    L.ds_create.argtypes = [C.POINTER(ds_config), C.POINTER(ds_buffers), C.POINTER(vp)]
    L.ds_worker_compress.argtypes = [vp, vp, u32, vp]
    L.ds_server_aggregate_compress.argtypes = [vp, u32, u32, vp]
    L.ds_apply_update.argtypes = [vp, vp]
    L.ds_destroy.argtypes = [vp]
    L.ds_step_host.argtypes = [vp, vp, vp, u32, vp, vp, vp]
    L.ds_topk_worker_static.argtypes = [vp, vp, C.c_uint64, C.c_uint64, vp, vp, vp, vp]
    L.ds_worker_compress_rows.argtypes = [vp, vp, u32, u32, u32, vp]
    L.ds_server_aggregate_compress_slice.argtypes = [vp, u32, u32, C.c_uint64, C.c_uint64, vp]
    L.ds_apply_update_slice.argtypes = [vp, C.c_uint64, C.c_uint64, vp]
    L.ds_server_topk_slice_begin.argtypes = [vp, u32, C.c_uint64, C.c_uint64, vp, vp]
    L.ds_server_topk_slice_digit.argtypes = [vp, C.c_int, C.c_uint64, C.c_uint64, vp, vp, vp]
    L.ds_server_topk_slice_emit.argtypes = [vp, C.c_uint64, C.c_uint64, u32, u32, C.c_uint64, u32, vp]
    L.ds_apply_update_sparse_range.argtypes = [vp, C.c_uint64, C.c_uint64, vp]
    for name in EXPORTS:
        getattr(L, name).restype = C.c_int
    L.ds_last_error.restype = C.c_char_p
    L.ds_kernel_launches.restype = C.c_uint64
    _lib = L
    return L


def _qspec(q: Q) -> ds_qspec:
    levels = {"clip": q.bits, "rsparse": q.keep_one_in}.get(q.op, q.levels)
    norm = {"sign1": q.norm, "rsparse": q.scaled}.get(q.op, 0)
    return ds_qspec(OPS[q.op], q.chunk, q.k, levels, norm)


def make_config(n: int, d: int, gamma: float, worker_q: Q, server_q: Q, seed: int, compensate: bool = True,
                delta_w_rows: int = 0) -> ds_config:
    return ds_config(n, delta_w_rows, d, gamma, 0 if compensate else DS_NO_COMPENSATION, _qspec(worker_q), _qspec(server_q), seed)


def get_layout(cfg: ds_config, which: int) -> ds_payload_layout:
    out = ds_payload_layout()
    rc = load_library().ds_get_layout(C.byref(cfg), which, C.byref(out))
    if rc != DS_OK:
        raise DsqError(rc, "ds_get_layout")
    return out


_VIEW_DTYPES = {
    "identity": (("c", torch.float32),),
    "sign1": (("bits", torch.int32), ("scale", torch.float32)),
    "topk": (("idx", torch.int32), ("val", torch.float32)),
    "qsgd": (("lvl", torch.uint8), ("sgn", torch.int32), ("step", torch.float32)),
    "rsparse": (("val", torch.float32), ("off", torch.int32)),
    "ternary": (("sgn", torch.int32), ("nz", torch.int32), ("scale", torch.float32)),
    "clip": (("hi", torch.int16),),      # 8-bit entries when 24 bits are cleared, see payload_views
}


def payload_views(buf: torch.Tensor, layout: ds_payload_layout, q: Q, rows: int) -> list[dict]:
    """Typed views of the sub-arrays of each payload inside the raw byte buffer (no copies).
    uint32 / uint16 fields are exposed as int32 / int16 tensors with the same bits."""
    out = []
    fields = _VIEW_DTYPES[q.op]
    if q.op == "clip" and q.bits == 24:
        fields = (("hi", torch.uint8),)
    for i in range(rows):
        base = i * layout.stride
        views = {}
        for j, (name, dt) in enumerate(fields):
            nbytes = layout.count[j] * torch.empty(0, dtype=dt).element_size()
            views[name] = buf[base + layout.off[j]: base + layout.off[j] + nbytes].view(dt)
        out.append(views)
    return out


DS_STATIC_TOPK_MAX_D = 1 << 23


def topk_worker_static(g: torch.Tensor, delta: torch.Tensor, k: int, idx: torch.Tensor | None, val: torch.Tensor | None,
                       dev_status: torch.Tensor, stream=None) -> None:
    """ds_topk_worker_static: top-k with error feedback for one vector, using the library's built-in
    scratch array, for callers that cannot allocate device memory where they compress (inside a
    stream capture, or as a guest of a framework that owns the memory pool).  All tensors are the
    caller's; delta is updated in place.  Calls on different streams must not overlap."""
    s = stream if stream is not None else torch.cuda.current_stream(g.device)
    rc = load_library().ds_topk_worker_static(g.data_ptr(), delta.data_ptr(), g.numel(), k,
                                              None if idx is None else idx.data_ptr(),
                                              None if val is None else val.data_ptr(), dev_status.data_ptr(), s.cuda_stream)
    if rc != DS_OK:
        raise DsqError(rc, "ds_topk_worker_static")


class DoubleSqueeze:
    """One DoubleSqueeze state (x, delta_w, delta_s) on one GPU, stepped through the C ABI."""

    GUARD_BYTES = 256          # sentinel bytes on each side of a buffer when guard=True
    GUARD_PATTERN = 0xA5

    def __init__(self, n: int, d: int, gamma: float, worker_q: Q, server_q: Q, seed: int = 0,
                 device: str | torch.device = "cuda", x0: torch.Tensor | None = None, guard: bool = False,
                 payload_fill: int = 0, compensate: bool = True, delta_w_rows: int = 0):
        """delta_w_rows = R < n: this instance is one rank of a deployment with R workers per GPU and keeps
        only their errors (see ds_config.delta_w_rows).
        compensate=False: the methods of Section 5.1 that keep no error (DS_NO_COMPENSATION): delta_w
        and delta_s are then empty tensors unless the library asks for delta_s as scratch.
        guard=True surrounds every buffer handed to the library with GUARD_BYTES sentinel bytes
        (check_guards() tells whether any was overwritten): a debugging aid for out-of-bounds writes.
        payload_fill: byte the payload buffers start out with (the library must overwrite every byte
        it defines whatever they held)."""
        if not torch.cuda.is_available():
            raise RuntimeError("paper_1905_05957_b200 needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.device = torch.device(device)
        self.n, self.d, self.gamma, self.seed = n, d, gamma, seed
        self.worker_q, self.server_q = worker_q, server_q
        self.compensate = compensate
        self.cfg = make_config(n, d, gamma, worker_q, server_q, seed, compensate, delta_w_rows)
        bufs = ds_buffers()
        rc = self.lib.ds_create(C.byref(self.cfg), C.byref(bufs), None)
        if rc != DS_NEED_BUFFERS:
            raise DsqError(rc, "ds_create (size query)")
        dev = self.device
        self._guarded = []

        def alloc(nbytes: int, fill: int = 0) -> torch.Tensor:
            """nbytes of device memory as a byte tensor (16-byte aligned), optionally between guards."""
            if not guard:
                return torch.full((nbytes,), fill, dtype=torch.uint8, device=dev) if fill else \
                    torch.zeros(nbytes, dtype=torch.uint8, device=dev)
            G = self.GUARD_BYTES
            raw = torch.full((nbytes + 2 * G,), self.GUARD_PATTERN, dtype=torch.uint8, device=dev)
            raw[G:G + nbytes] = fill
            self._guarded.append((raw, nbytes))
            return raw[G:G + nbytes]

        self.x = alloc(d * 4).view(torch.float32)
        if x0 is not None:
            self.x.copy_(x0.to(device=dev, dtype=torch.float32).reshape(-1))
        self.delta_w = alloc(bufs.delta_w_bytes).view(torch.float32).view(-1, d) if bufs.delta_w_bytes else alloc(0).view(torch.float32).view(n, 0)
        self.delta_s = alloc(bufs.delta_s_bytes).view(torch.float32)
        self.worker_payload = alloc(bufs.worker_payload_bytes, payload_fill)
        self.server_payload = alloc(bufs.server_payload_bytes, payload_fill)
        self.workspace = alloc(max(bufs.workspace_bytes, 16))
        self.dev_status = alloc(16).view(torch.int32)
        bufs.x = self.x.data_ptr()
        bufs.delta_w = self.delta_w.data_ptr() if bufs.delta_w_bytes else None
        bufs.delta_s = self.delta_s.data_ptr() if bufs.delta_s_bytes else None
        bufs.worker_payload, bufs.server_payload = self.worker_payload.data_ptr(), self.server_payload.data_ptr()
        bufs.workspace, bufs.dev_status = self.workspace.data_ptr(), self.dev_status.data_ptr()
        self.bufs = bufs
        self.workspace_bytes = bufs.workspace_bytes
        h = C.c_void_p()
        rc = self.lib.ds_create(C.byref(self.cfg), C.byref(bufs), C.byref(h))
        if rc != DS_OK:
            raise DsqError(rc, "ds_create")
        self.handle = h
        self.worker_layout = get_layout(self.cfg, 0)
        self.server_layout = get_layout(self.cfg, 1)

    def check_guards(self) -> bool:
        """True if no sentinel byte around any buffer has changed (always True without guard=True)."""
        G = self.GUARD_BYTES
        for raw, nbytes in self._guarded:
            if not bool((raw[:G] == self.GUARD_PATTERN).all()) or not bool((raw[G + nbytes:] == self.GUARD_PATTERN).all()):
                return False
        return True

    @classmethod
    def for_workload(cls, wl: Workload, device="cuda") -> "DoubleSqueeze":
        return cls(wl.n, wl.d, wl.gamma, wl.worker_q, wl.server_q, wl.seed, device, compensate=wl.compensate)

    # -- the three calls of one iteration -----------------------------------------------------
    def _stream(self, stream) -> int:
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        return s.cuda_stream

    def _check(self, rc: int, what: str):
        if rc != DS_OK:
            raise DsqError(rc, what, self.lib.ds_last_error().decode())

    def worker_compress(self, g: torch.Tensor, step: int, stream=None):
        assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous() and g.numel() == self.n * self.d
        self._check(self.lib.ds_worker_compress(self.handle, g.data_ptr(), step, self._stream(stream)),
                    "ds_worker_compress")

    def server_aggregate_compress(self, step: int, fuse_apply: bool = False, stream=None):
        self._check(self.lib.ds_server_aggregate_compress(self.handle, step, DS_FUSE_APPLY if fuse_apply else 0,
                                                          self._stream(stream)), "ds_server_aggregate_compress")

    def apply_update(self, stream=None):
        self._check(self.lib.ds_apply_update(self.handle, self._stream(stream)), "ds_apply_update")

    # -- the same passes over some of the workers / a slice of d (one GPU per worker deployments) ---
    def worker_compress_rows(self, g_rows: torch.Tensor, row0: int, step: int, stream=None):
        assert g_rows.is_cuda and g_rows.dtype == torch.float32 and g_rows.is_contiguous() and g_rows.numel() % self.d == 0
        self._check(self.lib.ds_worker_compress_rows(self.handle, g_rows.data_ptr(), row0, g_rows.numel() // self.d, step,
                                                     self._stream(stream)), "ds_worker_compress_rows")

    def server_aggregate_compress_slice(self, step: int, lo: int, hi: int, fuse_apply: bool = False, stream=None):
        self._check(self.lib.ds_server_aggregate_compress_slice(self.handle, step, DS_FUSE_APPLY if fuse_apply else 0, lo, hi,
                                                                self._stream(stream)), "ds_server_aggregate_compress_slice")

    def apply_update_slice(self, lo: int, hi: int, stream=None):
        self._check(self.lib.ds_apply_update_slice(self.handle, lo, hi, self._stream(stream)), "ds_apply_update_slice")

    # -- global top-k on the server pass over a slice (the stages between which histograms are summed across GPUs) ---
    def server_topk_slice_begin(self, step: int, lo: int, hi: int, hist: torch.Tensor, stream=None):
        self._check(self.lib.ds_server_topk_slice_begin(self.handle, step, lo, hi, hist.data_ptr(), self._stream(stream)),
                    "ds_server_topk_slice_begin")

    def server_topk_slice_digit(self, level: int, lo: int, hi: int, hist_sum: torch.Tensor, hist_next: torch.Tensor, stream=None):
        self._check(self.lib.ds_server_topk_slice_digit(self.handle, level, lo, hi, hist_sum.data_ptr(), hist_next.data_ptr(),
                                                        self._stream(stream)), "ds_server_topk_slice_digit")

    def server_topk_slice_emit(self, lo: int, hi: int, ties_to_keep: int, count: int, first_slot: int, fuse_apply: bool = True,
                               stream=None):
        self._check(self.lib.ds_server_topk_slice_emit(self.handle, lo, hi, ties_to_keep, count, first_slot,
                                                       DS_FUSE_APPLY if fuse_apply else 0, self._stream(stream)),
                    "ds_server_topk_slice_emit")

    def apply_update_sparse_range(self, first_slot: int, count: int, stream=None):
        self._check(self.lib.ds_apply_update_sparse_range(self.handle, first_slot, count, self._stream(stream)),
                    "ds_apply_update_sparse_range")

    def step(self, g: torch.Tensor, t: int, fuse_apply: bool = True, stream=None):
        self.worker_compress(g, t, stream)
        self.server_aggregate_compress(t, fuse_apply, stream)
        if not fuse_apply:
            self.apply_update(stream)

    def step_host(self, g_host: torch.Tensor, g_dev: torch.Tensor, t: int, server_payload_host=None, x_host=None,
                  stream=None):
        """Host-buffer form: H2D of g, the fused step, D2H of the server payload and/or x; asynchronous."""
        assert not g_host.is_cuda and g_host.is_contiguous() and g_dev.is_cuda
        sp = server_payload_host.data_ptr() if server_payload_host is not None else None
        xp = x_host.data_ptr() if x_host is not None else None
        self._check(self.lib.ds_step_host(self.handle, g_host.data_ptr(), g_dev.data_ptr(), t, sp, xp,
                                          self._stream(stream)), "ds_step_host")

    # -- views ----------------------------------------------------------------------------------
    def worker_views(self) -> list[dict]:
        return payload_views(self.worker_payload, self.worker_layout, self.worker_q, self.n)

    def server_views(self) -> dict:
        return payload_views(self.server_payload, self.server_layout, self.server_q, 1)[0]

    def device_status(self) -> int:
        """Word 0 of dev_status: the DS_DEV_* flags."""
        return int(self.dev_status[0].item())

    def topk_routes(self) -> tuple[int, int]:
        """(predicted, full): how many top-k selections so far ran with the threshold band predicted
        from earlier steps, and how many went through the full histogram (dev_status words 1, 2)."""
        w = self.dev_status.cpu()
        return int(w[1]), int(w[2])

    def close(self):
        if getattr(self, "handle", None):
            self.lib.ds_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
