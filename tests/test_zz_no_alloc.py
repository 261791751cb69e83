"""The allocation-free entry point (collected last: if it fails under -x every other test has run).

ds_topk_worker_static serves callers that may not allocate device memory at the point of use --
code inside a stream capture, or a plug-in whose host framework owns the memory pool -- by keeping
the selection scratch in an array that is part of the library.  It must give exactly what the
regular worker pass gives for the same vector, also when called twice in a row (the array keeps
the previous call's contents)."""
import numpy as np
import pytest
import torch

from paper_1905_05957_b200 import DoubleSqueeze, Q, binding

pytestmark = pytest.mark.gpu


def _regular(g, delta0, k):
    d = g.numel()
    ds = DoubleSqueeze(1, d, 0.1, Q("topk", k=k), Q("identity"), seed=0)
    ds.delta_w.copy_(delta0.view(1, d))
    ds.worker_compress(g.view(1, d).contiguous(), 0)
    torch.cuda.synchronize()
    v = ds.worker_views()[0]
    out = v["idx"].clone(), v["val"].clone(), ds.delta_w.view(-1).clone()
    assert ds.device_status() == 0
    ds.close()
    return out


def _check_against_regular(g, delta, k):
    d = g.numel()
    idx = torch.full((max(k, 1),), -1, dtype=torch.int32, device="cuda")
    val = torch.full((max(k, 1),), -1.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    want_idx, want_val, want_delta = _regular(g, delta, k)
    # with nothing to keep the two output arrays may be absent
    binding.topk_worker_static(g, delta, k, idx if k else None, val if k else None, status)
    torch.cuda.synchronize()
    assert torch.equal(idx[:k], want_idx)
    assert torch.equal(val[:k].view(torch.int32), want_val.view(torch.int32))
    assert torch.equal(delta.view(torch.int32), want_delta.view(torch.int32))
    assert int(status.item()) == 0


@pytest.mark.parametrize("d,k", [(100_000, 1000), (8192 * 3 + 5, 77), (1 << 20, 10_485)])
def test_static_scratch_entry_matches_the_regular_one_twice_in_a_row(d, k):
    gen = torch.Generator(device="cuda").manual_seed(d)
    delta = torch.zeros(d, device="cuda")
    for call in range(2):                      # the second call meets the first call's leftovers
        g = torch.randn(d, device="cuda", generator=gen)
        if call == 1:
            g[::3] = torch.round(g[::3] * 2) / 2   # plenty of equal magnitudes: the tie rule is exercised
        _check_against_regular(g, delta, k)


@pytest.mark.parametrize("d,k", [(1, 1), (1, 0), (33, 7), (300, 0), (4095, 4095), (8192, 8192), (70_000, 1), (70_000, 69_999)])
def test_static_scratch_entry_small_and_extreme_k(d, k):
    gen = torch.Generator(device="cuda").manual_seed(7 * d + k)
    delta = torch.randn(d, device="cuda", generator=gen) * 0.3
    for call in range(2):
        _check_against_regular(torch.randn(d, device="cuda", generator=gen), delta, k)


def test_static_scratch_entry_ties_across_segments():
    """All-equal and integer-valued vectors longer than two 32768-entry segments: the tie quota is
    split over segments and the lowest indices win."""
    d = 3 * 32768 + 1000
    for k in (1, 40_000, d - 1):
        delta = torch.zeros(d, device="cuda")
        _check_against_regular(torch.full((d,), -2.5, device="cuda"), delta, k)
        gen = torch.Generator(device="cuda").manual_seed(k)
        g = torch.randint(-3, 4, (d,), device="cuda", generator=gen).float()
        _check_against_regular(g, delta, k)


def test_static_scratch_entry_rows_only_four_byte_aligned():
    """g and delta that start 4 bytes past a 16-byte boundary (d % 4 == 0): the scalar-load path."""
    d, k = 40_000, 400
    gen = torch.Generator(device="cuda").manual_seed(11)
    g_store = torch.randn(d + 1, device="cuda", generator=gen)
    delta_store = torch.randn(d + 1, device="cuda", generator=gen) * 0.1
    g, delta = g_store[1:], delta_store[1:]
    assert g.data_ptr() % 16 == 4 and delta.data_ptr() % 16 == 4
    for call in range(2):
        _check_against_regular(g, delta, k)
        g_store.normal_(generator=gen)


def test_static_scratch_entry_at_its_size_limit():
    """d = DS_STATIC_TOPK_MAX_D: the selection needs nearly all of the built-in scratch."""
    d = binding.DS_STATIC_TOPK_MAX_D
    gen = torch.Generator(device="cuda").manual_seed(23)
    delta = torch.randn(d, device="cuda", generator=gen) * 0.2
    for call, k in enumerate((d // 100, 12_345)):
        _check_against_regular(torch.randn(d, device="cuda", generator=gen), delta, k)


def test_static_scratch_entry_rejects_oversize_and_bad_arguments():
    lib = binding.load_library()
    d = binding.DS_STATIC_TOPK_MAX_D + 4
    small = torch.zeros(16, device="cuda")
    i32 = torch.zeros(16, dtype=torch.int32, device="cuda")
    # too large for the built-in scratch: refused before anything is launched (buffers are not touched)
    rc = lib.ds_topk_worker_static(small.data_ptr(), small.data_ptr(), d, 1, i32.data_ptr(), small.data_ptr(),
                                   i32.data_ptr(), None)
    assert rc == binding.DS_ERR_UNSUPPORTED
    rc = lib.ds_topk_worker_static(small.data_ptr(), small.data_ptr(), 16, 17, i32.data_ptr(), small.data_ptr(),
                                   i32.data_ptr(), None)
    assert rc == binding.DS_ERR_INVALID_ARG
    rc = lib.ds_topk_worker_static(None, small.data_ptr(), 16, 1, i32.data_ptr(), small.data_ptr(), i32.data_ptr(), None)
    assert rc == binding.DS_ERR_INVALID_ARG
    torch.cuda.synchronize()
