"""civic_select_large_static: the selection for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them: a serving engine
that gave all device memory to its own pool when it started, a plugin without an allocator, a
step with a hard memory cap.  For them the library carries a fixed 2 MiB scratch array and this
entry point, which takes inputs and the output only.  The test calls it through the C ABI twice
in a row on different inputs (the second call finds the first call's leftovers in the shared
scratch and must still be right) and compares with civic_select_large, which is given a
workspace, and with the CPU oracle; the results are index arrays, so the comparisons are exact.
It also checks what the entry point is for: around the two calls the device's free memory and
torch's allocator statistics do not move, and each call is the five launches that go through the
scratch (a shape that fitted the one-launch cluster path would not touch it).

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.  It passes on its own in a fresh process as well.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_28115_b200 import build, civic

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def test_static_scratch_matches_workspace_version_on_two_calls_in_a_row():
    lib = civic.load()
    rng = np.random.default_rng(404)
    # two different problems, both larger than one thread block can hold
    cases = [(civic.SelectDesc(64, 56, 56, 4, 4, 1, 66901), 2, "quant"),
             (civic.SelectDesc(40, 60, 44, 4, 4, 2, 40000), 3, "uniform")]
    prepared, expected = [], []
    for desc, n_seg, kind in cases:
        n = desc.t * desc.h * desc.w
        u = rng.random((n_seg, n))
        scores_host = (np.floor(u * 256) / 256 if kind == "quant" else u).astype(np.float32)
        expected.append(oracle.default.select(scores_host, desc.t, desc.h, desc.w, desc.region_h, desc.region_w,
                                              desc.floor_per_region, desc.k))
        scores = torch.from_numpy(scores_host).to(DEV)
        want = torch.empty((n_seg, desc.k), dtype=torch.int32, device=DEV)
        got = torch.full((n_seg, desc.k), -1, dtype=torch.int32, device=DEV)
        ws = torch.empty(civic.select_workspace_bytes(desc, n_seg), dtype=torch.uint8, device=DEV)
        assert ws.numel() <= civic.select_static_scratch_bytes()
        civic.civic_select_large(scores, desc, keep_idx=want, workspace=ws)
        prepared.append((desc, n_seg, scores, want, got))
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    # a first call, so that loading the kernels and looking up the scratch address are behind us
    desc, n_seg, scores, _, got = prepared[0]
    assert lib.civic_select_large_static(scores.data_ptr(), n_seg, ctypes.byref(desc), got.data_ptr(), 0,
                                         stream) == civic.CIVIC_OK
    torch.cuda.synchronize()
    got.fill_(-1)
    torch.cuda.synchronize()

    # the two calls under test, back to back on one stream, straight through the C ABI
    free_before, _ = torch.cuda.mem_get_info()
    stats_before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
    launches = civic.launch_count()
    for desc, n_seg, scores, _, got in prepared:
        status = lib.civic_select_large_static(scores.data_ptr(), n_seg, ctypes.byref(desc), got.data_ptr(), 0,
                                               stream)
        assert status == civic.CIVIC_OK, civic.STATUS_NAMES[status]
        launches += 5  # the five launches that communicate through the scratch, not the cluster path
        assert civic.launch_count() == launches
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated or freed"
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == stats_before
    for (_, _, _, want, got), want_oracle in zip(prepared, expected):
        assert np.array_equal(got.cpu().numpy(), want_oracle)  # the definition
        assert torch.equal(got, want)                          # and the sibling entry point

    # and once more in the opposite order through the binding
    for desc, n_seg, scores, want, got in reversed(prepared):
        got.fill_(-1)
        civic.civic_select_large_static(scores, desc, got)
        assert torch.equal(got, want)


def test_static_scratch_rejects_what_does_not_fit():
    lib = civic.load()
    cap = civic.select_static_scratch_bytes()
    assert cap == 2 << 20
    big = civic.SelectDesc(1200, 64, 64, 8, 8, 0, 1000)  # 4.9 M tokens: one flag byte each
    assert civic.select_workspace_bytes(big, 1) > cap
    before = civic.launch_count()
    status = lib.civic_select_large_static(0x1000, 1, ctypes.byref(big), 0x2000, 0, None)
    assert civic.STATUS_NAMES[status] == "CIVIC_ERR_WORKSPACE"
    assert civic.launch_count() == before
    with pytest.raises(civic.CivicError, match="WORKSPACE"):
        civic.civic_select_large_static(torch.zeros((1, 1200 * 64 * 64), device=DEV), big,
                                        torch.empty((1, 1000), dtype=torch.int32, device=DEV))
