"""The allocation-free offset-table entry point against the regular kernel-map build (GPU, through the C ABI).

This file sorts last on purpose: a run that stops at the first failure has then already run every other test.
The entry point exists for callers that cannot allocate device memory when they need the table (a plug-in
running inside another framework's execution step, a loop with a memory budget fixed at start-up); its hash
table lives in a fixed array inside the library, which all calls on a GPU share and which keeps the previous
call's contents.  Two calls in a row with different inputs therefore check that nothing stale leaks through.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def _reference_table(coords_np, kernel, dilation):
    coords = torch.from_numpy(coords_np).cuda()
    km = binding.spconv_build_kmap(coords, 1, dilation, kernel, True)
    table = km.nbr.clone()
    km.close()
    return coords, table


def _noalloc_table(coords, kernel, dilation):
    out = torch.full((kernel ** 3, coords.shape[0]), -7, dtype=torch.int32, device="cuda")   # caller-owned output
    binding.spconv_subm_offset_table_noalloc(coords, kernel, dilation, out)
    torch.cuda.synchronize()
    return out


def test_two_calls_in_a_row_match_the_regular_entry_point():
    big = wl.shuffle_rows(wl.lidar_sweep(1), seed=1)                          # ~78k voxels: most of the fixed table
    assert len(big) <= binding.NOALLOC_MAX_VOXELS
    small = wl.shuffle_rows(wl.random_blob(3000, 20, seed=5, batches=2), seed=2)
    for coords_np, kernel, dilation in ((big, 3, 1), (small, 3, 2), (small, 5, 1), (big, 3, 1)):
        coords, want = _reference_table(coords_np, kernel, dilation)
        got = _noalloc_table(coords, kernel, dilation)
        assert torch.equal(got, want)                                          # integer table: bit-exact
        # and against the CPU oracle's offset table (submanifold rows keep the input numbering on both sides)
        ref = oracle.build_kmap(coords_np, kernel, 1, dilation, True)["oft"]
        assert np.array_equal(got.cpu().numpy().T, ref)


def test_second_call_takes_no_device_memory():
    """Neither the caching allocator of the tensor library nor the driver's free-memory figure moves across a
    call made with caller-owned tensors (the first call on a device may load the library's module; later ones
    may not take anything)."""
    coords_np = wl.shuffle_rows(wl.random_blob(4000, 22, seed=3), seed=4)
    coords = torch.from_numpy(coords_np).cuda()
    out = torch.empty(27, len(coords_np), dtype=torch.int32, device="cuda")
    binding.spconv_subm_offset_table_noalloc(coords, 3, 1, out)
    torch.cuda.synchronize()
    reserved, allocated = torch.cuda.memory_reserved(), torch.cuda.memory_allocated()
    free_before, _ = torch.cuda.mem_get_info()
    binding.spconv_subm_offset_table_noalloc(coords, 3, 1, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_reserved() == reserved and torch.cuda.memory_allocated() == allocated
    assert free_after == free_before
    assert np.array_equal(out.cpu().numpy().T, oracle.build_kmap(coords_np, 3, 1, 1, True)["oft"])


def test_limits_and_input_errors_are_reported():
    E = binding.SpconvError
    too_many = torch.zeros(binding.NOALLOC_MAX_VOXELS + 1, 4, dtype=torch.int32, device="cuda")
    out = torch.empty(27, too_many.shape[0], dtype=torch.int32, device="cuda")
    with pytest.raises(E) as e:
        binding.spconv_subm_offset_table_noalloc(too_many, 3, 1, out)
    assert e.value.status == 9 and "maximum" in str(e.value)
    dup = torch.tensor([[0, 1, 1, 1], [0, 2, 2, 2], [0, 1, 1, 1]], dtype=torch.int32, device="cuda")
    with pytest.raises(E) as e:
        binding.spconv_subm_offset_table_noalloc(dup, 3, 1, torch.empty(27, 3, dtype=torch.int32, device="cuda"))
    assert e.value.status == 3
    with pytest.raises(E) as e:                                                # even kernel: not a submanifold layer
        binding.spconv_subm_offset_table_noalloc(dup[:2].contiguous(), 2, 1, torch.empty(8, 2, dtype=torch.int32, device="cuda"))
    assert e.value.status == 1
    # after the errors the shared table still serves a correct call
    coords_np = wl.random_blob(500, 10, seed=9)
    coords, want = _reference_table(coords_np, 3, 1)
    assert torch.equal(_noalloc_table(coords, 3, 1), want)
    empty = torch.zeros(0, 4, dtype=torch.int32, device="cuda")
    binding.spconv_subm_offset_table_noalloc(empty, 3, 1, torch.empty(27, 0, dtype=torch.int32, device="cuda"))
