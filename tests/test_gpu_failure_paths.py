"""Failure paths that only a test hook can reach, in the accepted form: a bound runs out, the kernel gives up by
itself and reports through a status word that the host reads; nothing faults, traps or waits without a limit, and
the next ordinary call on the same context (and the same handle) succeeds."""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import TOL, rel_err

pytestmark = pytest.mark.gpu


def test_location_table_full_is_reported_and_the_next_build_succeeds():
    """A location table forced to 1024 slots cannot take 3000 rows: the bounded probe sequence runs out and the
    build returns SPCONV_ERR_TABLE_FULL (4) for submanifold, strided and inverse maps; with the hook off the same
    input builds and matches the oracle."""
    coords_np = wl.shuffle_rows(wl.random_blob(3000, 20, 1), seed=2)
    coords = torch.from_numpy(coords_np).cuda()
    binding.spconv_test_hook(binding.HOOK_TABLE_SLOTS, 1024)
    try:
        for stride, subm in ((1, True), (2, False)):
            with pytest.raises(binding.SpconvError) as e:
                binding.spconv_build_kmap(coords, stride, 1, 3, subm)
            assert e.value.status == 4
        with pytest.raises(binding.SpconvError) as e:
            binding.spconv_build_inverse_kmap(coords[:10].contiguous(), coords, 2, 1, 3)
        assert e.value.status == 4
        small = wl.random_blob(500, 10, 3)                                 # fits the forced table
        km = binding.spconv_build_kmap(torch.from_numpy(small).cuda(), 1, 1, 3, True)
        assert np.array_equal(km.nbr.cpu().numpy().T, oracle.build_kmap(small, 3, 1, 1, True)["oft"])
    finally:
        binding.spconv_test_hook(binding.HOOK_TABLE_SLOTS, 0)
    km = binding.spconv_build_kmap(coords, 1, 1, 3, True)
    ref = oracle.build_kmap(coords_np, 3, 1, 1, True)
    assert np.array_equal(km.nbr.cpu().numpy().T, ref["oft"]) and km.total_pairs == len(ref["pair_in"])


@pytest.mark.parametrize("cin,cout", [(64, 64), (128, 128), (16, 32), (64, 128)])
def test_pipeline_wait_runs_out_is_reported_and_the_next_forward_is_exact(cin, cout):
    """With the waits' time limit shortened to 300 us and the weights of CTA 0's first step withheld, the wait for
    that step gives up: the launch returns by itself, spconv_last_device_status reports SPCONV_ERR_PIPE_TIMEOUT (7)
    once, and status words 1-2 name the wait and the CTA.  With the hook off, the next forward on the same handle
    gives the oracle's rows and the same bits as a forward made before the fault.  The shapes cover the ways the
    weights travel (inside the stage with one and with several offsets per step, in slots of their own)."""
    coords = wl.shuffle_rows(wl.random_blob(4000, 22, 5), seed=1)
    km = binding.spconv_build_kmap(torch.from_numpy(coords).cuda(), 1, 1, 3, True)
    x_np, w_np = wl.features(len(coords), cin, "bf16", 0), wl.weights(27, cin, cout, "bf16", 0)
    x = torch.from_numpy(x_np).to(torch.bfloat16).cuda()
    w = torch.from_numpy(w_np).to(torch.bfloat16).cuda()
    before = binding.spconv_forward(x, w, km, algo="tcgen05")
    torch.cuda.synchronize()
    assert binding.spconv_last_device_status(km) == 0
    binding.spconv_test_hook(binding.HOOK_PIPE_WAIT_LIMIT_US, 300)
    try:
        binding.spconv_forward(x, w, km, algo="tcgen05")
        torch.cuda.synchronize()                                           # the launch ends by itself
        words = binding.spconv_kmap_status_words(km)
        assert words[0] & 8, words                                         # the time-out bit
        assert words[1] & 0x80000000 and words[2] == 1, [hex(v) for v in words[:3]]   # a wait is named; CTA 0 (stored + 1)
        assert binding.spconv_last_device_status(km) == 7
        assert binding.spconv_last_device_status(km) == 0                  # reported once, then cleared
    finally:
        binding.spconv_test_hook(binding.HOOK_PIPE_WAIT_LIMIT_US, 0)
    after = binding.spconv_forward(x, w, km, algo="tcgen05")
    torch.cuda.synchronize()
    assert binding.spconv_last_device_status(km) == 0
    assert torch.equal(after, before)
    ref = oracle.forward(x_np, w_np, np.ascontiguousarray(km.nbr.cpu().numpy().T))
    assert rel_err(after, ref) <= TOL["bf16"]


def test_unknown_hook_is_refused():
    with pytest.raises(binding.SpconvError) as e:
        binding.spconv_test_hook(99, 1)
    assert e.value.status == 1
