"""Two host threads use the library at the same time, each on its own stream: builds, forwards and whole-layer calls.

The library keeps per-thread side streams and tensor-map caches, a mutex-guarded pool of pinned report buffers and
per-device capacities computed once; every result must be bit-identical to the one the same call gives alone
(the kernel map's numbering and the forward's accumulation order do not depend on timing).
"""
import threading

import numpy as np
import pytest
import torch

from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import kmap_to_numpy, to_device

pytestmark = pytest.mark.gpu


def _job(coords, x, w, rounds, results, errors, slot):
    try:
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            t = torch.from_numpy(coords).cuda()
            outs = []
            for i in range(rounds):
                if i % 2 == 0:
                    km = binding.spconv_build_kmap(t, 1, 1, 3, True)
                    y = binding.spconv_forward(x, w, km)
                else:
                    km = binding.spconv_build_kmap(t, 2, 1, 3, False)
                    y = None
                stream.synchronize()
                assert binding.spconv_last_device_status(km) == 0
                d = kmap_to_numpy(km)
                outs.append((d["oft"].copy(), d["offset_start"].copy(), d["out_coords"].copy(), None if y is None else y.clone()))
                km.close()
            results[slot] = outs
    except BaseException as e:   # noqa: BLE001 - reported by the main thread
        errors[slot] = e


def test_two_threads_two_streams_give_the_single_thread_results():
    sweeps = [wl.lidar_sweep(0)[:30000].copy(), wl.shuffle_rows(wl.random_blob(20000, 40, seed=5, batches=2), seed=2)]
    xs = [to_device(wl.features(len(c), 32, "bf16", i), "bf16") for i, c in enumerate(sweeps)]
    w = to_device(wl.weights(27, 32, 64, "bf16", 0), "bf16")
    rounds = 6
    alone, errors = [None, None], [None, None]
    for s in range(2):
        _job(sweeps[s], xs[s], w, 2, alone, errors, s)
        assert errors[s] is None, errors[s]
    together, errors = [None, None], [None, None]
    threads = [threading.Thread(target=_job, args=(sweeps[s], xs[s], w, rounds, together, errors, s)) for s in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=120)
        assert not th.is_alive()
    for s in range(2):
        assert errors[s] is None, errors[s]
        for i, (oft, os_, oc, y) in enumerate(together[s]):
            ref = alone[s][i % 2]
            assert np.array_equal(oft, ref[0]) and np.array_equal(os_, ref[1]) and np.array_equal(oc, ref[2])
            if y is not None:
                assert torch.equal(y, ref[3])
