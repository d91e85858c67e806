"""Row-order and offsets-per-step options of the tensor-core forward: the same kernel map and the same rows.

The order of the row tiles and the number of offsets a pipeline step takes change padding and speed only
(grouping of pairs into matrix products, Sec. II-C); the map must stay bit-identical and the output rows must
match the oracle's within the feature tolerance for every combination.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import TOL, kmap_to_numpy, rel_err, to_device

pytestmark = pytest.mark.gpu


def _maps(coords, K, s, subm):
    t = torch.from_numpy(coords).cuda()
    a = binding.spconv_build_kmap(t, s, 1, K, subm)
    b = binding.spconv_build_kmap(t, s, 1, K, subm, row_order=binding.ROWS_AS_GIVEN)
    c = binding.spconv_build_kmap(t, s, 1, K, subm, row_order=binding.ROWS_BY_OFFSET_SET)
    return a, b, c


@pytest.mark.parametrize("K,s,subm", [(3, 1, True), (3, 2, False), (2, 2, False)])
def test_row_orders_give_the_same_map_and_rows(K, s, subm):
    coords = wl.shuffle_rows(wl.random_blob(5000, 26, seed=K + s, batches=2), seed=1)
    a, b, c = _maps(coords, K, s, subm)
    da, db, dc = kmap_to_numpy(a), kmap_to_numpy(b), kmap_to_numpy(c)
    for key in ("out_coords", "oft", "offset_start", "pair_in", "pair_out"):
        if key in ("pair_in", "pair_out") and not subm:
            continue                                    # strided pair order within an offset is not unique
        assert np.array_equal(da[key], db[key]), key
        assert np.array_equal(da[key], dc[key]), key
    tr = b.tile_rows.cpu().numpy().reshape(-1)
    assert np.array_equal(tr[:b.n_out], np.arange(b.n_out)) and (tr[b.n_out:] == -1).all()
    assert b.tile_blocks >= a.tile_blocks == c.tile_blocks
    x, w = wl.features(len(coords), 32, "bf16", 0), wl.weights(K ** 3, 32, 64, "bf16", 0)
    want = oracle.forward(x, w, da["oft"])
    xd, wd = to_device(x, "bf16"), to_device(w, "bf16")
    outs = []
    for km in (a, b):
        for algo in ("tcgen05", "tcgen05_single"):
            y = binding.spconv_forward(xd, wd, km, algo=algo)
            torch.cuda.synchronize()
            assert binding.spconv_last_device_status(km) == 0
            assert rel_err(y, want) <= TOL["bf16"], (algo, km is a)
            outs.append(y)
    # the accumulation order over offsets is the same for every variant: identical bits
    for y in outs[1:]:
        assert torch.equal(outs[0], y)


def test_row_order_argument_is_checked():
    t = torch.from_numpy(wl.random_blob(100, 8, seed=0)).cuda()
    with pytest.raises(binding.SpconvError) as e:
        binding.spconv_build_kmap(t, 1, 1, 3, True, row_order=7)
    assert e.value.status == 1


def test_single_offset_algo_rejects_unsupported_shapes():
    t = torch.from_numpy(wl.random_blob(100, 8, seed=0)).cuda()
    km = binding.spconv_build_kmap(t, 1, 1, 3, True)
    x = torch.zeros(km.n_in, 24, device="cuda", dtype=torch.bfloat16)
    w = torch.zeros(27, 24, 16, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(binding.SpconvError):
        binding.spconv_forward(x, w, km, algo="tcgen05_single")
