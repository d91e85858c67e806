"""Kernel maps built through the dense-array location table (Sec. III-C.1, the paper's alternative to the hash
table for confined domains) against the oracle and against the hash-table build: identical bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2402_07710_b200 import binding, workloads as wl
from gpu_util import TOL, canon, kmap_to_numpy, rel_err, to_device
from kmap_util import assert_kmaps_equal

pytestmark = pytest.mark.gpu


def _both(coords_np, grid, K=3, d=1):
    coords = torch.from_numpy(coords_np).cuda()
    dense = binding.spconv_build_kmap_dense(coords, grid, d, K)
    hashed = binding.spconv_build_kmap(coords, 1, d, K, True)
    ref = oracle.build_kmap(coords_np, K, 1, d, True)
    a, b = kmap_to_numpy(dense), kmap_to_numpy(hashed)
    assert dense.n_out == ref["n_out"] and dense.total_pairs == len(ref["pair_in"])
    assert np.array_equal(a["oft"], ref["oft"]) and np.array_equal(a["out_coords"], coords_np)
    assert_kmaps_equal(canon(a), canon(ref))
    for key in a:                                    # the two builds differ in the table only
        assert np.array_equal(a[key], b[key]), key
    assert torch.equal(dense.tile_rows, hashed.tile_rows) and dense.tile_blocks == hashed.tile_blocks
    return dense, hashed


def test_config1_grid_64_cubed():
    cfg = wl.config(1)
    dense, hashed = _both(cfg["coords"], (1, 64, 64, 64))
    layer = cfg["layers"][0]
    x = wl.features(dense.n_in, layer["cin"], "f32", 0)
    w = wl.weights(27, layer["cin"], layer["cout"], "f32", 0)
    y1 = binding.spconv_forward(to_device(x, "f32"), to_device(w, "f32"), dense)
    y2 = binding.spconv_forward(to_device(x, "f32"), to_device(w, "f32"), hashed)
    assert torch.equal(y1, y2)
    ref = oracle.forward(x, w, np.ascontiguousarray(dense.nbr.cpu().numpy().T))
    assert rel_err(y1, ref) <= TOL["f32"]


@pytest.mark.parametrize("K,d", [(3, 1), (3, 2), (1, 1)])
def test_blob_in_a_128_cubed_grid_two_samples(K, d):
    """The largest grid the entry point takes (2 x 128^3 cells), a dense blob reaching its faces, shuffled rows."""
    blob = wl.random_blob(30000, 40, seed=3, batches=2)
    blob[:, 1:] += np.array([[0, 88, 0]], np.int32)       # push it against the y = 127 face
    edge = np.array([[0, 0, 0, 0], [1, 127, 127, 127], [0, 127, 0, 127], [1, 0, 127, 0]], np.int32)
    coords = np.unique(np.concatenate([blob, edge]), axis=0).astype(np.int32)
    assert coords[:, 1:].max() == 127 and coords[:, 1:].min() == 0
    dense, _ = _both(wl.shuffle_rows(coords, seed=5), (2, 128, 128, 128), K, d)
    assert dense.kvol == K ** 3


def test_dense_table_errors():
    E = binding.SpconvError
    ok = torch.tensor([[0, 1, 2, 3], [0, 1, 2, 4]], dtype=torch.int32, device="cuda")
    for bad_row in ([0, 8, 0, 0], [1, 0, 0, 0], [0, 0, 0, -1]):            # outside an 1 x 8 x 8 x 8 grid
        c = torch.tensor([[0, 1, 2, 3], bad_row], dtype=torch.int32, device="cuda")
        with pytest.raises(E) as e:
            binding.spconv_build_kmap_dense(c, (1, 8, 8, 8))
        assert e.value.status == 2
    dup = torch.tensor([[0, 1, 2, 3], [0, 4, 4, 4], [0, 1, 2, 3]], dtype=torch.int32, device="cuda")
    with pytest.raises(E) as e:
        binding.spconv_build_kmap_dense(dup, (1, 8, 8, 8))
    assert e.value.status == 3
    with pytest.raises(E) as e:                                             # more cells than the stated maximum
        binding.spconv_build_kmap_dense(ok, (4, 128, 128, 128))
    assert e.value.status == 9 and "maximum" in str(e.value)
    for kwargs in (dict(kernel_size=5), dict(kernel_size=2), dict(dilation=0)):
        with pytest.raises(E) as e:
            binding.spconv_build_kmap_dense(ok, (1, 8, 8, 8), **kwargs)
        assert e.value.status == 1
    with pytest.raises(E) as e:
        binding.spconv_build_kmap_dense(ok, (1, 8, 0, 8))
    assert e.value.status == 1
    km = binding.spconv_build_kmap_dense(ok, (1, 8, 8, 8))                  # the context still works
    assert km.n_out == 2 and km.total_pairs == 4
    empty = binding.spconv_build_kmap_dense(ok[:0].contiguous(), (1, 8, 8, 8))
    assert empty.n_out == 0
